/*
 * rslrl_b200 -- C ABI of the PPO learn-iteration hot path on one NVIDIA B200 (sm_100a).
 *
 * The paper (RSL-RL: A Learning Library for Robotics Research) describes the loop in its
 * section "Implementation Details": a Runner alternates environment stepping with agent
 * learning; the Algorithm is PPO (section "Features / Algorithms", after Schulman et al.
 * 2017) on MLP Networks; observations come in groups that are routed to different modules
 * (actor vs. privileged critic); environments use same-step reset and episodic time-outs
 * are handled properly; section "Auxiliary Techniques" adds mirrored-state augmentation with
 * an optional symmetry loss.  One learn iteration through this library is
 *
 *     for t in 0..T-1:   rslrl_act(obs_t)  ->  actions;   simulator steps;   rslrl_record_step(r, done, timeout)
 *     rslrl_gae(obs_T);   rslrl_ppo_update();
 *
 * Conventions
 *   - "d_" pointers are DEVICE pointers, "h_" pointers are HOST pointers.  Buffers passed in
 *     by the caller need the natural alignment of their element type (4 bytes for float)
 *     unless a call says otherwise, and must stay valid until the context's stream has
 *     executed the call.  Buffers owned by the library are 16-byte aligned.
 *   - All calls enqueue on the CUDA stream given to rslrl_create and return without a host
 *     synchronisation unless stated.  A context is not thread-safe.  In RSLRL_BF16 mode
 *     rslrl_ppo_update also uses a stream of its own for the minibatch gather and the
 *     shuffles; the caller's stream waits for everything enqueued there before the call
 *     returns, so work enqueued after the call is ordered behind all of the update's kernels.
 *   - Environment: RSLRL_SERIAL_LAUNCHES=1 switches programmatic dependent launch off.
 *   - Every function returns an rslrl_status; nothing throws, aborts or traps the device.
 *     Argument errors are found on the host before anything is launched.
 *     rslrl_last_error gives a human-readable message for the last failure of a context.
 *   - The library owns the context, the rollout storage, the parameters, the optimiser state
 *     and all scratch memory; it allocates them in rslrl_create and nowhere else.
 */
#ifndef RSLRL_B200_H
#define RSLRL_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RSLRL_OK = 0,
    RSLRL_ERR_INVALID_ARG = 1,   /* null pointer, negative size, unknown enum value           */
    RSLRL_ERR_SHAPE = 2,         /* e.g. T*N not divisible by the number of minibatches       */
    RSLRL_ERR_ALIGNMENT = 3,     /* a pointer does not have the alignment the call requires   */
    RSLRL_ERR_STATE = 4,         /* call order: act/record after T steps, gae before T steps  */
    RSLRL_ERR_UNSUPPORTED = 5,   /* a size beyond a documented limit                          */
    RSLRL_ERR_CUDA = 6,          /* a CUDA runtime call failed; see rslrl_last_error          */
    RSLRL_ERR_NONFINITE = 7,     /* a loss or gradient norm was not finite                    */
    RSLRL_ERR_TIMEOUT = 8        /* a bounded wait inside a kernel ran out; results since the
                                    last synchronising call are invalid; reported once         */
} rslrl_status;

/* Arithmetic of the hidden-layer matrix products.  Accumulation, bias, ELU, losses, master
 * weights, gradients and Adam are FP32 in every mode. */
typedef enum {
    RSLRL_FP32 = 0,              /* FP32 operands on the FP32 pipes                           */
    RSLRL_TF32 = 1,              /* FP32 storage; forward and data-gradient products on the
                                    tensor cores with TF32 operands, weight gradients on the
                                    FP32 pipes                                                 */
    RSLRL_BF16 = 2               /* BF16 operands on the tensor cores                         */
} rslrl_precision;

#define RSLRL_MAX_HIDDEN 8

/* Networks (paper: "Network architectures used by the algorithm"; MLPs, ELU hidden
 * activations, linear heads; diagonal Gaussian policy with a learned state-independent
 * log-std). */
typedef struct {
    int32_t num_envs;                         /* N                                             */
    int32_t num_steps;                        /* T                                             */
    int32_t actor_obs_dim;                    /* D_a                                           */
    int32_t critic_obs_dim;                   /* D_c                                           */
    int32_t num_actions;                      /* A  (1..64)                                    */
    int32_t shared_obs;                       /* 1: actor and critic read the same observation
                                                 (D_a == D_c); stored once                     */
    int32_t num_actor_hidden;                 /* 1..RSLRL_MAX_HIDDEN                           */
    int32_t actor_hidden[RSLRL_MAX_HIDDEN];
    int32_t num_critic_hidden;
    int32_t critic_hidden[RSLRL_MAX_HIDDEN];
    float   elu_alpha;                        /* 1.0                                           */
    int32_t precision;                        /* rslrl_precision                               */
} rslrl_model_cfg;

/* PPO hyper-parameters (Schulman et al. 2017, as named by the paper's "Algorithms"). */
typedef struct {
    float   gamma, lam;                       /* discount, GAE lambda                          */
    float   clip;                             /* surrogate clip range c                        */
    float   value_clip;                       /* value clip range c_v                          */
    float   value_coef;                       /* k_v                                           */
    float   entropy_coef;                     /* k_e                                           */
    int32_t use_clipped_value_loss;
    int32_t epochs, minibatches;              /* E, M; T*N must be divisible by M              */
    float   lr, lr_min, lr_max, lr_factor;    /* initial step size and the adaptive rule       */
    float   desired_kl;
    int32_t adaptive_lr;
    float   max_grad_norm;
    float   adam_b1, adam_b2, adam_eps;
    int32_t normalize_adv;                    /* normalise advantages inside rslrl_gae         */
    int32_t adv_std_unbiased;                 /* 1: divide the variance by B-1, 0: by B        */
    float   adv_eps;
    /* Symmetry augmentation (paper: "Auxiliary Techniques").  (S x)[i] = sign[i]*x[perm[i]].
     * HOST pointers, copied by rslrl_create; ignored when sym_enable == 0. */
    int32_t sym_enable;
    float   sym_coef;
    const int32_t *h_sym_obs_perm;  const float *h_sym_obs_sign;    /* [D_a] */
    const int32_t *h_sym_cobs_perm; const float *h_sym_cobs_sign;   /* [D_c] */
    const int32_t *h_sym_act_perm;  const float *h_sym_act_sign;    /* [A]   */
    uint64_t seed;                            /* keys the sampling noise and the shuffles      */
} rslrl_ppo_cfg;

/* Structure-of-arrays rollout storage (DEVICE pointers, owned by the context).  Every base
 * pointer is 16-byte aligned and every row stride is a multiple of 4 floats.  [t][n] arrays
 * are t-major so that consecutive environments are consecutive in memory. */
typedef struct {
    int32_t T, N;
    int32_t step;                             /* transitions recorded so far in this rollout   */
    int32_t obs_a_stride, obs_c_stride, act_stride;   /* row strides in floats                 */
    float  *obs_actor;                        /* [T][N][obs_a_stride]                          */
    float  *obs_critic;                       /* [T][N][obs_c_stride]; == obs_actor if shared  */
    float  *actions;                          /* [T][N][act_stride]                            */
    float  *mu;                               /* [T][N][act_stride]   policy mean at act time  */
    float  *sigma;                            /* [T][act_stride]      policy std  at act time  */
    float  *logp, *values, *rewards, *returns, *advantages;         /* [T][N]                  */
    uint8_t *dones, *timeouts;                /* [T][N] 0/1                                    */
} rslrl_storage;

/* Scalars of one rslrl_ppo_update call (means over its E*M minibatch steps, except where
 * stated). */
typedef struct {
    float   surrogate, value_loss, entropy, sym_loss, kl;
    float   first_surrogate, first_value_loss, first_kl, first_sym_loss;  /* first minibatch  */
    float   first_grad_norm, last_grad_norm;
    float   lr;                               /* learning rate after the call                  */
    int32_t steps;                            /* optimiser steps taken (E*M)                   */
    int32_t nonfinite;                        /* 1 if any loss / grad norm was not finite      */
} rslrl_update_stats;

typedef struct rslrl_ctx rslrl_ctx;

/* Number of FP32 parameters of the model, in the flat order
 *   actor  W1[in][out], b1, ..., Wout, bout, log_std[A],  critic W1, b1, ..., Wout, bout
 * with every W row-major [fan_in][fan_out].  Returns 0 on an invalid configuration. */
size_t rslrl_num_params(const rslrl_model_cfg *model);

/* Create a context on the current CUDA device.  `cuda_stream` is a cudaStream_t (NULL = the
 * legacy default stream).  Allocates storage, parameters (zero; log_std zero), optimiser state
 * and scratch.  Synchronises the stream once. */
rslrl_status rslrl_create(const rslrl_model_cfg *model, const rslrl_ppo_cfg *ppo,
                          void *cuda_stream, rslrl_ctx **out);
rslrl_status rslrl_destroy(rslrl_ctx *ctx);
const char  *rslrl_last_error(const rslrl_ctx *ctx);   /* ctx may be NULL: last create error  */

/* Borrowed view of the storage; pointers stay valid until rslrl_destroy. */
rslrl_status rslrl_storage_view(rslrl_ctx *ctx, rslrl_storage *out);

/* Parameters, last pre-clip gradient, Adam moments: HOST flat arrays of rslrl_num_params
 * floats.  These calls synchronise the stream. */
rslrl_status rslrl_set_params(rslrl_ctx *ctx, const float *h_flat, size_t n);
rslrl_status rslrl_get_params(rslrl_ctx *ctx, float *h_flat, size_t n);
rslrl_status rslrl_get_grads(rslrl_ctx *ctx, float *h_flat, size_t n);
rslrl_status rslrl_get_adam(rslrl_ctx *ctx, float *h_m, float *h_v, size_t n);
rslrl_status rslrl_set_adam(rslrl_ctx *ctx, const float *h_m, const float *h_v, size_t n);

/* Optimiser / counter state for checkpoint and resume.  set takes effect immediately. */
typedef struct {
    float    lr;                 /* current learning rate                                     */
    int32_t  adam_step;          /* optimiser steps taken so far                              */
    uint32_t global_step;        /* rslrl_act calls so far (indexes the sampling noise)       */
    uint32_t iteration;          /* rslrl_ppo_update calls so far (indexes the shuffles)      */
} rslrl_counters;
rslrl_status rslrl_get_counters(rslrl_ctx *ctx, rslrl_counters *out);
rslrl_status rslrl_set_counters(rslrl_ctx *ctx, const rslrl_counters *in);

/* (1) PPO rollout step (paper: "Algorithms", stochastic on-policy PPO; observation groups
 * routed to actor and critic).  For every environment n: mu = actor(o_a), V = critic(o_c),
 * a = mu + exp(log_std) * eps, eps ~ N(0,1) from Philox-4x32-10 keyed by the seed with counter
 * (n, global_step, action quad, 1), and the Gaussian log-density of a.  Writes row `step` of
 * the storage (observations, actions, mu, sigma, logp, values) and, if d_actions_out is not
 * NULL, the actions to d_actions_out[N][act_stride].
 *   d_actor_obs  [N][actor_obs_dim]  float32, dense rows (device)
 *   d_critic_obs [N][critic_obs_dim] float32 (device); with shared_obs it may be NULL or equal
 *                to d_actor_obs.
 * RSLRL_ERR_STATE if T steps were already taken in this rollout. */
rslrl_status rslrl_act(rslrl_ctx *ctx, const float *d_actor_obs, const float *d_critic_obs,
                       float *d_actions_out);

/* Record the simulator's answer to the last rslrl_act: rewards[N] float32, dones[N] and
 * timeouts[N] bytes (0/1; a time-out is also a done) -- device pointers.  Advances `step`. */
rslrl_status rslrl_record_step(rslrl_ctx *ctx, const float *d_rewards, const uint8_t *d_dones,
                               const uint8_t *d_timeouts);

/* (2) Returns and advantages (paper: "Implementation Details": proper handling of episodic
 * time-outs under same-step reset).  V_T = critic(o_T); reverse scan over t with A_T = 0:
 *     r~ = r_t + gamma V_t timeout_t;  delta = r~ + gamma V_{t+1} (1-done_t) - V_t
 *     A_t = delta + gamma lam (1-done_t) A_{t+1};   R_t = A_t + V_t
 * then, if normalize_adv, A <- (A - mean) / (std + adv_eps) over all T*N transitions.
 *   d_last_critic_obs [N][critic_obs_dim] float32 (device): the observation after the last step.
 * RSLRL_ERR_STATE unless exactly T steps were recorded. */
rslrl_status rslrl_gae(rslrl_ctx *ctx, const float *d_last_critic_obs);

/* (3) The minibatch PPO update (paper: "Algorithms" PPO; "Auxiliary Techniques" symmetry).
 * For E epochs: shuffle the T*N transitions with a keyed bijection, cut into M minibatches;
 * per minibatch: gather (plus mirrored copies when sym_enable), actor/critic forward, clipped
 * surrogate + clipped value loss - entropy bonus (+ symmetry loss), backward, KL(old||new) ->
 * adaptive learning rate, global grad-norm clip, Adam.  Starts a new rollout (step = 0).
 * If h_stats is not NULL the call synchronises the stream and fills it; otherwise it only
 * enqueues.  RSLRL_ERR_STATE unless rslrl_gae ran on this rollout. */
rslrl_status rslrl_ppo_update(rslrl_ctx *ctx, rslrl_update_stats *h_stats);

/* Variant of rslrl_ppo_update that stops after `max_steps` minibatch steps (tests compare the
 * state after exactly one optimiser step).  max_steps <= 0 means all E*M steps. */
rslrl_status rslrl_ppo_update_steps(rslrl_ctx *ctx, int32_t max_steps, rslrl_update_stats *h_stats);

/* Distillation step (paper: "Algorithms", the behaviour-cloning algorithm similar to DAgger: roll out the
 * student, relabel its data with expert actions, train the student on it).  The student is this
 * context's actor net; the rollout is the T steps collected with rslrl_act / rslrl_record_step
 * (rslrl_gae is not needed).  For E epochs over the same keyed minibatches as rslrl_ppo_update:
 * gather, actor forward, L = mean over rows and actions of (mu - a_expert)^2 (the paper names no
 * loss), backward, global grad-norm clip, Adam with the current learning rate (no KL rule).  The
 * critic and log_std receive a zero gradient.  Starts a new rollout (step = 0).
 *   d_expert_actions [T][N][act_stride] float32 (device), act_stride as in rslrl_storage; columns
 *   at and beyond num_actions are ignored.
 * Stats: surrogate / first_surrogate carry L; value_loss, kl, sym_loss are 0.
 * RSLRL_ERR_STATE unless exactly T steps were recorded; RSLRL_ERR_UNSUPPORTED with sym_enable. */
rslrl_status rslrl_distill_update(rslrl_ctx *ctx, const float *d_expert_actions, rslrl_update_stats *h_stats);
/* The same, stopping after `max_steps` minibatch steps (max_steps <= 0: all). */
rslrl_status rslrl_distill_update_steps(rslrl_ctx *ctx, const float *d_expert_actions, int32_t max_steps,
                                        rslrl_update_stats *h_stats);

/* Host-buffer variants of the per-step calls: the same work with the host<->device copies
 * inside the call (pinned host memory makes them asynchronous).  h_actions_out[N][A] dense;
 * when it is not NULL the call waits for the actions. */
rslrl_status rslrl_act_host(rslrl_ctx *ctx, const float *h_actor_obs, const float *h_critic_obs,
                            float *h_actions_out);
rslrl_status rslrl_record_step_host(rslrl_ctx *ctx, const float *h_rewards, const uint8_t *h_dones,
                                    const uint8_t *h_timeouts);
rslrl_status rslrl_gae_host(rslrl_ctx *ctx, const float *h_last_critic_obs);

/* Stand-alone pieces of the path on caller-owned DEVICE buffers (used for size sweeps and
 * roofline measurements; same kernels as the context calls).
 *
 * rslrl_gae_scan: the reverse scan and normalisation of (2) on [T][N] arrays, V_T given.
 *   d_scratch: at least rslrl_gae_scratch_bytes(T, N) bytes of device memory; d_advantages and
 *   d_scratch must be 16-byte aligned.
 * rslrl_minibatch_indices: row indices of minibatch k of `epoch` (the keyed Feistel shuffle of
 *   B = T*N rows cut into M chunks): d_rows_out[B/M] int32. */
size_t       rslrl_gae_scratch_bytes(int32_t T, int32_t N);
rslrl_status rslrl_gae_scan(const float *d_rewards, const float *d_values, const uint8_t *d_dones,
                            const uint8_t *d_timeouts, const float *d_last_values,
                            float *d_returns, float *d_advantages, int32_t T, int32_t N,
                            float gamma, float lam, int32_t normalize, int32_t unbiased,
                            float adv_eps, void *d_scratch, void *cuda_stream);
rslrl_status rslrl_minibatch_indices(uint64_t seed, uint32_t iteration, uint32_t epoch,
                                     int32_t batch, int32_t minibatches, int32_t k,
                                     int32_t *d_rows_out, void *cuda_stream);

/* rslrl_gae_scan without any allocation.  (The paper has no counterpart: this is an addition
 * for embedding the library, not a step of the method.)
 *
 * Meant for callers that cannot obtain device memory while they run -- a plug-in living inside
 * a simulator that owns the whole device pool, a fixed-period control loop that may not risk
 * the device-wide stall or the failure of an allocation, a process under a fixed memory
 * budget -- and so cannot supply the scratch buffer rslrl_gae_scan asks for.  The scratch sits
 * in a fixed array inside the library image instead (96 KiB per GPU that loads the library,
 * held until the process exits); the call itself allocates and frees nothing.
 *   - Same arguments, results and alignment rule as rslrl_gae_scan, minus d_scratch.
 *   - N may not exceed RSLRL_GAE_STATIC_MAX_ENVS: a larger N returns RSLRL_ERR_UNSUPPORTED and
 *     rslrl_last_error(NULL) says so; nothing is launched.
 *   - The first call on a device looks up the array's device address (once per device, with
 *     that device current); the CUDA runtime may load the part of the library that holds the
 *     array at that moment, which is the one point where this entry point can touch device
 *     memory management.  Make that first call during start-up, before any stream capture and
 *     before memory gets tight: a call with T = 0 or N = 0 does the lookup and nothing else.
 *     While the library's per-kernel profiling is switched on (rslrl_profile_enable) a call also
 *     creates CUDA events; leave profiling off where that matters.
 *   - Every call on a device uses the same array, which keeps what the previous call left in
 *     it.  The call needs nothing in it to start at zero, but two calls that overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them. */
#define RSLRL_GAE_STATIC_MAX_ENVS 1048576
rslrl_status rslrl_gae_scan_static(const float *d_rewards, const float *d_values, const uint8_t *d_dones,
                                   const uint8_t *d_timeouts, const float *d_last_values,
                                   float *d_returns, float *d_advantages, int32_t T, int32_t N,
                                   float gamma, float lam, int32_t normalize, int32_t unbiased,
                                   float adv_eps, void *cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Checking build.  Compiled with -DRSLRL_DEBUG the library (a) places every device allocation
 * between two 256-byte guard regions of a fixed pattern and (b) checks, in the kernels that index
 * through data they read (the shuffled row numbers of the minibatch gather, the row numbers and
 * the selected entries of the RND subset), that the index is in range; an index that is not is
 * replaced by 0 and recorded in a device flag.  Nothing traps and no access leaves its buffer
 * through these indices.  rslrl_debug_report, to be called between steps, synchronises the device
 * and writes (each pointer is host memory and may be NULL):
 *   h_debug_build     1 in the checking build, 0 otherwise (the other two are then always 0)
 *   h_damaged_guards  number of guard regions whose pattern was overwritten (an out-of-bounds write
 *                     next to an allocation): over all live allocations of the process, plus those
 *                     found damaged when their allocation was freed (these stay counted)
 *   h_index_fault     0, or the code of the worst index recorded since the last report (1 = a
 *                     minibatch row number, 2 = an RND row number, 3 = an RND entry index);
 *                     reading clears it.
 * Returns RSLRL_ERR_CUDA if the device reports an error. */
rslrl_status rslrl_debug_report(int32_t *h_debug_build, int32_t *h_damaged_guards, int32_t *h_index_fault);

/* ---------------------------------------------------------------------------------------------
 * Random network distillation on a subset of the state (paper: "Auxiliary Techniques", the
 * curiosity-driven intrinsic reward computed on selected states only).
 *
 * Two MLPs of the same shape read s = o[idx] (num_idx selected entries of an observation row):
 * a target g with fixed random weights and a predictor f.  Intrinsic reward of a row:
 *   r_int = (1/E) sum_j (f_j(s) - g_j(s))^2          (E = embed_dim)
 * rslrl_rnd_reward adds weight * r_int to a reward vector; rslrl_rnd_update regresses f on g
 * (loss = mean over the minibatch rows of r_int) with Adam at a fixed learning rate, over the
 * same kind of keyed minibatches as rslrl_ppo_update.  With precision RSLRL_FP32 all arithmetic is FP32; with
 * RSLRL_TF32 the matrix products of both nets (forward, data and weight gradients) run on the tensor cores with
 * TF32 operands read from the same FP32 buffers, everything else stays FP32 (tolerance class 5e-3).  (Observation
 * normalisation and reward-weight schedules, which the paper's library offers around this, are
 * left to the caller.)
 *
 * An rslrl_rnd owns its parameters, Adam moments and work buffers (device memory, all of it
 * allocated by rslrl_rnd_create from the limits in the config: no later call allocates); calls on one
 * object are not thread-safe; all work is enqueued on the stream given at creation.
 * Parameter vectors (host, float32) are in the order W1[in][out], b1, W2, b2, ... for the
 * layers num_idx -> hidden[0] -> ... -> embed_dim; hidden layers use ELU(alpha). */
typedef struct rslrl_rnd rslrl_rnd;

typedef struct {
    int32_t obs_dim;                    /* entries of an observation row; idx values are < obs_dim   */
    int32_t num_idx;                    /* 1..obs_dim                                                */
    const int32_t *h_idx;               /* [num_idx] host; copied                                    */
    int32_t num_hidden;                 /* 1..RSLRL_MAX_HIDDEN                                       */
    int32_t hidden[RSLRL_MAX_HIDDEN];
    int32_t embed_dim;                  /* E >= 1                                                    */
    float   elu_alpha;
    int32_t max_rows;                   /* largest `rows` of rslrl_rnd_reward and largest minibatch  */
    float   lr, adam_b1, adam_b2, adam_eps;
    int32_t max_batch;                  /* largest `batch` of rslrl_rnd_update (>= 1)                */
    int32_t max_epochs;                 /* largest `epochs` of rslrl_rnd_update (>= 1)               */
    int32_t max_minibatches;            /* largest `minibatches` of rslrl_rnd_update (>= 1)          */
    int32_t precision;                  /* RSLRL_FP32 or RSLRL_TF32 (RSLRL_BF16: RSLRL_ERR_UNSUPPORTED) */
} rslrl_rnd_cfg;

size_t       rslrl_rnd_num_params(const rslrl_rnd_cfg *cfg);      /* of one net; 0 if cfg is invalid */
rslrl_status rslrl_rnd_create(const rslrl_rnd_cfg *cfg, void *cuda_stream, rslrl_rnd **out);
rslrl_status rslrl_rnd_destroy(rslrl_rnd *rnd);
const char  *rslrl_rnd_last_error(const rslrl_rnd *rnd);          /* NULL: last create error         */
/* Host vectors of rslrl_rnd_num_params floats; set also zeroes the Adam moments and step count.
 * These calls synchronise the stream. */
rslrl_status rslrl_rnd_set_params(rslrl_rnd *rnd, const float *h_predictor, const float *h_target, size_t n);
rslrl_status rslrl_rnd_get_params(rslrl_rnd *rnd, float *h_predictor, size_t n);
rslrl_status rslrl_rnd_get_grads(rslrl_rnd *rnd, float *h_grad, size_t n);   /* of the last step     */

/* d_obs [rows][obs_stride] float32 (device), rows <= max_rows, obs_stride >= obs_dim.
 * d_rewards_inout [rows] (device, may be NULL): += weight * r_int.  d_r_int_out [rows] (device,
 * may be NULL): = r_int.  Only enqueues. */
rslrl_status rslrl_rnd_reward(rslrl_rnd *rnd, const float *d_obs, int32_t rows, int32_t obs_stride,
                              float weight, float *d_rewards_inout, float *d_r_int_out);

/* Predictor training on d_obs [batch][obs_stride]: for `epochs` epochs, shuffle the rows with
 * the keyed bijection of (seed, iteration, epoch), cut into `minibatches` chunks (batch must be
 * divisible; batch / minibatches <= max_rows), one Adam step per chunk; stops after max_steps
 * steps if max_steps > 0.  h_mean_loss (host, may be NULL): mean of the step losses, which makes
 * the call synchronise; h_first_loss likewise for the first step.
 * RSLRL_ERR_SHAPE for an indivisible batch, RSLRL_ERR_UNSUPPORTED beyond max_rows, max_batch,
 * max_epochs or max_minibatches. */
rslrl_status rslrl_rnd_update(rslrl_rnd *rnd, const float *d_obs, int32_t batch, int32_t obs_stride,
                              int32_t epochs, int32_t minibatches, uint64_t seed, uint32_t iteration,
                              int32_t max_steps, float *h_mean_loss, float *h_first_loss);

/* ---------------------------------------------------------------------------------------------
 * Recurrent memory layer (paper: "Implementation Details": recurrent networks through explicit
 * management of hidden states across rollouts and back-propagation through time).
 *
 * A GRU layer over a time-major rollout.  Per step t (gate order r, z, n):
 *   h_in(t) = (1 - reset) * h0 for t = 0, else (1 - done[t-1]) * h(t-1)   (same-step reset: zero state after done)
 *   r = sigmoid(x_t W_ir + b_ir + h_in W_hr + b_hr),  z likewise,
 *   n = tanh(x_t W_in + b_in + r * (h_in W_hn + b_hn)),  h(t) = (1 - z) n + z h_in
 * The paper names neither the cell nor the reset rule; these are this library's choices.
 * Parameters (host, float32): W_i[D][3H], b_i[3H], W_h[H][3H], b_h[3H], in this order.
 * With precision RSLRL_FP32 all arithmetic is FP32.  With RSLRL_TF32 the matrix products (input and state
 * products, their data gradients, the weight gradients) run on the tensor cores with TF32 operands read from
 * the same FP32 buffers and FP32 accumulation; gates, biases' gradients and everything else stay FP32
 * (tolerance class 5e-3 instead of 1e-4).  The object owns parameters, gradient and work buffers sized for
 * max_steps x max_envs; calls on one object are not thread-safe and enqueue on its stream. */
typedef struct rslrl_gru rslrl_gru;

typedef struct {
    int32_t input_dim;                  /* D >= 1                                                    */
    int32_t hidden_dim;                 /* H, a multiple of 4                                        */
    int32_t max_steps;                  /* largest T                                                 */
    int32_t max_envs;                   /* largest N; T * N < 2^30 and N * 3H < 2^31                 */
    int32_t precision;                  /* RSLRL_FP32 or RSLRL_TF32 (RSLRL_BF16: RSLRL_ERR_UNSUPPORTED) */
} rslrl_gru_cfg;

size_t       rslrl_gru_num_params(const rslrl_gru_cfg *cfg);      /* 0 if cfg is invalid             */
rslrl_status rslrl_gru_create(const rslrl_gru_cfg *cfg, void *cuda_stream, rslrl_gru **out);
rslrl_status rslrl_gru_destroy(rslrl_gru *gru);
const char  *rslrl_gru_last_error(const rslrl_gru *gru);          /* NULL: last create error         */
rslrl_status rslrl_gru_set_params(rslrl_gru *gru, const float *h_params, size_t n);   /* synchronises */
rslrl_status rslrl_gru_get_grads(rslrl_gru *gru, float *h_grad, size_t n);            /* synchronises */

/* Forward over T steps of N environments (device pointers, float buffers 16-byte aligned):
 *   d_x [T][N][x_stride] (x_stride a multiple of 4, >= D rounded up to 4; padding is not read as data),
 *   d_h0 [N][H] the state carried in, d_h0_reset [N] uint8 (may be NULL): environments whose step before
 *   this call reported done and therefore start from the zero state (with it, T calls of one step each
 *   give the states of one call of T steps), d_dones [T][N] uint8, d_h_out [T][N][H] = h(t).
 * d_x, d_dones and d_h0_reset must stay unchanged until rslrl_gru_backward has run.  Only enqueues. */
rslrl_status rslrl_gru_forward(rslrl_gru *gru, const float *d_x, int32_t x_stride, const float *d_h0,
                               const uint8_t *d_h0_reset, const uint8_t *d_dones, int32_t T, int32_t N,
                               float *d_h_out);

/* Back-propagation through the T steps of the last forward for L = sum_t <d_dh[t], h(t)>:
 *   d_dh [T][N][H]; d_dx [T][N][dx_stride] (may be NULL) = dL/dx; d_dh0 [N][H] (may be NULL) = dL/dh0
 *   (zero in the rows d_h0_reset flagged);
 * the parameter gradient is kept in the object (rslrl_gru_get_grads).  No gradient crosses a reset.
 * One backward per forward: RSLRL_ERR_STATE otherwise.  Only enqueues. */
rslrl_status rslrl_gru_backward(rslrl_gru *gru, const float *d_dh, float *d_dx, int32_t dx_stride, float *d_dh0);

/* Number of kernels this library has launched in the current process (all contexts). */
uint64_t     rslrl_kernel_launch_count(void);

/* Per-kernel timing for roofline reports.  While enabled, every kernel launch of the library
 * is bracketed by a pair of CUDA events on its stream (this slows the host side down; leave
 * it off when measuring throughput).  rslrl_profile_report waits for the recorded launches,
 * writes one line "family launches total_ms" per kernel family into h_text (NUL-terminated,
 * RSLRL_ERR_UNSUPPORTED if capacity is too small) and forgets them. */
rslrl_status rslrl_profile_enable(int32_t on);
rslrl_status rslrl_profile_report(char *h_text, size_t capacity);

#ifdef __cplusplus
}
#endif
#endif /* RSLRL_B200_H */
