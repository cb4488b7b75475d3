// Host-side launchers of the rslrl_b200 kernels (internal; the public boundary is
// include/rslrl_b200.h).  Every launcher enqueues on `stream` and returns the CUDA status of
// the launch.
#pragma once
#include <utility>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace rslrl {

// Counts one kernel launch; while profiling is on it also brackets the launch with CUDA events
// on `stream` so that the time of every kernel family can be reported.
struct LaunchScope {
    LaunchScope(const char* name, cudaStream_t stream);
    ~LaunchScope();
    const char* name; cudaStream_t stream; int slot;
};

// Brackets a run of consecutive launches of one kernel family with ONE event pair while profiling is on
// (the launches inside are counted, not bracketed), so that their dependent-launch overlap is kept.
struct FamilyScope {
    FamilyScope(const char* name, cudaStream_t stream);
    ~FamilyScope();
    cudaStream_t stream; int slot;
};

// Launch of a kernel that begins with chain_begin(): it may be scheduled before the preceding kernel
// of the stream has drained (programmatic stream serialisation), which hides launch latency and
// prologue.  Falls back to a plain launch when chained launches are switched off.
bool chained_launches_enabled();
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = chained_launches_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// ------------------------------------------------------------------------- SIMT FP32 GEMM
// C[M x N] = op(A)[M x K] * op(B)[K x N] followed by an epilogue.  Leading dimensions are
// multiples of 4 floats and base pointers 16-byte aligned.
enum GemmEpilogue {
    EPI_BIAS_ELU = 0,   // C = ELU(acc + bias[n]); columns [N, Cn) are written as 0
    EPI_BIAS = 1,       // C = acc + bias[n]
    EPI_DELU = 2,       // C = acc * ELU'(aux[m][n])        (aux = stored post-activation)
    EPI_PLAIN = 3       // C = acc                           (split partial of a weight gradient)
};

struct GemmProblem {
    const float* A; const float* B; float* C;
    const float* bias; const float* aux;
    int lda, ldb, ldc, ldaux;
    int M, N, K;
    int Cn;                 // columns written per row (N <= Cn <= ldc)
    int splits;             // the K range is cut into `splits` chunks of `kchunk`
    int kchunk;
    long long split_stride; // distance in floats between the C of consecutive splits
};

constexpr int kMaxGemmBatch = 8;
struct GemmBatch {
    GemmProblem p[kMaxGemmBatch];
    int count;
    float alpha;            // ELU alpha
};

// transA: A(m,k) = A[k*lda + m] instead of A[m*lda + k]; transB: B(k,n) = B[n*ldb + k].
cudaError_t launch_sgemm(const GemmBatch& b, bool transA, bool transB, int epilogue,
                         cudaStream_t stream);

// Column sums of X[rows][ld] over a split of the rows: out[s * split_stride + n].
constexpr int kMaxColsum = 16;
struct ColsumProblem { const void* X; float* out; int rows, n, ld; };
struct ColsumBatch { ColsumProblem p[kMaxColsum]; int count; int splits; long long split_stride; int is_bf16; };
cudaError_t launch_colsum(const ColsumBatch& b, cudaStream_t stream);

// ------------------------------------------------------------------------- rollout kernels
// dst[n][dst_ld] <- src[n][dim] (zero padded), optionally a second destination in bf16.
cudaError_t launch_pad_rows(const float* src, int dim, float* dst, int dst_ld,
                            __nv_bfloat16* dst16, int dst16_ld, int rows, cudaStream_t stream);

struct HeadParams {                 // final linear layers of actor and critic
    const float* Wa; const float* ba; int ldwa;      // [n_a][ldwa], ldwa = round4(A)
    const float* Wc; const float* bc; int ldwc;      // [n_c][ldwc], ldwc = 4
    const float* log_std;
    int n_a, n_c, A;                                  // widths of the last hidden layers
};

struct ActOut {
    float* actions; float* mu; float* sigma; float* logp; float* values;   // storage row t
    float* actions_out;                                                    // may be null
    int act_stride;
};
// Head + Gaussian sample + log-density for N rows; hidden activations are float or bf16.
cudaError_t launch_act_head(const void* Ha, int ldha, const void* Hc, int ldhc, bool bf16_act,
                            const HeadParams& hp, const ActOut& out, int N, uint64_t seed,
                            uint32_t global_step, cudaStream_t stream);
// Critic head only: values[N].
cudaError_t launch_value_head(const void* Hc, int ldhc, bool bf16_act, const HeadParams& hp,
                              float* values, int N, cudaStream_t stream);

cudaError_t launch_record_step(const float* rew, const uint8_t* dones, const uint8_t* timeouts,
                               float* s_rew, uint8_t* s_dones, uint8_t* s_timeouts, int N,
                               cudaStream_t stream);

// GAE reverse scan + block moments; then normalisation.  scratch: 3 floats per scan block.
int gae_scan_blocks(int N);
cudaError_t launch_gae(const float* rewards, const float* values, const uint8_t* dones,
                       const uint8_t* timeouts, const float* last_values, float* returns,
                       float* advantages, int T, int N, float gamma, float lam, int normalize,
                       int unbiased, float adv_eps, float* scratch, cudaStream_t stream);

// ------------------------------------------------------------------------- update kernels
struct SymTables {                  // device pointers; null when symmetry is off
    const int* obs_perm; const float* obs_sign;
    const int* cobs_perm; const float* cobs_sign;
    const int* act_perm; const float* act_sign;
};

struct GatherArgs {
    // storage
    const float* obs_a; const float* obs_c; const float* actions; const float* mu;
    const float* sigma; const float* logp; const float* values; const float* returns;
    const float* adv;
    int N, B, sa, sc, as, Da, Dc, A;                        // B = T * N transitions in storage
    int shared_obs;
    // minibatch destination (rows [0,Bmb) originals, [Bmb,2Bmb) mirrored when sym)
    float* x_a; float* x_c; int ldxa, ldxc;                 // fp32 (null in bf16 mode)
    __nv_bfloat16* x_a16; __nv_bfloat16* x_c16; int ldxa16, ldxc16;
    float* act_mb; float* mu_old; float* sigma_old;         // [R][as], [Bmb][as], [Bmb][as]
    float* logp_old; float* v_old; float* ret; float* adv_mb;   // [Bmb]
    const int* rows;                                        // [Bmb] source transition of every minibatch row
    int Bmb; int sym;
    SymTables st;
};
cudaError_t launch_gather(const GatherArgs& a, cudaStream_t stream, bool alone = false);
cudaError_t launch_perm_rows(uint64_t seed, uint32_t iteration, uint32_t epoch, uint32_t batch,
                             uint32_t first, int count, int* rows_out, cudaStream_t stream);
// The shuffles of epochs 0 .. epochs-1 of one iteration in one launch: rows_out[epoch][batch].
cudaError_t launch_perm_epochs(uint64_t seed, uint32_t iteration, int epochs, uint32_t batch, int* rows_out,
                               cudaStream_t stream);

struct LossHyper {
    float clip, value_clip, value_coef, entropy_coef, sym_coef, alpha;
    int use_clipped_value_loss;
};

// Slots of the loss sums; slot LS_COUNT holds the policy entropy.
enum { LS_SURR = 0, LS_VALUE = 1, LS_KL = 2, LS_SYM = 3, LS_COUNT = 4 };

struct HeadLossArgs {
    const void* Ha; const void* Hc; int ldha, ldhc; int bf16_act;
    HeadParams hp;
    const float* act_mb; const float* mu_old; const float* sigma_old; int as;
    const float* logp_old; const float* v_old; const float* ret; const float* adv;
    const float* act_sign; const int* act_perm;       // mirror of actions (null when sym off)
    int Bmb; int sym;
    int distill;                    // 1: act_mb holds expert actions and the loss is the mean squared error between the
                                    // policy mean and them (no critic, log_std, KL terms); its row sum lands in LS_SURR
    LossHyper h;
    // outputs
    float* dmu; int lddmu;          // [R][round4(A)]   fp32
    float* dv;                      // [R][4]  column 0 = dL/dV, columns 1..3 zero
    __nv_bfloat16* dmu16; int lddmu16; __nv_bfloat16* dv16; int lddv16;   // bf16 twins (may be null)
    void* dZa; void* dZc; int lddza, lddzc;           // dL/dz of the last hidden layers
    float* block_partials;          // [blocks][head_partial_stride()]  (losses, db_head, dlog_std)
    float* mu_out; float* v_out;    // optional copies of mu [R][as] and V [R] (may be null)
    int nblocks_used;               // set by the launcher: rows of block_partials that were written
    // optional (tensor-core head kernel only): per-block column sums of dZa / dZc, i.e. partial bias
    // gradients of the last hidden layers, [blocks][lddza] and [blocks][lddzc]
    float* colsum_a; float* colsum_c;
    int colsum_written;             // set by the launcher: 1 when those rows were produced
};
int head_loss_blocks(int Bmb);      // upper bound of nblocks_used (for sizing block_partials)
int head_partial_stride();
cudaError_t launch_head_loss(HeadLossArgs& a, cudaStream_t stream);
// BF16 activations: the heads and dL/dz on warp-level tensor-core instructions.
bool head_loss_mma_applicable(const HeadLossArgs& a);
cudaError_t launch_head_loss_mma(HeadLossArgs& a, cudaStream_t stream);

// A run of parameters (hidden-layer biases) whose gradient is the sum of `nslots` partial rows
// produced by the kernels that emit dZ, instead of the split partials.
struct BiasSource { int p_off, n; const float* slots; int nslots, ld; };
constexpr int kMaxBiasSources = 16;

struct ReduceArgs {
    const float* partials; int splits; long long split_stride;   // gradient partials [splits][P]
    float* grad; int P;                                            // padded device layout
    float* sumsq_partials;          // [reduce_blocks(P)]
    // head_loss block partials: the head-bias and log_std gradients and the loss sums are
    // finished here (loss sums -> loss_sums[0..LS_COUNT), entropy -> loss_sums[LS_COUNT])
    const float* block_partials; int nblocks;
    int off_ba, off_logstd, off_bc, A;
    float entropy_coef; const float* log_std; float* loss_sums;
    int n_bias; BiasSource bias[kMaxBiasSources];
};
int reduce_blocks(int P);
cudaError_t launch_reduce(const ReduceArgs& a, cudaStream_t stream);

// One hidden layer's low-precision operand copies (see the tensor-core engine).
struct CvtRange {
    int w_off, b_off, in, out, out_p;          // location in the padded FP32 parameter vector
    __nv_bfloat16* wt; int ld_wt;               // [out][ld_wt]
    __nv_bfloat16* wn; int ld_wn;               // [in][ld_wn], may be null
    __nv_bfloat16* wt_lo;                       // [out][ld_wt] what BF16 rounding left of the weight, may be null
    float* bias_pad;                            // [>= out] zero-padded FP32 bias copy
};
constexpr int kMaxCvt = 16;

struct AdamArgs {
    float* param; float* m; float* v; const float* grad; int P;
    const float* sumsq_partials; int nsumsq;
    const float* loss_sums;
    float inv_rows_all, inv_rows_orig, inv_sym;      // 1/R, 1/Bmb, 1/(Bmb*A)
    float* lr_io;                   // [2] double-buffered learning rate
    int* step_io;                   // [2] double-buffered optimiser step count
    int parity;                     // which slot is current
    float lr_min, lr_max, lr_factor, desired_kl; int adaptive;
    float max_norm, b1, b2, eps;
    float* stats_row;               // [8]: surr, value, entropy, sym, kl, grad_norm, lr, nonfinite
    // BF16 mode: the operand copies of the weights are refreshed by the same pass
    int n_cvt; CvtRange cvt[kMaxCvt];
};
cudaError_t launch_adam(const AdamArgs& a, cudaStream_t stream);

}  // namespace rslrl
