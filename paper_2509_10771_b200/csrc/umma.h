// Tensor-core engine (RSLRL_BF16): hidden-layer products of act, forward and backward on
// tcgen05 tiles fed by TMA, with FP32 accumulation in tensor memory.
#pragma once
#include "../../include/rslrl_b200.h"
#include "common.cuh"
#include "kernels.h"
#include <string>

namespace rslrl {

struct UmmaSetup {
    rslrl_model_cfg model;
    int N, Bmb, R;                 // rollout rows per act call, minibatch rows, rows incl. mirrored
    cudaStream_t stream;
    float* param; int P_dev;       // FP32 master parameters (padded device layout)
    float* partials; int splits;   // weight-gradient partials [splits][P_dev]
    int nl[2], in_dim[2];          // layers per net (head included), observation widths
    int in[2][kMaxLayers], out[2][kMaxLayers], out_p[2][kMaxLayers];
    size_t w_off[2][kMaxLayers], b_off[2][kMaxLayers];
    size_t logstd_off;
};

struct UmmaEngine;

UmmaEngine* umma_create(const UmmaSetup& s, std::string* err);
void umma_destroy(UmmaEngine* e);
// Splits of the contraction per weight-gradient problem [net][layer] (head = last layer) and their
// maximum, which is the number of partial rows the gradient buffer needs.
struct WgradPlan { int splits[2][kMaxLayers]; int max_splits; };
WgradPlan umma_wgrad_plan(const UmmaSetup& s);
// Re-derive the low-precision operand copies of the weights from the FP32 masters (after
// rslrl_set_params; the optimiser step refreshes them itself, see umma_fill_cvt).
cudaError_t umma_refresh_weights(UmmaEngine* e);
// Tell the Adam kernel where the operand copies of every hidden layer live.
void umma_fill_cvt(UmmaEngine* e, AdamArgs* a);
// Tell the gradient reduction which hidden-layer bias gradients arrive as partial rows written by
// the data-gradient epilogue and, when hl.colsum_written, by the head/loss kernel.
void umma_fill_bias_sources(UmmaEngine* e, ReduceArgs* r, const HeadLossArgs& hl);
// Hidden layers on N rollout rows.  d_obs_* are dense [N][dim] FP32 rows; when store_* is not
// null the padded FP32 copy of the observations is also written there (row strides sa / sc).
// Returns the last hidden activations of both nets (actor's only when do_actor).  Where the
// fused kernel applies the heads run in the same launch: it samples the actions (do_actor) and
// writes the rollout outputs named by `out` (values only when !do_actor) and sets *heads_done.
cudaError_t umma_act_forward(UmmaEngine* e, const float* d_obs_a, const float* d_obs_c, float* store_a,
                             float* store_c, int sa, int sc, bool do_actor, const ActOut& out,
                             const float* log_std, uint64_t seed, uint32_t global_step, bool* heads_done,
                             const void** ha, int* ldha, const void** hc, int* ldhc);
// Point the gather at one of the engine's two minibatch input buffers (buf = 0 or 1); the forward
// and backward launches take the same index.  With two buffers the gather of the next minibatch
// can run while the current one is worked on.
void umma_gather_targets(UmmaEngine* e, GatherArgs* g, int buf);
// actor_only (distillation): the critic's launches are left out; umma_zero_critic_gradients, once before the
// first such step, zeroes what its data-gradient launches would have written, so that the weight-gradient
// launch (which still covers both nets) yields a zero critic gradient.
cudaError_t umma_update_forward(UmmaEngine* e, int buf, bool actor_only);
cudaError_t umma_zero_critic_gradients(UmmaEngine* e);
// Point the head/loss kernel at the engine's last hidden activations and dZ buffers.
void umma_head_loss_targets(UmmaEngine* e, HeadLossArgs* a);
// Data gradients, weight-gradient partials and bias-gradient partials of all hidden layers
// and heads, from the dZ / d_head buffers the head/loss kernel filled.  last_bias_done: the
// head/loss kernel already produced the bias-gradient partials of the last hidden layers.
cudaError_t umma_update_backward(UmmaEngine* e, bool last_bias_done, int buf, bool actor_only);
// Synchronises the stream and returns the device error code (0 = none; otherwise the role
// whose bounded wait expired); a non-zero code is cleared once it has been read.
cudaError_t umma_read_error(UmmaEngine* e, int* host_code);

}  // namespace rslrl
