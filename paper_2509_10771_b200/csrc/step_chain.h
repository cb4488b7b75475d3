// Row-local part of a minibatch step as ONE kernel (RSLRL_BF16, no mirrored rows): for every
// 128-row tile and net, all hidden layers forward, the head, the PPO loss terms and their
// gradient, and the data gradients back to the first hidden layer, with the activations of a
// tile staying in shared memory between the layers.  What the weight-gradient kernel needs
// afterwards (post-activations, dL/dz of every layer, the head gradient) is written to global
// memory once on the way.
#pragma once
#include "common.cuh"
#include "kernels.h"
#include <string>

namespace rslrl {

constexpr int kStepChainLayers = 4;       // hidden layers per net the kernel can chain

struct StepChainNet {
    int nh;                               // hidden layers
    int kp;                               // padded observation width (multiple of 64)
    int pw[kStepChainLayers];             // padded hidden widths (multiples of 64)
    int is_actor, A;                      // head: A outputs (1 for the critic)
    const __nv_bfloat16* x16;             // [rows][kp] minibatch observations
    const __nv_bfloat16* wt[kStepChainLayers];   // [pw l][k in]  forward operands
    const __nv_bfloat16* wn[kStepChainLayers];   // [pw l-1][pw l] data-gradient operands (l >= 1)
    const __nv_bfloat16* wht;             // [64][pw last]  head weights, output-major (rows >= A zero)
    const __nv_bfloat16* whn;             // [pw last][64]  head weights, input-major
    const float* bias_pad[kStepChainLayers];     // zero-padded hidden biases
    const float* head_bias;               // [64] zero-padded head bias
    __nv_bfloat16* h[kStepChainLayers];   // [rows][pw l] post-activations (out)
    __nv_bfloat16* dz[kStepChainLayers];  // [rows][pw l] dL/dz (out)
    __nv_bfloat16* dhead16;               // [rows][64] dL/d(head output) (out)
    float* colsum[kStepChainLayers];      // [4 * row tiles][pw l] column sums of dz per 32-row slice (out)
};

struct StepChainSetup {
    int rows;
    StepChainNet net[2];                  // actor, critic
    const float* log_std;                 // [A] of the actor
    float alpha;
    int* error;                           // device flag raised when a bounded wait expires
    int num_sms;
};

struct StepChainLoss {
    const float* act_mb; const float* mu_old; const float* sigma_old; int as;   // [rows][as]
    const float* logp_old; const float* v_old; const float* ret; const float* adv;   // [rows]
    float clip, value_clip, value_coef; int use_clipped_value_loss;
    float* block_partials;                // [blocks][head_partial_stride()] loss sums, head-bias and log_std gradients
};

struct StepChain;
// nullptr when the widths do not fit the kernel (err says why, empty if simply not applicable).
StepChain* step_chain_create(const StepChainSetup& s, std::string* err);
void step_chain_destroy(StepChain* c);
int step_chain_blocks(const StepChain* c);          // rows of block_partials the launch writes
int step_chain_colsum_rows(int rows);               // rows of each colsum array
cudaError_t step_chain_launch(StepChain* c, const StepChainLoss& loss, cudaStream_t stream);

}  // namespace rslrl
