// Tensor-core engine of the RSLRL_TF32 mode: the hidden-layer products of act, forward and data
// gradient as tcgen05 kind::tf32 GEMMs on the FP32 buffers of the FP32 mode (operands are read as
// FP32 and used with TF32 precision by the tensor cores; accumulation, bias, ELU and everything
// else stay FP32), and the weight gradients of all layers likewise.  Head products, bias gradients, loss and
// optimiser are the FP32 mode's kernels.
#pragma once
#include "../../include/rslrl_b200.h"
#include "common.cuh"
#include "kernels.h"
#include <string>

namespace rslrl {

struct Tf32Setup {
    int N, R, T;                            // rollout rows per act call, minibatch rows incl. mirrored, rollout steps
    cudaStream_t stream;
    float elu_alpha;
    const float* param;                     // FP32 master parameters (padded device layout)
    int nl[2], in_dim[2], in_ld[2];         // layers per net (head included), observation widths and row strides
    int in[2][kMaxLayers], out[2][kMaxLayers], out_p[2][kMaxLayers], hid_ld[2][kMaxLayers];
    size_t w_off[2][kMaxLayers], b_off[2][kMaxLayers];
    const float* obs_storage[2]; int obs_stride[2];   // rollout observations [T * N][stride] (act reads step t in place)
    const float* last_obs_c;                          // [N][obs_stride[1]]: the observation after the last step
    const float* x[2];                                // minibatch inputs [R][in_ld]
    float* act_h[2][kMaxLayers];                      // post-activations of act [N][hid_ld]
    float* up_h[2][kMaxLayers];                       // post-activations of the update [R][hid_ld]
    float* up_dz[2][kMaxLayers];                      // dL/dz of the update [R][hid_ld]
    const float* dhead[2]; int ld_dhead[2];           // dL/d(head output) of the update [R][ld]: policy mean, value
    float* partials; long long split_stride;          // weight-gradient partials [splits][split_stride], layer l at w_off
    int splits, kchunk;                               // minibatch rows per split: a multiple of 32
};

struct Tf32Engine;

Tf32Engine* tf32_create(const Tf32Setup& s, std::string* err);
void tf32_destroy(Tf32Engine* e);
// Transposed copies of the hidden-layer weights ([out][in], the contraction contiguous): the forward operand.
// After rslrl_set_params and after every optimiser step.
cudaError_t tf32_refresh_weights(Tf32Engine* e);
// Hidden layers of both nets on the rows of rollout step t (do_actor), or of the critic alone on last_obs_c.
cudaError_t tf32_act_forward(Tf32Engine* e, int t, bool do_actor);
// Hidden layers of both nets on the minibatch rows.
cudaError_t tf32_update_forward(Tf32Engine* e);
// dL/dz of hidden layer (top - back - 1) of every net that has one, from dL/dz of the layer above.
cudaError_t tf32_update_dgrad(Tf32Engine* e, int back);
// Weight-gradient partials of every layer of both nets, heads included (after the data gradients of the step).
cudaError_t tf32_update_wgrad(Tf32Engine* e);
// Synchronises the stream and returns the device error code (0 = none); a non-zero code is cleared once read.
cudaError_t tf32_read_error(Tf32Engine* e, int* host_code);

// ------------------------------------------------------------------------------------------------
// The same kernels for other callers (the recurrent layer): prepared launches on caller-owned buffers.
struct Tf32Op;
// Once per process before the first op: shared-memory attributes of the kernels; false (with a reason) on a
// device without these tensor cores.
bool tf32_ops_init(std::string* err);
// D[rows][ldd] = A[rows][k] (row stride lda) * B[n][k]^T (row stride ldb, the contraction contiguous) (+ bias[n],
// readable up to the next multiple of 32 entries, or null).  Pointers 16-byte aligned, strides multiples of 4 floats.
// n_store (0: n): columns of D that are written; those from n on come out as zero.
Tf32Op* tf32_op_gemm(const float* A, int rows, int k, int lda, const float* B, int n, int ldb, float* D, int ldd,
                     const float* bias, int* error_dev, int n_store = 0);
// The same product with an activation epilogue: kind 0: D = ELU(A B^T + bias) (bias as above); kind 1: D = (A B^T) *
// ELU'(aux), aux [rows][ldd] holding the stored post-activations.
Tf32Op* tf32_op_gemm_act(int kind, const float* A, int rows, int k, int lda, const float* B, int n, int ldb, float* D, int ldd,
                         const float* bias_or_aux, float alpha, int* error_dev, int n_store = 0);
// out_i[s][m_i][ld_out_i] (s-th slice at s * split_stride floats) = A_i[rows s][m_i]^T B_i[rows s][n_i] for up to eight
// pairs, rows s = [s * kchunk, (s + 1) * kchunk) cut at `rows`; kchunk a multiple of 32; n_store_i columns are written.
struct Tf32WgradDesc { const float* A; int lda, m; const float* B; int ldb, n, n_store; float* out; int ld_out; };
Tf32Op* tf32_op_wgrad(const Tf32WgradDesc* d, int count, int rows, int splits, int kchunk, long long split_stride, int* error_dev);
cudaError_t tf32_op_launch(const Tf32Op* op, cudaStream_t stream);
void tf32_op_free(Tf32Op* op);
// dst[out][ld_dst] = src[in][ld_src]^T (FP32), on the stream
cudaError_t tf32_transpose(const float* src, int in, int out, int ld_src, float* dst, int ld_dst, cudaStream_t stream);

}  // namespace rslrl
