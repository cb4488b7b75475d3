// A GRU memory layer over a time-major rollout x[T][N][D] with explicit hidden-state management
// (state carried in through h0, reset to zero after a step that reported done) and back-propagation
// through time.  FP32: the input products of all T steps run as one SIMT GEMM before the time loop
// (and their gradients as one after it); inside the loop a step is one recurrent product plus one
// gate kernel.  A context of its own, independent of rslrl_ctx.
//
//   r = sigmoid(gi_r + gh_r), z = sigmoid(gi_z + gh_z), n = tanh(gi_n + r * gh_n),
//   h' = (1 - z) n + z h_in,   gi = x W_i + b_i,  gh = h_in W_h + b_h,  h_in(t) = (1 - done[t-1]) h(t-1)
#include "guard.h"
#include "../../include/rslrl_b200.h"
#include "common.cuh"
#include "kernels.h"
#include "tf32.h"

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <string>
#include <vector>

using namespace rslrl;

namespace {

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

// d h_in = d gh W_h^T has few output tiles and a K range of 3H: it is computed as kTmpSplits partial products
// over thirds of that range, which the consumers add in a fixed order
constexpr int kTmpSplits = 3;

__device__ __forceinline__ float sigmoid_f(float a) { return 1.0f / (1.0f + expf(-a)); }

// Step t, one thread per (row, j).  gi/gh: [N][3H] pre-activations of this step; on return gi holds (r, z, n).
// h_out[row][j] = h'; h_next_in (may be null) = done ? 0 : h'.
__global__ void __launch_bounds__(256) gru_gate_kernel(float* __restrict__ gi, const float* __restrict__ gh,
                                                       const float* __restrict__ h_in, const uint8_t* __restrict__ done,
                                                       float* __restrict__ h_out, float* __restrict__ h_next_in, int N, int H) {
    chain_begin();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * H) return;
    const int row = i / H, j = i - row * H;
    float* a = gi + (size_t)row * 3 * H;
    const float* b = gh + (size_t)row * 3 * H;
    const float r = sigmoid_f(a[j] + b[j]);
    const float z = sigmoid_f(a[H + j] + b[H + j]);
    const float n = tanhf(a[2 * H + j] + r * b[2 * H + j]);
    const float hp = h_in[i];
    const float h = (1.0f - z) * n + z * hp;
    a[j] = r; a[H + j] = z; a[2 * H + j] = n;
    h_out[i] = h;
    if (h_next_in) h_next_in[i] = done[row] ? 0.f : h;
}

// Step t of the reverse pass.  rzn: (r, z, n) of the step, replaced by d gi; gh: third block holds gh_n, replaced by d gh.
// dh = dh_seq + (carry_done ? (carry_done[row] ? 0 : dhz + sum of the tmp slabs) : 0); dhz <- dh * z.
__global__ void __launch_bounds__(256) gru_gate_bwd_kernel(float* __restrict__ rzn, float* __restrict__ gh,
                                                           const float* __restrict__ h_in, const float* __restrict__ dh_seq,
                                                           const uint8_t* __restrict__ carry_done, float* __restrict__ dhz,
                                                           const float* __restrict__ tmp, size_t tmp_stride, int N, int H) {
    chain_begin();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * H) return;
    const int row = i / H, j = i - row * H;
    float* a = rzn + (size_t)row * 3 * H;
    float* b = gh + (size_t)row * 3 * H;
    float dh = dh_seq[i];
    if (carry_done && !carry_done[row]) {
        float back = tmp[i];
#pragma unroll
        for (int k = 1; k < kTmpSplits; ++k) back += tmp[i + k * tmp_stride];
        dh += dhz[i] + back;
    }
    const float r = a[j], z = a[H + j], n = a[2 * H + j], ghn = b[2 * H + j], hp = h_in[i];
    const float da_n = dh * (1.0f - z) * (1.0f - n * n);
    const float da_z = dh * (hp - n) * z * (1.0f - z);
    const float da_r = da_n * ghn * r * (1.0f - r);
    a[j] = da_r; a[H + j] = da_z; a[2 * H + j] = da_n;
    b[j] = da_r; b[H + j] = da_z; b[2 * H + j] = da_n * r;
    dhz[i] = dh * z;
}

// out = a + (sum of the slabs of b), zero in the rows flagged by reset (may be null)
__global__ void gru_add_kernel(const float* __restrict__ a, const float* __restrict__ b, size_t b_stride,
                               const uint8_t* __restrict__ reset, float* __restrict__ out, int N, int H) {
    chain_begin();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * H) return;
    float back = b[i];
#pragma unroll
    for (int k = 1; k < kTmpSplits; ++k) back += b[i + k * b_stride];
    out[i] = (reset && reset[i / H]) ? 0.f : a[i] + back;
}

// h_in(0) = h0, zero in the rows flagged by reset (may be null)
__global__ void gru_init_state_kernel(const float* __restrict__ h0, const uint8_t* __restrict__ reset, float* __restrict__ h_in,
                                      int N, int H) {
    chain_begin();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N * H) h_in[i] = (reset && reset[i / H]) ? 0.f : h0[i];
}

__global__ void gru_reduce_kernel(const float* __restrict__ partials, int splits, size_t stride, float* __restrict__ grad, int P) {
    chain_begin();
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    float s = 0.f;
    for (int k = 0; k < splits; ++k) s += partials[(size_t)k * stride + p];
    grad[p] = s;
}

}  // namespace

struct rslrl_gru {
    rslrl_gru_cfg cfg{};
    cudaStream_t stream = nullptr;
    int D = 0, H = 0, P = 0, max_T = 0, max_N = 0, max_splits = 1;
    size_t off_wi = 0, off_bi = 0, off_wh = 0, off_bh = 0;
    std::vector<void*> allocs;
    float *param = nullptr, *grad = nullptr, *partials = nullptr;
    float *gi = nullptr, *gh = nullptr, *hin = nullptr, *dhz = nullptr, *tmp = nullptr;
    // what the last forward saw (backward reads them again)
    const float* x = nullptr; int x_stride = 0; const uint8_t* dones = nullptr; const uint8_t* h0_reset = nullptr;
    int T = 0, N = 0;
    bool forward_done = false;
    std::string err;
    // RSLRL_TF32: transposed weight copies (the forward operands, contraction contiguous), biases padded to 32
    // entries, the device error word of the tensor-core kernels, and the prepared launches of the shapes seen last
    bool tf32 = false;
    float *wi_t = nullptr, *wh_t = nullptr, *bi_pad = nullptr, *bh_pad = nullptr;
    int ld_wi_t = 0, ld_wh_t = 0;
    int* tc_error = nullptr;
    struct Ops {
        const float* x = nullptr; int x_stride = 0; float* dx = nullptr; int dx_stride = 0; int T = 0, N = 0;
        rslrl::Tf32Op* gi = nullptr; rslrl::Tf32Op* dx_op = nullptr; rslrl::Tf32Op* wgrad = nullptr;
        std::vector<rslrl::Tf32Op*> gh, dh;       // one per step
    } ops;
};

namespace {

std::string g_gru_create_error;

rslrl_status gfail(rslrl_gru* g, rslrl_status s, const char* fmt, ...);

// RSLRL_TF32: the prepared tensor-core launches depend on the caller's x pointer and on T and N; they are built when
// those change (host work only: tensor maps) and kept for the calls that follow.
constexpr int kGruWgradRowsPerSplit = 32;
void gru_wgrad_split(size_t rows, int* splits, int* kchunk) {
    *splits = (int)std::max<size_t>(1, std::min<size_t>(32, rows / 512));
    const int per = (int)((rows + *splits - 1) / *splits);
    *kchunk = (per + kGruWgradRowsPerSplit - 1) / kGruWgradRowsPerSplit * kGruWgradRowsPerSplit;
}

void drop_ops(rslrl_gru* g);
rslrl_status prepare_ops(rslrl_gru* g, const float* d_x, int x_stride, int T, int N) {
    rslrl_gru::Ops& o = g->ops;
    if (o.gi && o.x == d_x && o.x_stride == x_stride && o.T == T && o.N == N) return RSLRL_OK;
    drop_ops(g);
    const int H = g->H, D = g->D, G3 = 3 * H;
    const size_t rows = (size_t)T * N;
    bool ok = true;
    o.gi = tf32_op_gemm(d_x, (int)rows, D, x_stride, g->wi_t, G3, g->ld_wi_t, g->gi, G3, g->bi_pad, g->tc_error);
    ok = ok && o.gi;
    for (int t = 0; ok && t < T; ++t) {
        float* gh_t = g->gh + (size_t)t * N * G3;
        const float* hin_t = g->hin + (size_t)t * N * H;
        // gh_t = h_in W_h + b_h;  tmp = d gh_t W_h^T (W_h as stored is the operand with the contraction contiguous)
        o.gh.push_back(tf32_op_gemm(hin_t, N, H, H, g->wh_t, G3, g->ld_wh_t, gh_t, G3, g->bh_pad, g->tc_error));
        o.dh.push_back(tf32_op_gemm(gh_t, N, G3, G3, g->param + g->off_wh, H, G3, g->tmp, H, nullptr, g->tc_error));
        ok = o.gh.back() && o.dh.back();
    }
    if (ok) {
        int splits, kchunk;
        gru_wgrad_split(rows, &splits, &kchunk);
        const Tf32WgradDesc d[2] = {
            {d_x, x_stride, D, g->gi, G3, G3, G3, g->partials + g->off_wi, G3},
            {g->hin, H, H, g->gh, G3, G3, G3, g->partials + g->off_wh, G3}};
        o.wgrad = tf32_op_wgrad(d, 2, (int)rows, splits, kchunk, (long long)g->P, g->tc_error);
        ok = o.wgrad != nullptr;
    }
    if (!ok) { drop_ops(g); return gfail(g, RSLRL_ERR_CUDA, "could not prepare the tensor-core launches (tensor map encoding)"); }
    o.x = d_x; o.x_stride = x_stride; o.T = T; o.N = N;
    return RSLRL_OK;
}

void drop_ops(rslrl_gru* g) {
    tf32_op_free(g->ops.gi); tf32_op_free(g->ops.dx_op); tf32_op_free(g->ops.wgrad);
    for (Tf32Op* o : g->ops.gh) tf32_op_free(o);
    for (Tf32Op* o : g->ops.dh) tf32_op_free(o);
    g->ops = rslrl_gru::Ops{};
}

rslrl_status gfail(rslrl_gru* g, rslrl_status s, const char* fmt, ...) {
    char buf[512];
    va_list ap; va_start(ap, fmt); vsnprintf(buf, sizeof(buf), fmt, ap); va_end(ap);
    if (g) g->err = buf; else g_gru_create_error = buf;
    return s;
}

#define GCU(g, call)                                                                             \
    do {                                                                                         \
        cudaError_t e__ = (call);                                                                \
        if (e__ != cudaSuccess)                                                                  \
            return gfail(g, RSLRL_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e__));   \
    } while (0)

bool valid_cfg(const rslrl_gru_cfg* c, std::string* why) {
    auto bad = [&](const char* m) { if (why) *why = m; return false; };
    if (!c) return bad("config is null");
    if (c->input_dim < 1 || c->input_dim > 16384) return bad("input_dim out of range");
    if (c->hidden_dim < 4 || c->hidden_dim > 4096 || c->hidden_dim % 4) return bad("hidden_dim must be a multiple of 4 in [4, 4096]");
    if (c->max_steps < 1 || c->max_envs < 1) return bad("max_steps and max_envs must be positive");
    if ((long long)c->max_steps * c->max_envs >= (1ll << 30)) return bad("max_steps * max_envs must be below 2^30");
    if ((long long)c->max_envs * 3 * c->hidden_dim >= (1ll << 31)) return bad("max_envs * 3 * hidden_dim must be below 2^31");
    if (c->precision < RSLRL_FP32 || c->precision > RSLRL_BF16) return bad("unknown precision");
    return true;
}

template <typename T>
bool dalloc(rslrl_gru* g, T** p, size_t count) {
    void* q = nullptr;
    const size_t bytes = std::max<size_t>(count * sizeof(T), 256);
    if (guarded_malloc(&q, bytes) != cudaSuccess) return false;
    g->allocs.push_back(q);
    if (cudaMemsetAsync(q, 0, bytes, g->stream) != cudaSuccess) return false;
    *p = (T*)q;
    return true;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

size_t rslrl_gru_num_params(const rslrl_gru_cfg* c) {
    if (!valid_cfg(c, nullptr)) return 0;
    const size_t D = c->input_dim, H = c->hidden_dim;
    return D * 3 * H + 3 * H + H * 3 * H + 3 * H;
}

const char* rslrl_gru_last_error(const rslrl_gru* g) { return g ? g->err.c_str() : g_gru_create_error.c_str(); }

rslrl_status rslrl_gru_destroy(rslrl_gru* g) {
    if (!g) return RSLRL_ERR_INVALID_ARG;
    cudaStreamSynchronize(g->stream);
    drop_ops(g);
    for (void* p : g->allocs) guarded_free(p);
    delete g;
    return RSLRL_OK;
}

rslrl_status rslrl_gru_create(const rslrl_gru_cfg* cfg, void* cuda_stream, rslrl_gru** out) {
    if (!out) return gfail(nullptr, RSLRL_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    std::string why;
    if (!valid_cfg(cfg, &why)) return gfail(nullptr, RSLRL_ERR_INVALID_ARG, "%s", why.c_str());
    if (cfg->precision == RSLRL_BF16) return gfail(nullptr, RSLRL_ERR_UNSUPPORTED, "the recurrent layer has no BF16 mode");
    if (cfg->precision == RSLRL_TF32) {
        std::string terr;
        if (!tf32_ops_init(&terr)) return gfail(nullptr, RSLRL_ERR_UNSUPPORTED, "tensor-core mode: %s", terr.c_str());
    }
    rslrl_gru* g = new rslrl_gru();
    g->cfg = *cfg;
    g->tf32 = cfg->precision == RSLRL_TF32;
    g->stream = (cudaStream_t)cuda_stream;
    g->D = cfg->input_dim; g->H = cfg->hidden_dim; g->max_T = cfg->max_steps; g->max_N = cfg->max_envs;
    const size_t D = g->D, H = g->H;
    g->off_wi = 0; g->off_bi = D * 3 * H; g->off_wh = g->off_bi + 3 * H; g->off_bh = g->off_wh + H * 3 * H;
    g->P = (int)(g->off_bh + 3 * H);
    const size_t rows = (size_t)g->max_T * g->max_N;
    g->max_splits = (int)std::max<size_t>(1, std::min<size_t>(32, rows / 512));
    g->ld_wi_t = round_up(g->D, 4); g->ld_wh_t = round_up(g->H, 4);
    const bool tc_ok = !g->tf32 ||
                       (dalloc(g, &g->wi_t, 3 * H * g->ld_wi_t) && dalloc(g, &g->wh_t, 3 * H * g->ld_wh_t) &&
                        dalloc(g, &g->bi_pad, (size_t)round_up((int)(3 * H), 32)) && dalloc(g, &g->bh_pad, (size_t)round_up((int)(3 * H), 32)) &&
                        dalloc(g, &g->tc_error, 1));
    const bool ok = tc_ok && dalloc(g, &g->param, (size_t)g->P) && dalloc(g, &g->grad, (size_t)g->P) &&
                    dalloc(g, &g->partials, (size_t)g->P * g->max_splits) && dalloc(g, &g->gi, rows * 3 * H) &&
                    dalloc(g, &g->gh, rows * 3 * H) && dalloc(g, &g->hin, rows * H) &&
                    dalloc(g, &g->dhz, (size_t)g->max_N * H) && dalloc(g, &g->tmp, (size_t)kTmpSplits * g->max_N * H) &&
                    cudaStreamSynchronize(g->stream) == cudaSuccess;
    if (!ok) {
        g_gru_create_error = std::string("device allocation failed: ") + cudaGetErrorString(cudaGetLastError());
        rslrl_gru_destroy(g);
        return RSLRL_ERR_CUDA;
    }
    *out = g;
    return RSLRL_OK;
}

rslrl_status rslrl_gru_set_params(rslrl_gru* g, const float* h, size_t n) {
    if (!g || !h) return RSLRL_ERR_INVALID_ARG;
    if (n != (size_t)g->P) return gfail(g, RSLRL_ERR_SHAPE, "expected %d parameters, got %zu", g->P, n);
    GCU(g, cudaMemcpyAsync(g->param, h, sizeof(float) * n, cudaMemcpyHostToDevice, g->stream));
    if (g->tf32) {
        const int G3 = 3 * g->H;
        GCU(g, tf32_transpose(g->param + g->off_wi, g->D, G3, G3, g->wi_t, g->ld_wi_t, g->stream));
        GCU(g, tf32_transpose(g->param + g->off_wh, g->H, G3, G3, g->wh_t, g->ld_wh_t, g->stream));
        GCU(g, cudaMemcpyAsync(g->bi_pad, g->param + g->off_bi, sizeof(float) * G3, cudaMemcpyDeviceToDevice, g->stream));
        GCU(g, cudaMemcpyAsync(g->bh_pad, g->param + g->off_bh, sizeof(float) * G3, cudaMemcpyDeviceToDevice, g->stream));
    }
    GCU(g, cudaStreamSynchronize(g->stream));
    g->forward_done = false;
    return RSLRL_OK;
}

rslrl_status rslrl_gru_get_grads(rslrl_gru* g, float* h, size_t n) {
    if (!g || !h) return RSLRL_ERR_INVALID_ARG;
    if (n != (size_t)g->P) return gfail(g, RSLRL_ERR_SHAPE, "expected %d parameters, got %zu", g->P, n);
    GCU(g, cudaMemcpyAsync(h, g->grad, sizeof(float) * n, cudaMemcpyDeviceToHost, g->stream));
    int code = 0;
    if (g->tf32) GCU(g, cudaMemcpyAsync(&code, g->tc_error, sizeof(int), cudaMemcpyDeviceToHost, g->stream));
    GCU(g, cudaStreamSynchronize(g->stream));
    if (code != 0) {                     // reported once
        GCU(g, cudaMemsetAsync(g->tc_error, 0, sizeof(int), g->stream));
        return gfail(g, RSLRL_ERR_TIMEOUT, "a bounded wait in a tensor-core kernel expired (role %d)", code);
    }
    return RSLRL_OK;
}

rslrl_status rslrl_gru_forward(rslrl_gru* g, const float* d_x, int32_t x_stride, const float* d_h0, const uint8_t* d_h0_reset,
                               const uint8_t* d_dones, int32_t T, int32_t N, float* d_h_out) {
    if (!g || !d_x || !d_h0 || !d_dones || !d_h_out) return RSLRL_ERR_INVALID_ARG;
    if (T < 1 || N < 1) return gfail(g, RSLRL_ERR_INVALID_ARG, "T and N must be positive");
    if (T > g->max_T || N > g->max_N) return gfail(g, RSLRL_ERR_UNSUPPORTED, "T = %d, N = %d exceed max_steps = %d, max_envs = %d", T, N, g->max_T, g->max_N);
    if (x_stride < round_up(g->D, 4) || x_stride % 4) return gfail(g, RSLRL_ERR_SHAPE, "x_stride must be a multiple of 4 and at least input_dim rounded up to 4");
    if (!aligned16(d_x) || !aligned16(d_h0) || !aligned16(d_h_out)) return gfail(g, RSLRL_ERR_ALIGNMENT, "float buffers must be 16-byte aligned");
    const int H = g->H, D = g->D, G3 = 3 * H;
    const size_t rows = (size_t)T * N;
    g->forward_done = false;
    if (g->tf32) {
        const rslrl_status ps = prepare_ops(g, d_x, x_stride, T, N);
        if (ps != RSLRL_OK) return ps;
    }
    // input products of all steps at once: gi = x W_i + b_i
    if (g->tf32) {
        GCU(g, tf32_op_launch(g->ops.gi, g->stream));
    } else {
        GemmBatch b{};
        GemmProblem& p = b.p[b.count++];
        p.A = d_x; p.lda = x_stride; p.B = g->param + g->off_wi; p.ldb = G3; p.C = g->gi; p.ldc = G3;
        p.bias = g->param + g->off_bi; p.M = (int)rows; p.N = G3; p.K = D; p.Cn = G3;
        p.splits = 1; p.kchunk = round_up(D, 8); p.split_stride = 0;
        GCU(g, launch_sgemm(b, false, false, EPI_BIAS, g->stream));
    }
    const int blocks = (N * H + 255) / 256;
    {
        LaunchScope scope_("gru_init_state", g->stream);
        GCU(g, launch_chained(gru_init_state_kernel, dim3(blocks), dim3(256), 0, g->stream, d_h0, d_h0_reset, g->hin, (int)N, H));
    }
    for (int t = 0; t < T; ++t) {
        float* gi_t = g->gi + (size_t)t * N * G3;
        float* gh_t = g->gh + (size_t)t * N * G3;
        const float* hin_t = g->hin + (size_t)t * N * H;
        if (g->tf32) {
            GCU(g, tf32_op_launch(g->ops.gh[t], g->stream));
        } else {
            GemmBatch b{};
            GemmProblem& p = b.p[b.count++];
            p.A = hin_t; p.lda = H; p.B = g->param + g->off_wh; p.ldb = G3; p.C = gh_t; p.ldc = G3;
            p.bias = g->param + g->off_bh; p.M = N; p.N = G3; p.K = H; p.Cn = G3;
            p.splits = 1; p.kchunk = round_up(H, 8); p.split_stride = 0;
            GCU(g, launch_sgemm(b, false, false, EPI_BIAS, g->stream));
        }
        LaunchScope scope_("gru_gate", g->stream);
        GCU(g, launch_chained(gru_gate_kernel, dim3(blocks), dim3(256), 0, g->stream, gi_t, (const float*)gh_t, hin_t,
                              d_dones + (size_t)t * N, d_h_out + (size_t)t * N * H,
                              t + 1 < T ? g->hin + (size_t)(t + 1) * N * H : (float*)nullptr, (int)N, H));
    }
    g->x = d_x; g->x_stride = x_stride; g->dones = d_dones; g->h0_reset = d_h0_reset; g->T = T; g->N = N;
    g->forward_done = true;
    return RSLRL_OK;
}

rslrl_status rslrl_gru_backward(rslrl_gru* g, const float* d_dh, float* d_dx, int32_t dx_stride, float* d_dh0) {
    if (!g || !d_dh) return RSLRL_ERR_INVALID_ARG;
    if (!g->forward_done) return gfail(g, RSLRL_ERR_STATE, "rslrl_gru_backward needs a preceding rslrl_gru_forward (one backward per forward)");
    if (d_dx && (dx_stride < round_up(g->D, 4) || dx_stride % 4)) return gfail(g, RSLRL_ERR_SHAPE, "dx_stride must be a multiple of 4 and at least input_dim rounded up to 4");
    if (!aligned16(d_dh) || (d_dx && !aligned16(d_dx)) || (d_dh0 && !aligned16(d_dh0))) return gfail(g, RSLRL_ERR_ALIGNMENT, "float buffers must be 16-byte aligned");
    const int H = g->H, D = g->D, G3 = 3 * H, T = g->T, N = g->N;
    const size_t rows = (size_t)T * N;
    g->forward_done = false;                 // the saved gates are overwritten by their gradients
    const int blocks = (N * H + 255) / 256;
    for (int t = T - 1; t >= 0; --t) {
        float* gi_t = g->gi + (size_t)t * N * G3;
        float* gh_t = g->gh + (size_t)t * N * G3;
        {
            LaunchScope scope_("gru_gate_bwd", g->stream);
            GCU(g, launch_chained(gru_gate_bwd_kernel, dim3(blocks), dim3(256), 0, g->stream, gi_t, gh_t,
                                  (const float*)(g->hin + (size_t)t * N * H), d_dh + (size_t)t * N * H,
                                  t + 1 < T ? g->dones + (size_t)t * N : (const uint8_t*)nullptr, g->dhz, (const float*)g->tmp,
                                  (size_t)g->max_N * H, N, H));
        }
        // tmp = d gh W_h^T (the tensor-core product fills the first of the slices the gate kernel adds up; the
        // others stay zero)
        if (g->tf32) {
            GCU(g, tf32_op_launch(g->ops.dh[t], g->stream));
            continue;
        }
        GemmBatch b{};
        GemmProblem& p = b.p[b.count++];
        p.A = gh_t; p.lda = G3; p.B = g->param + g->off_wh; p.ldb = G3; p.C = g->tmp; p.ldc = H;
        p.M = N; p.N = H; p.K = G3; p.Cn = H;
        p.splits = kTmpSplits; p.kchunk = round_up((G3 + kTmpSplits - 1) / kTmpSplits, 8); p.split_stride = (long long)g->max_N * H;
        GCU(g, launch_sgemm(b, false, true, EPI_PLAIN, g->stream));
    }
    if (d_dh0) {
        LaunchScope scope_("gru_add", g->stream);
        GCU(g, launch_chained(gru_add_kernel, dim3(blocks), dim3(256), 0, g->stream, (const float*)g->dhz, (const float*)g->tmp, (size_t)g->max_N * H, g->h0_reset, d_dh0, N, H));
    }
    if (d_dx && g->tf32) {
        // dx = d gi W_i^T (W_i as stored is the operand with the contraction contiguous)
        rslrl_gru::Ops& o = g->ops;
        if (!o.dx_op || o.dx != d_dx || o.dx_stride != dx_stride) {
            tf32_op_free(o.dx_op);
            o.dx_op = tf32_op_gemm(g->gi, (int)rows, G3, G3, g->param + g->off_wi, D, G3, d_dx, dx_stride, nullptr, g->tc_error, round_up(D, 4));
            if (!o.dx_op) return gfail(g, RSLRL_ERR_CUDA, "could not prepare the tensor-core launch of dx (tensor map encoding)");
            o.dx = d_dx; o.dx_stride = dx_stride;
        }
        GCU(g, tf32_op_launch(o.dx_op, g->stream));
    } else if (d_dx) {
        GemmBatch b{};
        GemmProblem& p = b.p[b.count++];
        p.A = g->gi; p.lda = G3; p.B = g->param + g->off_wi; p.ldb = G3; p.C = d_dx; p.ldc = dx_stride;
        p.M = (int)rows; p.N = D; p.K = G3; p.Cn = round_up(D, 4); p.splits = 1; p.kchunk = round_up(G3, 8); p.split_stride = 0;
        GCU(g, launch_sgemm(b, false, true, EPI_PLAIN, g->stream));
    }
    // parameter gradients over all steps: dW_i = x^T d gi, dW_h = h_in^T d gh, biases = column sums
    int splits, kchunk;
    gru_wgrad_split(rows, &splits, &kchunk);
    if (g->tf32) GCU(g, tf32_op_launch(g->ops.wgrad, g->stream));
    {
        GemmBatch b{};
        GemmProblem& p = b.p[b.count++];
        p.A = g->x; p.lda = g->x_stride; p.B = g->gi; p.ldb = G3; p.C = g->partials + g->off_wi; p.ldc = G3;
        p.M = D; p.N = G3; p.K = (int)rows; p.Cn = G3; p.splits = splits; p.kchunk = kchunk; p.split_stride = g->P;
        GemmProblem& q = b.p[b.count++];
        q.A = g->hin; q.lda = H; q.B = g->gh; q.ldb = G3; q.C = g->partials + g->off_wh; q.ldc = G3;
        q.M = H; q.N = G3; q.K = (int)rows; q.Cn = G3; q.splits = splits; q.kchunk = kchunk; q.split_stride = g->P;
        if (!g->tf32) GCU(g, launch_sgemm(b, true, false, EPI_PLAIN, g->stream));
        ColsumBatch cs{};
        cs.splits = splits; cs.split_stride = g->P; cs.is_bf16 = 0;
        cs.p[cs.count++] = ColsumProblem{g->gi, g->partials + g->off_bi, (int)rows, G3, G3};
        cs.p[cs.count++] = ColsumProblem{g->gh, g->partials + g->off_bh, (int)rows, G3, G3};
        GCU(g, launch_colsum(cs, g->stream));
    }
    LaunchScope scope_("gru_reduce", g->stream);
    GCU(g, launch_chained(gru_reduce_kernel, dim3((g->P + 255) / 256), dim3(256), 0, g->stream, (const float*)g->partials, splits,
                          (size_t)g->P, g->grad, g->P));
    return RSLRL_OK;
}

}  // extern "C"
