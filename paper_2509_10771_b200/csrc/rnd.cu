// Random network distillation on a subset of the state: a fixed target MLP g and a trained
// predictor MLP f read s = o[idx]; the intrinsic reward is mean_j (f_j(s) - g_j(s))^2 and the
// predictor is regressed on the target.  FP32 throughout (the nets are small and the reward is a
// difference of two nearly equal quantities once the predictor has learnt): the products run on
// the SIMT GEMM kernels, the rest are the small kernels below.  A context of its own, independent
// of rslrl_ctx: it works on observation rows the caller passes in.
#define RSLRL_INDEX_CHECKS
#include "guard.h"
#include "../../include/rslrl_b200.h"
#include "common.cuh"
#include "kernels.h"
#include "tf32.h"
#include <map>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <string>
#include <vector>

using namespace rslrl;

namespace rslrl { void set_global_error(const char* msg); }

namespace {

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

struct RLayer { int in, out, out_p; size_t w_off, b_off, w_flat, b_flat; int ld; };

// s[r][j] = obs[row(r)][idx[j]], row(r) = rows ? rows[r] : r; columns [ns, ld) are written as 0
__global__ void rnd_subset_kernel(const float* __restrict__ obs, int obs_stride, int obs_dim, const int* __restrict__ rows,
                                  int rows_limit, const int* __restrict__ idx, int ns, float* __restrict__ s, int ld, int n) {
    chain_begin();
    const long long total = (long long)n * ld;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(i / ld), j = (int)(i - (long long)r * ld);
        const size_t src = rows ? (size_t)checked_index((uint32_t)rows[r], (uint32_t)rows_limit, 2) : (size_t)r;
        s[i] = j < ns ? obs[src * obs_stride + checked_index((uint32_t)idx[j], (uint32_t)obs_dim, 3)] : 0.f;
    }
}

// One warp per row: e = sum_j (f_j - g_j)^2 / E.
//   g_rows != null: row r of f is compared with row g_rows[r] of g
//   rewards != null:  rewards[r] += weight * e;  r_int != null: r_int[r] = e
//   dout != null (training): dout[r][j] = 2 (f_j - g_j) * scale (scale = 1 / (rows E)), and the block's sum of e
//   goes to loss_partials[block] (warps added in order)
__global__ void __launch_bounds__(256) rnd_error_kernel(const float* __restrict__ f, const float* __restrict__ g,
                                                        const int* __restrict__ g_rows, int ld,
                                                        int E, int n, float weight, float* __restrict__ rewards,
                                                        float* __restrict__ r_int, float* __restrict__ dout, float scale,
                                                        float* __restrict__ loss_partials) {
    chain_begin();
    __shared__ float ws[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = blockIdx.x * 8 + warp;
    float e = 0.f;
    if (r < n) {
        const float* grow = g + (size_t)(g_rows ? g_rows[r] : r) * ld;       // the target's outputs may be stored per batch row
        for (int j = lane; j < E; j += 32) {
            const float d = f[(size_t)r * ld + j] - grow[j];
            e += d * d;
            if (dout) dout[(size_t)r * ld + j] = 2.0f * d * scale;
        }
        e = warp_sum(e) / (float)E;
        if (lane == 0) {
            if (rewards) rewards[r] += weight * e;
            if (r_int) r_int[r] = e;
        }
    }
    if (loss_partials) {
        if (lane == 0) ws[warp] = r < n ? e : 0.f;
        __syncthreads();
        if (threadIdx.x == 0) {
            float t = 0.f;
            for (int w = 0; w < 8; ++w) t += ws[w];
            loss_partials[blockIdx.x] = t;
        }
    }
}

// grad[p] = sum over splits (in order); Adam on the predictor; block 0 also adds up the loss partials.
__global__ void __launch_bounds__(256) rnd_adam_kernel(const float* __restrict__ partials, int splits, size_t split_stride,
                                                       float* __restrict__ grad, float* __restrict__ param,
                                                       float* __restrict__ m, float* __restrict__ v, int P, float lr,
                                                       float b1, float b2, float eps, float c1, float c2,
                                                       const float* __restrict__ loss_partials, int nloss, float inv_rows,
                                                       float* __restrict__ step_loss) {
    chain_begin();
    for (int p = blockIdx.x * blockDim.x + threadIdx.x; p < P; p += gridDim.x * blockDim.x) {
        float gsum = 0.f;
        for (int s = 0; s < splits; ++s) gsum += partials[(size_t)s * split_stride + p];
        grad[p] = gsum;
        const float mm = b1 * m[p] + (1.0f - b1) * gsum;
        const float vv = b2 * v[p] + (1.0f - b2) * gsum * gsum;
        m[p] = mm; v[p] = vv;
        param[p] -= lr * (mm * c1) / (sqrtf(vv * c2) + eps);
    }
    if (blockIdx.x == 0) {
        // fixed order: thread t adds partials t, t + 256, ...; then a tree over the 256 sums
        __shared__ float red[256];
        float t = 0.f;
        for (int i = threadIdx.x; i < nloss; i += 256) t += loss_partials[i];
        red[threadIdx.x] = t;
        __syncthreads();
        for (int w = 128; w > 0; w >>= 1) {
            if ((int)threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
            __syncthreads();
        }
        if (threadIdx.x == 0) *step_loss = red[0] * inv_rows;
    }
}

}  // namespace

struct rslrl_rnd {
    rslrl_rnd_cfg cfg{};
    cudaStream_t stream = nullptr;
    std::vector<RLayer> L;
    size_t P_flat = 0;
    int P_dev = 0;
    int ns = 0, lds = 0, E = 0, ldE = 0;
    int max_rows = 0, max_splits = 1;
    std::vector<void*> allocs;
    int* idx = nullptr;
    float *pf = nullptr, *pg = nullptr, *grad = nullptr, *m = nullptr, *v = nullptr, *partials = nullptr;
    float* s = nullptr;                       // [max_rows][lds] the selected state entries
    std::vector<float*> hf, hg, dz;           // per layer: activations of f and g, gradients at f's outputs
    float* loss_partials = nullptr; int max_loss_blocks = 0;
    float* step_loss = nullptr;                   // [max_epochs * max_minibatches]
    int* perm = nullptr;                          // [max_epochs][max_batch]
    float* gall = nullptr;                        // [max_batch][ldE] the target's outputs for every row of the batch
    long long adam_step = 0;
    std::string err;
    // RSLRL_TF32: transposed weight copies of both nets (the forward operands, contraction contiguous; the
    // predictor's are refreshed after every optimiser step), the device error word of the tensor-core kernels, and
    // the prepared launches per row count (tensor maps: host work only, built when a row count is first seen)
    bool tf32 = false;
    std::vector<float*> wt_f, wt_g; std::vector<int> ld_wt;
    int* tc_error = nullptr;
    struct RowsOps {
        std::vector<rslrl::Tf32Op*> fwd_f, fwd_g, dgrad;     // per layer (dgrad[l] produces dz[l - 1])
        rslrl::Tf32Op* wgrad = nullptr; int wgrad_splits = 0, wgrad_kchunk = 0;
    };
    std::map<int, RowsOps> ops;
};

namespace {

std::string g_rnd_create_error;

rslrl_status rfail(rslrl_rnd* r, rslrl_status s, const char* fmt, ...) {
    char buf[512];
    va_list ap; va_start(ap, fmt); vsnprintf(buf, sizeof(buf), fmt, ap); va_end(ap);
    if (r) r->err = buf; else g_rnd_create_error = buf;
    return s;
}

#define RCU(r, call)                                                                             \
    do {                                                                                         \
        cudaError_t e__ = (call);                                                                \
        if (e__ != cudaSuccess)                                                                  \
            return rfail(r, RSLRL_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e__));   \
    } while (0)

bool valid_cfg(const rslrl_rnd_cfg* c, std::string* why) {
    auto bad = [&](const char* m) { if (why) *why = m; return false; };
    if (!c) return bad("config is null");
    if (c->obs_dim < 1 || c->num_idx < 1 || c->num_idx > c->obs_dim) return bad("need 1 <= num_idx <= obs_dim");
    if (!c->h_idx) return bad("h_idx is null");
    for (int j = 0; j < c->num_idx; ++j)
        if (c->h_idx[j] < 0 || c->h_idx[j] >= c->obs_dim) return bad("an entry of h_idx is out of range");
    if (c->num_hidden < 1 || c->num_hidden > RSLRL_MAX_HIDDEN) return bad("num_hidden out of range");
    for (int l = 0; l < c->num_hidden; ++l)
        if (c->hidden[l] < 1 || c->hidden[l] > 8192) return bad("a hidden width is out of range");
    if (c->embed_dim < 1 || c->embed_dim > 8192) return bad("embed_dim out of range");
    if (c->max_rows < 1) return bad("max_rows must be positive");
    if (c->precision < RSLRL_FP32 || c->precision > RSLRL_BF16) return bad("unknown precision");
    if (c->max_batch < 1 || c->max_epochs < 1 || c->max_minibatches < 1) return bad("max_batch, max_epochs and max_minibatches must be positive");
    if ((long long)c->max_epochs * c->max_minibatches > (1 << 20)) return bad("max_epochs * max_minibatches exceeds 2^20 steps");
    if (!(c->lr > 0.f) || !(c->adam_eps > 0.f) || c->adam_b1 < 0.f || c->adam_b1 >= 1.f || c->adam_b2 < 0.f || c->adam_b2 >= 1.f)
        return bad("Adam settings out of range");
    return true;
}

void layer_dims(const rslrl_rnd_cfg* c, std::vector<RLayer>* out, size_t* p_flat, int* p_dev) {
    int in = c->num_idx;
    size_t flat = 0, dev = 0;
    out->clear();
    for (int l = 0; l <= c->num_hidden; ++l) {
        RLayer R{};
        R.in = in; R.out = l < c->num_hidden ? c->hidden[l] : c->embed_dim;
        R.out_p = round_up(R.out, 4); R.ld = round_up(R.out, 8);
        R.w_flat = flat; flat += (size_t)R.in * R.out; R.b_flat = flat; flat += R.out;
        R.w_off = dev; dev += (size_t)R.in * R.out_p; R.b_off = dev; dev += R.out_p;
        out->push_back(R);
        in = R.out;
    }
    *p_flat = flat; *p_dev = (int)dev;
}

template <typename T>
bool dalloc(rslrl_rnd* r, T** p, size_t count) {
    void* q = nullptr;
    const size_t bytes = std::max<size_t>(count * sizeof(T), 256);
    if (guarded_malloc(&q, bytes) != cudaSuccess) return false;
    r->allocs.push_back(q);
    if (cudaMemsetAsync(q, 0, bytes, r->stream) != cudaSuccess) return false;
    *p = (T*)q;
    return true;
}

int splits_for(int rows) { return std::max(1, std::min(32, rows / 512)); }

// the predictor (do_f) and / or the target (do_g) through all layers on `rows` rows of r->s; g_last, if not
// null, receives the target's last layer instead of the work buffer
// ---- RSLRL_TF32 ------------------------------------------------------------------------------------------
void drop_ops(rslrl_rnd* r) {
    for (auto& kv : r->ops) {
        for (Tf32Op* o : kv.second.fwd_f) tf32_op_free(o);
        for (Tf32Op* o : kv.second.fwd_g) tf32_op_free(o);
        for (Tf32Op* o : kv.second.dgrad) tf32_op_free(o);
        tf32_op_free(kv.second.wgrad);
    }
    r->ops.clear();
}

// Wt[out][in] of one net (0: predictor, 1: target) from its W[in][out_p]
rslrl_status refresh_transposes(rslrl_rnd* r, int net) {
    const float* par = net == 0 ? r->pf : r->pg;
    std::vector<float*>& wt = net == 0 ? r->wt_f : r->wt_g;
    for (size_t l = 0; l < r->L.size(); ++l)
        RCU(r, tf32_transpose(par + r->L[l].w_off, r->L[l].in, r->L[l].out, r->L[l].out_p, wt[l], r->ld_wt[l], r->stream));
    return RSLRL_OK;
}

// rows per weight-gradient split: a multiple of the tensor-core kernel's k-block in TF32 mode
int kchunk_for(const rslrl_rnd* r, int rows, int splits) { return round_up((rows + splits - 1) / splits, r->tf32 ? 32 : 8); }

rslrl_status ops_for(rslrl_rnd* r, int rows, rslrl_rnd::RowsOps** out) {
    auto it = r->ops.find(rows);
    if (it != r->ops.end()) { *out = &it->second; return RSLRL_OK; }
    rslrl_rnd::RowsOps o;
    const int nl = (int)r->L.size();
    bool ok = true;
    for (int l = 0; ok && l < nl; ++l) {
        const RLayer& Ly = r->L[l];
        for (int net = 0; ok && net < 2; ++net) {
            const float* par = net == 0 ? r->pf : r->pg;
            std::vector<float*>& h = net == 0 ? r->hf : r->hg;
            const float* A = l == 0 ? r->s : h[l - 1];
            const int lda = l == 0 ? r->lds : r->L[l - 1].ld;
            const float* B = (net == 0 ? r->wt_f : r->wt_g)[l];
            Tf32Op* op = l + 1 < nl
                ? tf32_op_gemm_act(0, A, rows, Ly.in, lda, B, Ly.out, r->ld_wt[l], h[l], Ly.ld, par + Ly.b_off, r->cfg.elu_alpha, r->tc_error, Ly.out_p)
                : tf32_op_gemm(A, rows, Ly.in, lda, B, Ly.out, r->ld_wt[l], h[l], Ly.ld, par + Ly.b_off, r->tc_error, Ly.out_p);
            (net == 0 ? o.fwd_f : o.fwd_g).push_back(op);
            ok = op != nullptr;
        }
    }
    o.dgrad.assign(nl, nullptr);
    for (int l = nl - 1; ok && l > 0; --l) {
        const RLayer& Ly = r->L[l];
        // dz[l-1] = (dz[l] W[l]^T) * ELU'(hf[l-1]); W[l] as stored is the operand with the contraction (out) contiguous
        o.dgrad[l] = tf32_op_gemm_act(1, r->dz[l], rows, Ly.out, Ly.ld, r->pf + Ly.w_off, Ly.in, Ly.out_p, r->dz[l - 1], r->L[l - 1].ld,
                                      r->hf[l - 1], r->cfg.elu_alpha, r->tc_error, r->L[l - 1].out_p);
        ok = o.dgrad[l] != nullptr;
    }
    if (ok) {
        o.wgrad_splits = splits_for(rows);
        o.wgrad_kchunk = kchunk_for(r, rows, o.wgrad_splits);
        std::vector<Tf32WgradDesc> d;
        for (int l = 0; l < nl; ++l) {
            const RLayer& Ly = r->L[l];
            d.push_back(Tf32WgradDesc{l == 0 ? r->s : r->hf[l - 1], l == 0 ? r->lds : r->L[l - 1].ld, Ly.in, r->dz[l], Ly.ld, Ly.out,
                                      Ly.out_p, r->partials + Ly.w_off, Ly.out_p});
        }
        o.wgrad = tf32_op_wgrad(d.data(), nl, rows, o.wgrad_splits, o.wgrad_kchunk, (long long)r->P_dev, r->tc_error);
        ok = o.wgrad != nullptr;
    }
    if (!ok) {
        for (Tf32Op* p : o.fwd_f) tf32_op_free(p);
        for (Tf32Op* p : o.fwd_g) tf32_op_free(p);
        for (Tf32Op* p : o.dgrad) tf32_op_free(p);
        tf32_op_free(o.wgrad);
        return rfail(r, RSLRL_ERR_CUDA, "could not prepare the tensor-core launches (tensor map encoding)");
    }
    *out = &(r->ops[rows] = o);
    return RSLRL_OK;
}

rslrl_status forward(rslrl_rnd* r, int rows, bool do_f, bool do_g, float* g_last) {
    const int nl = (int)r->L.size();
    if (r->tf32) {
        rslrl_rnd::RowsOps* o = nullptr;
        const rslrl_status ps = ops_for(r, rows, &o);
        if (ps != RSLRL_OK) return ps;
        for (int l = 0; l < nl; ++l) {
            if (do_f) RCU(r, tf32_op_launch(o->fwd_f[l], r->stream));
            if (do_g) RCU(r, tf32_op_launch(o->fwd_g[l], r->stream));
        }
        // the prepared launches write the target's outputs to its own buffer: copied to where the caller wants them
        if (do_g && g_last)
            RCU(r, cudaMemcpyAsync(g_last, r->hg.back(), sizeof(float) * (size_t)rows * r->ldE, cudaMemcpyDeviceToDevice, r->stream));
        return RSLRL_OK;
    }
    for (int l = 0; l < nl; ++l) {
        const RLayer& Ly = r->L[l];
        GemmBatch b{};
        b.alpha = r->cfg.elu_alpha;
        for (int net = 0; net < 2; ++net) {
            if (net == 0 ? !do_f : !do_g) continue;
            const float* par = net == 0 ? r->pf : r->pg;
            std::vector<float*>& h = net == 0 ? r->hf : r->hg;
            GemmProblem& p = b.p[b.count++];
            p.A = l == 0 ? r->s : h[l - 1]; p.lda = l == 0 ? r->lds : r->L[l - 1].ld;
            p.B = par + Ly.w_off; p.ldb = Ly.out_p;
            p.C = (net == 1 && l + 1 == nl && g_last) ? g_last : h[l]; p.ldc = Ly.ld;
            p.bias = par + Ly.b_off;
            p.M = rows; p.N = Ly.out; p.K = Ly.in; p.Cn = Ly.out_p;
            p.splits = 1; p.kchunk = round_up(Ly.in, 8); p.split_stride = 0;
        }
        RCU(r, launch_sgemm(b, false, false, l + 1 < nl ? EPI_BIAS_ELU : EPI_BIAS, r->stream));
    }
    return RSLRL_OK;
}

rslrl_status subset(rslrl_rnd* r, const float* d_obs, int obs_stride, const int* rows_idx, int rows, int rows_limit = 0) {
    const long long total = (long long)rows * r->lds;
    const int blocks = (int)std::min<long long>((total + 255) / 256, 148 * 16);
    LaunchScope scope_("rnd_subset", r->stream);
    RCU(r, launch_chained(rnd_subset_kernel, dim3(blocks), dim3(256), 0, r->stream, d_obs, obs_stride, (int)r->cfg.obs_dim, rows_idx,
                          rows_limit, (const int*)r->idx, r->ns, r->s, r->lds, rows));
    return RSLRL_OK;
}

// gradients of the predictor from dz[last] (already filled) into r->partials: first the chain of data
// gradients, then the weight gradients of all layers in one launch and all bias gradients in another
rslrl_status backward(rslrl_rnd* r, int rows, int splits, int kchunk) {
    const int nl = (int)r->L.size();
    rslrl_rnd::RowsOps* tc = nullptr;
    if (r->tf32) {
        const rslrl_status ps = ops_for(r, rows, &tc);
        if (ps != RSLRL_OK) return ps;
        if (tc->wgrad_splits != splits || tc->wgrad_kchunk != kchunk) return rfail(r, RSLRL_ERR_STATE, "weight-gradient splits do not match the prepared launch");
        for (int l = nl - 1; l > 0; --l) RCU(r, tf32_op_launch(tc->dgrad[l], r->stream));
        RCU(r, tf32_op_launch(tc->wgrad, r->stream));
    }
    for (int l = nl - 1; l > 0 && !tc; --l) {
        const RLayer& Ly = r->L[l];
        GemmBatch dg{};
        dg.alpha = r->cfg.elu_alpha;
        GemmProblem& d = dg.p[dg.count++];
        d.A = r->dz[l]; d.lda = Ly.ld;
        d.B = r->pf + Ly.w_off; d.ldb = Ly.out_p;
        d.C = r->dz[l - 1]; d.ldc = r->L[l - 1].ld;
        d.aux = r->hf[l - 1]; d.ldaux = r->L[l - 1].ld;
        d.M = rows; d.N = Ly.in; d.K = Ly.out; d.Cn = r->L[l - 1].ld;
        d.splits = 1; d.kchunk = round_up(Ly.out, 8); d.split_stride = 0;
        RCU(r, launch_sgemm(dg, false, true, EPI_DELU, r->stream));
    }
    for (int l0 = 0; l0 < nl && !tc; l0 += kMaxGemmBatch) {
        GemmBatch wg{};
        for (int l = l0; l < std::min(nl, l0 + kMaxGemmBatch); ++l) {
            const RLayer& Ly = r->L[l];
            GemmProblem& p = wg.p[wg.count++];
            p.A = l == 0 ? r->s : r->hf[l - 1]; p.lda = l == 0 ? r->lds : r->L[l - 1].ld;
            p.B = r->dz[l]; p.ldb = Ly.ld;
            p.C = r->partials + Ly.w_off; p.ldc = Ly.out_p;
            p.M = Ly.in; p.N = Ly.out; p.K = rows; p.Cn = Ly.out_p;
            p.splits = splits; p.kchunk = kchunk; p.split_stride = r->P_dev;
        }
        RCU(r, launch_sgemm(wg, true, false, EPI_PLAIN, r->stream));
    }
    ColsumBatch cs{};
    cs.splits = splits; cs.split_stride = r->P_dev; cs.is_bf16 = 0;
    for (int l = 0; l < nl; ++l) {
        const RLayer& Ly = r->L[l];
        ColsumProblem& q = cs.p[cs.count++];
        q.X = r->dz[l]; q.out = r->partials + Ly.b_off; q.rows = rows; q.n = Ly.out; q.ld = Ly.ld;
    }
    RCU(r, launch_colsum(cs, r->stream));
    return RSLRL_OK;
}

}  // namespace

extern "C" {

size_t rslrl_rnd_num_params(const rslrl_rnd_cfg* cfg) {
    if (!valid_cfg(cfg, nullptr)) return 0;
    std::vector<RLayer> L; size_t flat; int dev;
    layer_dims(cfg, &L, &flat, &dev);
    return flat;
}

const char* rslrl_rnd_last_error(const rslrl_rnd* r) { return r ? r->err.c_str() : g_rnd_create_error.c_str(); }

rslrl_status rslrl_rnd_destroy(rslrl_rnd* r) {
    if (!r) return RSLRL_ERR_INVALID_ARG;
    cudaStreamSynchronize(r->stream);
    drop_ops(r);
    for (void* p : r->allocs) guarded_free(p);
    delete r;
    return RSLRL_OK;
}

rslrl_status rslrl_rnd_create(const rslrl_rnd_cfg* cfg, void* cuda_stream, rslrl_rnd** out) {
    if (!out) return rfail(nullptr, RSLRL_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    std::string why;
    if (!valid_cfg(cfg, &why)) return rfail(nullptr, RSLRL_ERR_INVALID_ARG, "%s", why.c_str());
    if (cfg->precision == RSLRL_BF16) return rfail(nullptr, RSLRL_ERR_UNSUPPORTED, "random network distillation has no BF16 mode");
    if (cfg->precision == RSLRL_TF32) {
        std::string terr;
        if (!tf32_ops_init(&terr)) return rfail(nullptr, RSLRL_ERR_UNSUPPORTED, "tensor-core mode: %s", terr.c_str());
    }
    rslrl_rnd* r = new rslrl_rnd();
    r->cfg = *cfg; r->cfg.h_idx = nullptr;
    r->tf32 = cfg->precision == RSLRL_TF32;
    r->stream = (cudaStream_t)cuda_stream;
    layer_dims(cfg, &r->L, &r->P_flat, &r->P_dev);
    r->ns = cfg->num_idx; r->lds = round_up(r->ns, 4);
    r->E = cfg->embed_dim; r->ldE = r->L.back().ld;
    r->max_rows = cfg->max_rows; r->max_splits = splits_for(cfg->max_rows);
    r->max_loss_blocks = (cfg->max_rows + 7) / 8;
    const size_t rows = (size_t)cfg->max_rows;
    // (32 floats of slack behind the parameter vectors: the tensor-core epilogues read biases in groups of 32)
    bool ok = dalloc(r, &r->idx, (size_t)r->ns) && dalloc(r, &r->pf, (size_t)r->P_dev + 32) && dalloc(r, &r->pg, (size_t)r->P_dev + 32) &&
              dalloc(r, &r->grad, (size_t)r->P_dev) && dalloc(r, &r->m, (size_t)r->P_dev) && dalloc(r, &r->v, (size_t)r->P_dev) &&
              dalloc(r, &r->partials, (size_t)r->P_dev * r->max_splits) && dalloc(r, &r->s, rows * r->lds) &&
              dalloc(r, &r->loss_partials, (size_t)r->max_loss_blocks) &&
              dalloc(r, &r->perm, (size_t)cfg->max_epochs * cfg->max_batch) &&
              dalloc(r, &r->step_loss, (size_t)cfg->max_epochs * cfg->max_minibatches) &&
              dalloc(r, &r->gall, (size_t)cfg->max_batch * r->ldE);
    for (size_t l = 0; ok && l < r->L.size(); ++l) {
        float *a = nullptr, *b = nullptr, *c = nullptr;
        ok = dalloc(r, &a, rows * r->L[l].ld) && dalloc(r, &b, rows * r->L[l].ld) && dalloc(r, &c, rows * r->L[l].ld);
        r->hf.push_back(a); r->hg.push_back(b); r->dz.push_back(c);
    }
    if (ok && r->tf32) {
        ok = dalloc(r, &r->tc_error, 1);
        for (size_t l = 0; ok && l < r->L.size(); ++l) {
            float *a = nullptr, *b = nullptr;
            const int ld = round_up(r->L[l].in, 4);
            ok = dalloc(r, &a, (size_t)r->L[l].out * ld) && dalloc(r, &b, (size_t)r->L[l].out * ld);
            r->wt_f.push_back(a); r->wt_g.push_back(b); r->ld_wt.push_back(ld);
        }
    }
    if (ok) ok = cudaMemcpyAsync(r->idx, cfg->h_idx, sizeof(int) * r->ns, cudaMemcpyHostToDevice, r->stream) == cudaSuccess &&
                 cudaStreamSynchronize(r->stream) == cudaSuccess;
    if (!ok) {
        g_rnd_create_error = std::string("device allocation failed: ") + cudaGetErrorString(cudaGetLastError());
        rslrl_rnd_destroy(r);
        return RSLRL_ERR_CUDA;
    }
    *out = r;
    return RSLRL_OK;
}

rslrl_status rslrl_rnd_set_params(rslrl_rnd* r, const float* h_predictor, const float* h_target, size_t n) {
    if (!r || !h_predictor || !h_target) return RSLRL_ERR_INVALID_ARG;
    if (n != r->P_flat) return rfail(r, RSLRL_ERR_SHAPE, "expected %zu parameters, got %zu", r->P_flat, n);
    std::vector<float> dev((size_t)r->P_dev);
    for (int net = 0; net < 2; ++net) {
        const float* h = net == 0 ? h_predictor : h_target;
        std::fill(dev.begin(), dev.end(), 0.f);
        for (const RLayer& Ly : r->L) {
            for (int i = 0; i < Ly.in; ++i)
                for (int o = 0; o < Ly.out; ++o) dev[Ly.w_off + (size_t)i * Ly.out_p + o] = h[Ly.w_flat + (size_t)i * Ly.out + o];
            for (int o = 0; o < Ly.out; ++o) dev[Ly.b_off + o] = h[Ly.b_flat + o];
        }
        RCU(r, cudaMemcpyAsync(net == 0 ? r->pf : r->pg, dev.data(), sizeof(float) * dev.size(), cudaMemcpyHostToDevice, r->stream));
        RCU(r, cudaStreamSynchronize(r->stream));
    }
    RCU(r, cudaMemsetAsync(r->m, 0, sizeof(float) * r->P_dev, r->stream));
    RCU(r, cudaMemsetAsync(r->v, 0, sizeof(float) * r->P_dev, r->stream));
    RCU(r, cudaMemsetAsync(r->grad, 0, sizeof(float) * r->P_dev, r->stream));
    if (r->tf32) {
        rslrl_status ts = refresh_transposes(r, 0);
        if (ts == RSLRL_OK) ts = refresh_transposes(r, 1);
        if (ts != RSLRL_OK) return ts;
    }
    RCU(r, cudaStreamSynchronize(r->stream));
    r->adam_step = 0;
    return RSLRL_OK;
}

static rslrl_status rnd_get_vec(rslrl_rnd* r, const float* d, float* h, size_t n) {
    if (!r || !h) return RSLRL_ERR_INVALID_ARG;
    if (n != r->P_flat) return rfail(r, RSLRL_ERR_SHAPE, "expected %zu parameters, got %zu", r->P_flat, n);
    std::vector<float> dev((size_t)r->P_dev);
    RCU(r, cudaMemcpyAsync(dev.data(), d, sizeof(float) * dev.size(), cudaMemcpyDeviceToHost, r->stream));
    int code = 0;
    if (r->tf32) RCU(r, cudaMemcpyAsync(&code, r->tc_error, sizeof(int), cudaMemcpyDeviceToHost, r->stream));
    RCU(r, cudaStreamSynchronize(r->stream));
    if (code != 0) {                     // reported once
        RCU(r, cudaMemsetAsync(r->tc_error, 0, sizeof(int), r->stream));
        return rfail(r, RSLRL_ERR_TIMEOUT, "a bounded wait in a tensor-core kernel expired (role %d)", code);
    }
    for (const RLayer& Ly : r->L) {
        for (int i = 0; i < Ly.in; ++i)
            for (int o = 0; o < Ly.out; ++o) h[Ly.w_flat + (size_t)i * Ly.out + o] = dev[Ly.w_off + (size_t)i * Ly.out_p + o];
        for (int o = 0; o < Ly.out; ++o) h[Ly.b_flat + o] = dev[Ly.b_off + o];
    }
    return RSLRL_OK;
}

rslrl_status rslrl_rnd_get_params(rslrl_rnd* r, float* h, size_t n) { return r ? rnd_get_vec(r, r->pf, h, n) : RSLRL_ERR_INVALID_ARG; }
rslrl_status rslrl_rnd_get_grads(rslrl_rnd* r, float* h, size_t n) { return r ? rnd_get_vec(r, r->grad, h, n) : RSLRL_ERR_INVALID_ARG; }

rslrl_status rslrl_rnd_reward(rslrl_rnd* r, const float* d_obs, int32_t rows, int32_t obs_stride, float weight,
                              float* d_rewards_inout, float* d_r_int_out) {
    if (!r || !d_obs) return RSLRL_ERR_INVALID_ARG;
    if (rows < 0 || obs_stride < r->cfg.obs_dim) return rfail(r, RSLRL_ERR_INVALID_ARG, "rows must be >= 0 and obs_stride >= obs_dim");
    if (rows > r->max_rows) return rfail(r, RSLRL_ERR_UNSUPPORTED, "rows = %d exceeds max_rows = %d", rows, r->max_rows);
    if (rows == 0 || (!d_rewards_inout && !d_r_int_out)) return RSLRL_OK;
    rslrl_status s = subset(r, d_obs, obs_stride, nullptr, rows);
    if (s != RSLRL_OK) return s;
    s = forward(r, rows, true, true, nullptr);
    if (s != RSLRL_OK) return s;
    LaunchScope scope_("rnd_error", r->stream);
    RCU(r, launch_chained(rnd_error_kernel, dim3((rows + 7) / 8), dim3(256), 0, r->stream, (const float*)r->hf.back(),
                          (const float*)r->hg.back(), (const int*)nullptr, r->ldE, r->E, (int)rows, weight, d_rewards_inout, d_r_int_out,
                          (float*)nullptr, 0.f, (float*)nullptr));
    return RSLRL_OK;
}

rslrl_status rslrl_rnd_update(rslrl_rnd* r, const float* d_obs, int32_t batch, int32_t obs_stride, int32_t epochs,
                              int32_t minibatches, uint64_t seed, uint32_t iteration, int32_t max_steps, float* h_mean_loss,
                              float* h_first_loss) {
    if (!r || !d_obs) return RSLRL_ERR_INVALID_ARG;
    if (batch < 1 || epochs < 1 || minibatches < 1 || obs_stride < r->cfg.obs_dim)
        return rfail(r, RSLRL_ERR_INVALID_ARG, "batch, epochs and minibatches must be positive and obs_stride >= obs_dim");
    if (batch % minibatches) return rfail(r, RSLRL_ERR_SHAPE, "batch = %d is not divisible by %d minibatches", batch, minibatches);
    const int rows = batch / minibatches;
    if (rows > r->max_rows) return rfail(r, RSLRL_ERR_UNSUPPORTED, "minibatch of %d rows exceeds max_rows = %d", rows, r->max_rows);
    long long nsteps = (long long)epochs * minibatches;
    if (max_steps > 0) nsteps = std::min<long long>(nsteps, max_steps);
    if (batch > r->cfg.max_batch || epochs > r->cfg.max_epochs || minibatches > r->cfg.max_minibatches)
        return rfail(r, RSLRL_ERR_UNSUPPORTED, "batch %d / epochs %d / minibatches %d exceed the limits given at creation (%d / %d / %d)",
                     batch, epochs, minibatches, r->cfg.max_batch, r->cfg.max_epochs, r->cfg.max_minibatches);
    RCU(r, launch_perm_epochs(seed, iteration, epochs, (uint32_t)batch, r->perm, r->stream));
    // the target is fixed: its outputs for all rows of the batch are computed once and looked up by the steps
    for (int r0 = 0; r0 < batch; r0 += r->max_rows) {
        const int n = std::min(r->max_rows, batch - r0);
        rslrl_status s = subset(r, d_obs + (size_t)r0 * obs_stride, obs_stride, nullptr, n);
        if (s != RSLRL_OK) return s;
        if ((s = forward(r, n, false, true, r->gall + (size_t)r0 * r->ldE)) != RSLRL_OK) return s;
    }
    const int splits = splits_for(rows);
    const int kchunk = kchunk_for(r, rows, splits);
    const int nloss = (rows + 7) / 8;
    const float scale = 1.0f / ((float)rows * (float)r->E);
    const rslrl_rnd_cfg& c = r->cfg;
    int done = 0;
    for (int e = 0; e < epochs && done < nsteps; ++e) {
        for (int k = 0; k < minibatches && done < nsteps; ++k, ++done) {
            const int* rows_idx = r->perm + (size_t)e * batch + (size_t)k * rows;
            rslrl_status s = subset(r, d_obs, obs_stride, rows_idx, rows, batch);
            if (s != RSLRL_OK) return s;
            if ((s = forward(r, rows, true, false, nullptr)) != RSLRL_OK) return s;
            {
                LaunchScope scope_("rnd_error", r->stream);
                RCU(r, launch_chained(rnd_error_kernel, dim3(nloss), dim3(256), 0, r->stream, (const float*)r->hf.back(),
                                      (const float*)r->gall, rows_idx, r->ldE, r->E, rows, 0.f, (float*)nullptr, (float*)nullptr,
                                      r->dz.back(), scale, r->loss_partials));
            }
            if ((s = backward(r, rows, splits, kchunk)) != RSLRL_OK) return s;
            r->adam_step++;
            const float c1 = (float)(1.0 / (1.0 - std::pow((double)c.adam_b1, (double)r->adam_step)));
            const float c2 = (float)(1.0 / (1.0 - std::pow((double)c.adam_b2, (double)r->adam_step)));
            LaunchScope scope_("rnd_adam", r->stream);
            RCU(r, launch_chained(rnd_adam_kernel, dim3(std::min(148 * 4, (r->P_dev + 255) / 256)), dim3(256), 0, r->stream,
                                  (const float*)r->partials, splits, (size_t)r->P_dev, r->grad, r->pf, r->m, r->v, r->P_dev,
                                  c.lr, c.adam_b1, c.adam_b2, c.adam_eps, c1, c2, (const float*)r->loss_partials, nloss,
                                  1.0f / (float)rows, r->step_loss + done));
            if (r->tf32 && (s = refresh_transposes(r, 0)) != RSLRL_OK) return s;      // the forward operands of the next step
        }
    }
    if (h_mean_loss || h_first_loss) {
        std::vector<float> h((size_t)done);
        RCU(r, cudaMemcpyAsync(h.data(), r->step_loss, sizeof(float) * done, cudaMemcpyDeviceToHost, r->stream));
        RCU(r, cudaStreamSynchronize(r->stream));
        double t = 0.0;
        for (float x : h) t += x;
        if (h_mean_loss) *h_mean_loss = (float)(t / done);
        if (h_first_loss) *h_first_loss = h[0];
    }
    return RSLRL_OK;
}

}  // extern "C"
