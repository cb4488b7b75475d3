// The C ABI of rslrl_b200: context, rollout storage, and the host-side sequencing of the
// kernels that make up act / gae / ppo_update.  No arithmetic of the method lives here.
#include "guard.h"
#include "../../include/rslrl_b200.h"
#include "common.cuh"
#include "kernels.h"
#include "umma.h"
#include "tf32.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

using namespace rslrl;

namespace {

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

struct Layer {
    int in, out, out_p;        // fan-in, fan-out, fan-out rounded up to 4
    size_t w_off, b_off;       // offsets in the padded device parameter vector
    size_t w_flat, b_flat;     // offsets in the caller's flat vector
};

struct Net {
    int nl = 0;                // layers including the head
    Layer L[kMaxLayers];
    int in_dim = 0, in_ld = 0;
    int hid_ld[kMaxLayers];    // row stride of the post-activation of hidden layer l
};

std::string g_create_error;

}  // namespace

namespace rslrl {
// Message returned by rslrl_last_error(NULL); used by entry points that have no context.
void set_global_error(const char* msg) { g_create_error = msg; }
}  // namespace rslrl

struct rslrl_ctx {
    rslrl_model_cfg mc;
    rslrl_ppo_cfg pc;
    cudaStream_t stream = nullptr;
    Net actor, critic;
    size_t logstd_off = 0, logstd_flat = 0;
    size_t P_flat = 0;
    int P_dev = 0;
    int prec = RSLRL_FP32;

    std::vector<void*> allocs;
    // parameters and optimiser
    float *param = nullptr, *grad = nullptr, *adam_m = nullptr, *adam_v = nullptr;
    float* lr_io = nullptr; int* step_io = nullptr; int parity = 0;
    // storage
    rslrl_storage st{};
    float* last_obs_c = nullptr;          // [N][sc] padded copy of o_T
    float* last_values = nullptr;         // [N]
    float* gae_scratch = nullptr;
    // act workspace
    void* act_h[2][kMaxLayers] = {};      // post-activations [N][ld] per net per hidden layer
    // update workspace
    int Bmb = 0, R = 0, splits = 1, kchunk = 0;
    float *x_a = nullptr, *x_c = nullptr;
    // gathered minibatch items, two sets: while one minibatch is worked on, the next is gathered
    float *act_mb[2] = {}, *mu_old[2] = {}, *sigma_old[2] = {};
    float *logp_old[2] = {}, *v_old[2] = {}, *ret_mb[2] = {}, *adv_mb[2] = {};
    cudaStream_t side = nullptr;          // the gather of the next minibatch runs here
    cudaEvent_t ev_ready = nullptr, ev_gathered[2] = {}, ev_consumed[2] = {};
    void* up_h[2][kMaxLayers] = {};
    void* up_dz[2][kMaxLayers] = {};
    float *dmu = nullptr, *dv = nullptr; int lddmu = 0;
    int* perm[2] = {};                    // [epochs][T*N] shuffles of one iteration; with a gather stream two sets, so that
                                          // the next iteration's are resolved while this one's are still being read
    int perm_cur = 0;                     // the set the current iteration reads
    uint32_t perm_iteration[2] = {0xFFFFFFFFu, 0xFFFFFFFFu};   // which iteration's shuffles each set holds (or is being filled with)
    cudaEvent_t ev_side_idle = nullptr;   // everything enqueued on the gather stream so far
    float *partials = nullptr, *block_partials = nullptr, *sumsq_partials = nullptr, *loss_sums = nullptr;
    float* stats_dev = nullptr; float* stats_host = nullptr; int max_stat_rows = 0;
    SymTables sym{};
    // host-variant staging
    float *stage_obs_a = nullptr, *stage_obs_c = nullptr, *stage_act = nullptr, *stage_rew = nullptr;
    uint8_t *stage_done = nullptr, *stage_to = nullptr;
    // rewards | dones | time-outs of one step, packed: pinned host copy and its device twin, so that
    // rslrl_record_step_host needs one transfer; the event marks the last transfer out of the host copy
    uint8_t *pack_host = nullptr, *pack_dev = nullptr;
    cudaEvent_t pack_sent = nullptr; bool pack_in_flight = false;
    // tensor-core engines (BF16 mode; TF32 mode: hidden-layer products on the FP32 mode's buffers)
    UmmaEngine* umma = nullptr;
    Tf32Engine* tf32 = nullptr;
    // host state
    int step = 0; bool act_pending = false; bool gae_done = false;
    uint32_t global_step = 0, iteration = 0;
    std::string err;
};

namespace {

rslrl_status fail(rslrl_ctx* c, rslrl_status s, const char* fmt, ...) {
    char buf[512];
    va_list ap; va_start(ap, fmt); vsnprintf(buf, sizeof buf, fmt, ap); va_end(ap);
    if (c) c->err = buf; else g_create_error = buf;
    return s;
}

#define CU(ctx, call)                                                                          \
    do {                                                                                       \
        cudaError_t e__ = (call);                                                              \
        if (e__ != cudaSuccess)                                                                \
            return fail(ctx, RSLRL_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e__)); \
    } while (0)

#define TRY(expr) do { rslrl_status s__ = (expr); if (s__ != RSLRL_OK) return s__; } while (0)

bool valid_model(const rslrl_model_cfg* m, std::string* why) {
    auto bad = [&](const char* s) { if (why) *why = s; return false; };
    if (!m) return bad("model config is null");
    if (m->num_envs <= 0 || m->num_steps <= 0) return bad("num_envs and num_steps must be positive");
    if (m->actor_obs_dim <= 0 || m->critic_obs_dim <= 0) return bad("observation dims must be positive");
    if (m->num_actions <= 0 || m->num_actions > kMaxActions) return bad("num_actions must be in 1..64");
    if (m->num_actor_hidden < 1 || m->num_actor_hidden > RSLRL_MAX_HIDDEN ||
        m->num_critic_hidden < 1 || m->num_critic_hidden > RSLRL_MAX_HIDDEN)
        return bad("number of hidden layers must be in 1..8");
    for (int i = 0; i < m->num_actor_hidden; ++i) if (m->actor_hidden[i] <= 0) return bad("hidden width must be positive");
    for (int i = 0; i < m->num_critic_hidden; ++i) if (m->critic_hidden[i] <= 0) return bad("hidden width must be positive");
    if (m->shared_obs && m->actor_obs_dim != m->critic_obs_dim) return bad("shared_obs needs equal observation dims");
    if (m->precision < RSLRL_FP32 || m->precision > RSLRL_BF16) return bad("unknown precision");
    return true;
}

void build_net(Net& n, int in_dim, const int32_t* hidden, int nh, int out_dim, size_t& dev_off, size_t& flat_off) {
    n.nl = nh + 1;
    n.in_dim = in_dim;
    n.in_ld = round_up(in_dim, 4);
    int in = in_dim;
    for (int l = 0; l < n.nl; ++l) {
        Layer& L = n.L[l];
        L.in = in;
        L.out = l < nh ? hidden[l] : out_dim;
        L.out_p = round_up(L.out, 4);
        L.w_off = dev_off; dev_off += (size_t)L.in * L.out_p;
        L.b_off = dev_off; dev_off += L.out_p;
        L.w_flat = flat_off; flat_off += (size_t)L.in * L.out;
        L.b_flat = flat_off; flat_off += L.out;
        n.hid_ld[l] = round_up(L.out, 8);      // activation rows are walked in 32-byte pieces
        in = L.out;
    }
}

template <typename T>
rslrl_status dev_alloc(rslrl_ctx* c, T** p, size_t count) {
    void* q = nullptr;
    const size_t bytes = std::max<size_t>(count, 1) * sizeof(T);
    CU(c, guarded_malloc(&q, bytes));
    c->allocs.push_back(q);
    CU(c, cudaMemsetAsync(q, 0, bytes, c->stream));
    *p = reinterpret_cast<T*>(q);
    return RSLRL_OK;
}

// flat (caller) <-> padded (device) parameter vectors
void flat_to_dev(const rslrl_ctx* c, const float* flat, std::vector<float>& dev) {
    dev.assign(c->P_dev, 0.f);
    const Net* nets[2] = {&c->actor, &c->critic};
    for (int ni = 0; ni < 2; ++ni)
        for (int l = 0; l < nets[ni]->nl; ++l) {
            const Layer& L = nets[ni]->L[l];
            for (int i = 0; i < L.in; ++i)
                for (int o = 0; o < L.out; ++o) dev[L.w_off + (size_t)i * L.out_p + o] = flat[L.w_flat + (size_t)i * L.out + o];
            for (int o = 0; o < L.out; ++o) dev[L.b_off + o] = flat[L.b_flat + o];
        }
    for (int i = 0; i < c->mc.num_actions; ++i) dev[c->logstd_off + i] = flat[c->logstd_flat + i];
}

void dev_to_flat(const rslrl_ctx* c, const std::vector<float>& dev, float* flat) {
    const Net* nets[2] = {&c->actor, &c->critic};
    for (int ni = 0; ni < 2; ++ni)
        for (int l = 0; l < nets[ni]->nl; ++l) {
            const Layer& L = nets[ni]->L[l];
            for (int i = 0; i < L.in; ++i)
                for (int o = 0; o < L.out; ++o) flat[L.w_flat + (size_t)i * L.out + o] = dev[L.w_off + (size_t)i * L.out_p + o];
            for (int o = 0; o < L.out; ++o) flat[L.b_flat + o] = dev[L.b_off + o];
        }
    for (int i = 0; i < c->mc.num_actions; ++i) flat[c->logstd_flat + i] = dev[c->logstd_off + i];
}

HeadParams head_params(const rslrl_ctx* c) {
    const Layer& ha = c->actor.L[c->actor.nl - 1];
    const Layer& hc = c->critic.L[c->critic.nl - 1];
    HeadParams hp;
    hp.Wa = c->param + ha.w_off; hp.ba = c->param + ha.b_off; hp.ldwa = ha.out_p;
    hp.Wc = c->param + hc.w_off; hp.bc = c->param + hc.b_off; hp.ldwc = hc.out_p;
    hp.log_std = c->param + c->logstd_off;
    hp.n_a = ha.in; hp.n_c = hc.in; hp.A = c->mc.num_actions;
    return hp;
}

void fill_setup(const rslrl_ctx* c, UmmaSetup& us) {
    us.model = c->mc; us.N = c->st.N; us.Bmb = c->Bmb; us.R = c->R; us.stream = c->stream;
    us.param = c->param; us.P_dev = c->P_dev; us.partials = c->partials; us.splits = c->splits;
    us.logstd_off = c->logstd_off;
    const Net* nets[2] = {&c->actor, &c->critic};
    for (int ni = 0; ni < 2; ++ni) {
        us.nl[ni] = nets[ni]->nl; us.in_dim[ni] = nets[ni]->in_dim;
        for (int l = 0; l < nets[ni]->nl; ++l) {
            us.in[ni][l] = nets[ni]->L[l].in; us.out[ni][l] = nets[ni]->L[l].out;
            us.out_p[ni][l] = nets[ni]->L[l].out_p;
            us.w_off[ni][l] = nets[ni]->L[l].w_off; us.b_off[ni][l] = nets[ni]->L[l].b_off;
        }
    }
}

// Hidden layers of the selected nets on `rows` rows, FP32 mode: one batched SIMT GEMM launch
// per layer.  x[net]: input [rows][in_ld]; h[net][l]: post-activations.
rslrl_status forward_hidden_fp32(rslrl_ctx* c, bool do_actor, bool do_critic, const float* xa, const float* xc,
                                 int rows, void* const h[2][kMaxLayers]) {
    const Net* nets[2] = {&c->actor, &c->critic};
    const float* x[2] = {xa, xc};
    const bool on[2] = {do_actor, do_critic};
    const int maxl = std::max(do_actor ? c->actor.nl - 1 : 0, do_critic ? c->critic.nl - 1 : 0);
    for (int l = 0; l < maxl; ++l) {
        GemmBatch b{};
        b.alpha = c->mc.elu_alpha;
        for (int ni = 0; ni < 2; ++ni) {
            if (!on[ni] || l >= nets[ni]->nl - 1) continue;
            const Layer& L = nets[ni]->L[l];
            GemmProblem& p = b.p[b.count++];
            p.A = l == 0 ? x[ni] : (const float*)h[ni][l - 1];
            p.lda = l == 0 ? nets[ni]->in_ld : nets[ni]->hid_ld[l - 1];
            p.B = c->param + L.w_off; p.ldb = L.out_p;
            p.C = (float*)h[ni][l]; p.ldc = nets[ni]->hid_ld[l];
            p.bias = c->param + L.b_off; p.aux = nullptr; p.ldaux = 0;
            p.M = rows; p.N = L.out; p.K = L.in; p.Cn = L.out_p;
            p.splits = 1; p.kchunk = round_up(L.in, 8); p.split_stride = 0;
        }
        if (b.count) CU(c, launch_sgemm(b, false, false, EPI_BIAS_ELU, c->stream));
    }
    return RSLRL_OK;
}

rslrl_status backward_fp32(rslrl_ctx* c) {
    const Net* nets[2] = {&c->actor, &c->critic};
    const float* x[2] = {c->x_a, c->mc.shared_obs ? c->x_a : c->x_c};
    const float* dhead[2] = {c->dmu, c->dv};
    const int ldhead[2] = {c->lddmu, 4};
    const int R = c->R;
    // head weight gradients: dW = H_last^T d_head (TF32 mode: with the other layers in the tensor-core launch below)
    if (!c->tf32) {
        GemmBatch b{};
        for (int ni = 0; ni < 2; ++ni) {
            const Net& n = *nets[ni];
            const Layer& L = n.L[n.nl - 1];
            GemmProblem& p = b.p[b.count++];
            p.A = (const float*)c->up_h[ni][n.nl - 2]; p.lda = n.hid_ld[n.nl - 2];
            p.B = dhead[ni]; p.ldb = ldhead[ni];
            p.C = c->partials + L.w_off; p.ldc = L.out_p;
            p.M = L.in; p.N = L.out; p.K = R; p.Cn = L.out_p;
            p.splits = c->splits; p.kchunk = c->kchunk; p.split_stride = c->P_dev;
        }
        CU(c, launch_sgemm(b, true, false, EPI_PLAIN, c->stream));
    }
    const int maxh = std::max(c->actor.nl - 1, c->critic.nl - 1);
    ColsumBatch cs{};                              // bias gradients of every hidden layer: one launch after the loop
    cs.splits = c->splits; cs.split_stride = c->P_dev; cs.is_bf16 = 0;
    for (int back = 0; back < maxh; ++back) {
        GemmBatch wg{}, dg{};
        dg.alpha = c->mc.elu_alpha;
        for (int ni = 0; ni < 2; ++ni) {
            const Net& n = *nets[ni];
            const int l = n.nl - 2 - back;         // hidden layer index, from the top
            if (l < 0) continue;
            const Layer& L = n.L[l];
            const float* dz = (const float*)c->up_dz[ni][l];
            const float* hin = l == 0 ? x[ni] : (const float*)c->up_h[ni][l - 1];
            const int ldin = l == 0 ? n.in_ld : n.hid_ld[l - 1];
            if (!c->tf32) {                         // TF32 mode: one tensor-core launch for all layers, below
                GemmProblem& p = wg.p[wg.count++];
                p.A = hin; p.lda = ldin; p.B = dz; p.ldb = n.hid_ld[l];
                p.C = c->partials + L.w_off; p.ldc = L.out_p;
                p.M = L.in; p.N = L.out; p.K = R; p.Cn = L.out_p;
                p.splits = c->splits; p.kchunk = c->kchunk; p.split_stride = c->P_dev;
            }
            ColsumProblem& q = cs.p[cs.count++];
            q.X = dz; q.out = c->partials + L.b_off; q.rows = R; q.n = L.out; q.ld = n.hid_ld[l];
            if (l > 0) {
                GemmProblem& d = dg.p[dg.count++];
                d.A = dz; d.lda = n.hid_ld[l];
                d.B = c->param + L.w_off; d.ldb = L.out_p;
                d.C = (float*)c->up_dz[ni][l - 1]; d.ldc = n.hid_ld[l - 1];
                d.aux = (const float*)c->up_h[ni][l - 1]; d.ldaux = n.hid_ld[l - 1];
                d.M = R; d.N = L.in; d.K = L.out; d.Cn = n.hid_ld[l - 1];
                d.splits = 1; d.kchunk = round_up(L.out, 8); d.split_stride = 0;
            }
        }
        if (wg.count) CU(c, launch_sgemm(wg, true, false, EPI_PLAIN, c->stream));
        if (dg.count) {
            if (c->tf32) CU(c, tf32_update_dgrad(c->tf32, back));
            else CU(c, launch_sgemm(dg, false, true, EPI_DELU, c->stream));
        }
    }
    if (cs.count) CU(c, launch_colsum(cs, c->stream));
    if (c->tf32) CU(c, tf32_update_wgrad(c->tf32));
    return RSLRL_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

// After a host synchronisation: did a bounded wait inside a tensor-core kernel expire?
rslrl_status check_engine(rslrl_ctx* c) {
    if (!c->umma && !c->tf32) return RSLRL_OK;
    int code = 0;
    if (c->umma) CU(c, umma_read_error(c->umma, &code));
    else CU(c, tf32_read_error(c->tf32, &code));
    if (code != 0) return fail(c, RSLRL_ERR_TIMEOUT, "a bounded wait in a tensor-core kernel expired (role %d)", code);
    return RSLRL_OK;
}

}  // namespace

// =========================================================================================
extern "C" {

size_t rslrl_num_params(const rslrl_model_cfg* m) {
    if (!valid_model(m, nullptr)) return 0;
    size_t n = 0;
    int in = m->actor_obs_dim;
    for (int i = 0; i < m->num_actor_hidden; ++i) { n += (size_t)in * m->actor_hidden[i] + m->actor_hidden[i]; in = m->actor_hidden[i]; }
    n += (size_t)in * m->num_actions + m->num_actions + m->num_actions;
    in = m->critic_obs_dim;
    for (int i = 0; i < m->num_critic_hidden; ++i) { n += (size_t)in * m->critic_hidden[i] + m->critic_hidden[i]; in = m->critic_hidden[i]; }
    n += (size_t)in + 1;
    return n;
}

const char* rslrl_last_error(const rslrl_ctx* c) { return c ? c->err.c_str() : g_create_error.c_str(); }

rslrl_status rslrl_destroy(rslrl_ctx* c) {
    if (!c) return RSLRL_ERR_INVALID_ARG;
    cudaStreamSynchronize(c->stream);
    if (c->side) { cudaStreamSynchronize(c->side); cudaStreamDestroy(c->side); }
    if (c->ev_ready) cudaEventDestroy(c->ev_ready);
    if (c->ev_side_idle) cudaEventDestroy(c->ev_side_idle);
    for (int b = 0; b < 2; ++b) {
        if (c->ev_gathered[b]) cudaEventDestroy(c->ev_gathered[b]);
        if (c->ev_consumed[b]) cudaEventDestroy(c->ev_consumed[b]);
    }
    if (c->umma) umma_destroy(c->umma);
    if (c->tf32) tf32_destroy(c->tf32);
    for (void* p : c->allocs) guarded_free(p);
    if (c->stats_host) cudaFreeHost(c->stats_host);
    if (c->pack_host) cudaFreeHost(c->pack_host);
    if (c->pack_sent) cudaEventDestroy(c->pack_sent);
    delete c;
    return RSLRL_OK;
}

rslrl_status rslrl_create(const rslrl_model_cfg* m, const rslrl_ppo_cfg* p, void* stream, rslrl_ctx** out) {
    if (!out) return fail(nullptr, RSLRL_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    std::string why;
    if (!valid_model(m, &why)) return fail(nullptr, RSLRL_ERR_INVALID_ARG, "%s", why.c_str());
    if (!p) return fail(nullptr, RSLRL_ERR_INVALID_ARG, "ppo config is null");
    if (p->epochs <= 0 || p->minibatches <= 0) return fail(nullptr, RSLRL_ERR_INVALID_ARG, "epochs and minibatches must be positive");
    const long long B = (long long)m->num_envs * m->num_steps;
    if (B >= (1ll << 30)) return fail(nullptr, RSLRL_ERR_UNSUPPORTED, "T*N must be below 2^30");
    if (B % p->minibatches) return fail(nullptr, RSLRL_ERR_SHAPE, "T*N = %lld is not divisible by %d minibatches", B, p->minibatches);
    if (p->sym_enable && (!p->h_sym_obs_perm || !p->h_sym_obs_sign || !p->h_sym_act_perm || !p->h_sym_act_sign ||
                          (!m->shared_obs && (!p->h_sym_cobs_perm || !p->h_sym_cobs_sign))))
        return fail(nullptr, RSLRL_ERR_INVALID_ARG, "symmetry enabled but a mirror table is null");
    if (p->sym_enable) {
        auto check = [](const int32_t* perm, int n) {
            for (int i = 0; i < n; ++i) if (perm[i] < 0 || perm[i] >= n) return false;
            return true;
        };
        if (!check(p->h_sym_obs_perm, m->actor_obs_dim) || !check(p->h_sym_act_perm, m->num_actions) ||
            (!m->shared_obs && !check(p->h_sym_cobs_perm, m->critic_obs_dim)))
            return fail(nullptr, RSLRL_ERR_INVALID_ARG, "a mirror permutation has an index out of range");
    }

    rslrl_ctx* c = new rslrl_ctx();
    c->mc = *m; c->pc = *p; c->stream = (cudaStream_t)stream; c->prec = m->precision;
    c->pc.h_sym_obs_perm = c->pc.h_sym_cobs_perm = c->pc.h_sym_act_perm = nullptr;
    c->pc.h_sym_obs_sign = c->pc.h_sym_cobs_sign = c->pc.h_sym_act_sign = nullptr;
    auto bail = [&](rslrl_status s) { g_create_error = c->err; rslrl_destroy(c); return s; };

    size_t dev_off = 0, flat_off = 0;
    build_net(c->actor, m->actor_obs_dim, m->actor_hidden, m->num_actor_hidden, m->num_actions, dev_off, flat_off);
    c->logstd_off = dev_off; dev_off += round_up(m->num_actions, 4);
    c->logstd_flat = flat_off; flat_off += m->num_actions;
    build_net(c->critic, m->critic_obs_dim, m->critic_hidden, m->num_critic_hidden, 1, dev_off, flat_off);
    c->P_dev = (int)dev_off; c->P_flat = flat_off;

    const int N = m->num_envs, T = m->num_steps, A = m->num_actions;
    const int sa = c->actor.in_ld, sc = c->critic.in_ld, as = round_up(A, 4);
    rslrl_status s;
#define A_(ptr, count) if ((s = dev_alloc(c, &(ptr), (size_t)(count))) != RSLRL_OK) return bail(s)
    A_(c->param, c->P_dev); A_(c->grad, c->P_dev); A_(c->adam_m, c->P_dev); A_(c->adam_v, c->P_dev);
    A_(c->lr_io, 2); A_(c->step_io, 2);
    // storage
    c->st.T = T; c->st.N = N; c->st.step = 0;
    c->st.obs_a_stride = sa; c->st.obs_c_stride = sc; c->st.act_stride = as;
    A_(c->st.obs_actor, (size_t)T * N * sa);
    if (m->shared_obs) c->st.obs_critic = c->st.obs_actor; else A_(c->st.obs_critic, (size_t)T * N * sc);
    A_(c->st.actions, (size_t)T * N * as); A_(c->st.mu, (size_t)T * N * as); A_(c->st.sigma, (size_t)T * as);
    A_(c->st.logp, (size_t)T * N); A_(c->st.values, (size_t)T * N); A_(c->st.rewards, (size_t)T * N);
    A_(c->st.returns, (size_t)T * N); A_(c->st.advantages, (size_t)T * N);
    A_(c->st.dones, (size_t)T * N); A_(c->st.timeouts, (size_t)T * N);
    A_(c->last_obs_c, (size_t)N * sc); A_(c->last_values, N);
    A_(c->gae_scratch, (size_t)3 * gae_scan_blocks(N));
    // update workspace
    c->Bmb = (int)(B / p->minibatches);
    c->R = p->sym_enable ? 2 * c->Bmb : c->Bmb;
    if (c->prec != RSLRL_BF16) {
        c->splits = std::max(1, std::min(32, c->R / 512));
    } else {
        // one wave of weight-gradient work items over the SMs; every problem has its own number of splits
        UmmaSetup probe{}; fill_setup(c, probe);
        c->splits = umma_wgrad_plan(probe).max_splits;
    }
    // rows per split: a multiple of the k-step of whichever kernel forms the weight gradients
    c->kchunk = round_up((c->R + c->splits - 1) / c->splits, c->prec == RSLRL_TF32 ? 32 : 8);
    c->lddmu = as;
    for (int b = 0; b < 2; ++b) {
        A_(c->act_mb[b], (size_t)c->R * as); A_(c->mu_old[b], (size_t)c->Bmb * as); A_(c->sigma_old[b], (size_t)c->Bmb * as);
        A_(c->logp_old[b], c->Bmb); A_(c->v_old[b], c->Bmb); A_(c->ret_mb[b], c->Bmb); A_(c->adv_mb[b], c->Bmb);
    }
    A_(c->dmu, (size_t)c->R * as); A_(c->dv, (size_t)c->R * 4);
    A_(c->perm[0], (size_t)B * p->epochs);
    A_(c->partials, (size_t)c->splits * c->P_dev);
    A_(c->block_partials, (size_t)std::max(head_loss_blocks(c->Bmb), 256) * head_partial_stride());
    A_(c->sumsq_partials, reduce_blocks(c->P_dev)); A_(c->loss_sums, 8);
    c->max_stat_rows = p->epochs * p->minibatches;
    A_(c->stats_dev, (size_t)c->max_stat_rows * 8);
    if (cudaMallocHost((void**)&c->stats_host, (size_t)c->max_stat_rows * 8 * sizeof(float)) != cudaSuccess) {
        c->err = "cudaMallocHost failed"; return bail(RSLRL_ERR_CUDA);
    }
    if (c->prec != RSLRL_BF16) {
        const Net* nets[2] = {&c->actor, &c->critic};
        A_(c->x_a, (size_t)c->R * sa);
        if (!m->shared_obs) A_(c->x_c, (size_t)c->R * sc);
        for (int ni = 0; ni < 2; ++ni)
            for (int l = 0; l < nets[ni]->nl - 1; ++l) {
                float* q;
                A_(q, (size_t)N * nets[ni]->hid_ld[l]); c->act_h[ni][l] = q;
                A_(q, (size_t)c->R * nets[ni]->hid_ld[l]); c->up_h[ni][l] = q;
                A_(q, (size_t)c->R * nets[ni]->hid_ld[l]); c->up_dz[ni][l] = q;
            }
        if (c->prec == RSLRL_TF32) {
            Tf32Setup ts{};
            ts.N = N; ts.R = c->R; ts.T = T; ts.stream = c->stream; ts.elu_alpha = m->elu_alpha; ts.param = c->param;
            for (int ni = 0; ni < 2; ++ni) {
                ts.nl[ni] = nets[ni]->nl; ts.in_dim[ni] = nets[ni]->in_dim; ts.in_ld[ni] = nets[ni]->in_ld;
                for (int l = 0; l < nets[ni]->nl; ++l) {
                    ts.in[ni][l] = nets[ni]->L[l].in; ts.out[ni][l] = nets[ni]->L[l].out; ts.out_p[ni][l] = nets[ni]->L[l].out_p;
                    ts.hid_ld[ni][l] = nets[ni]->hid_ld[l];
                    ts.w_off[ni][l] = nets[ni]->L[l].w_off; ts.b_off[ni][l] = nets[ni]->L[l].b_off;
                    ts.act_h[ni][l] = (float*)c->act_h[ni][l]; ts.up_h[ni][l] = (float*)c->up_h[ni][l]; ts.up_dz[ni][l] = (float*)c->up_dz[ni][l];
                }
            }
            ts.obs_storage[0] = c->st.obs_actor; ts.obs_stride[0] = sa;
            ts.obs_storage[1] = c->st.obs_critic; ts.obs_stride[1] = sc;
            ts.last_obs_c = c->last_obs_c;
            ts.x[0] = c->x_a; ts.x[1] = m->shared_obs ? c->x_a : c->x_c;
            ts.dhead[0] = c->dmu; ts.ld_dhead[0] = c->lddmu; ts.dhead[1] = c->dv; ts.ld_dhead[1] = 4;
            ts.partials = c->partials; ts.split_stride = c->P_dev; ts.splits = c->splits; ts.kchunk = c->kchunk;
            std::string terr;
            c->tf32 = tf32_create(ts, &terr);
            if (!c->tf32) { c->err = "tensor-core engine: " + terr; return bail(RSLRL_ERR_UNSUPPORTED); }
        }
    } else {
        UmmaSetup us{}; fill_setup(c, us);
        std::string uerr;
        c->umma = umma_create(us, &uerr);
        if (!c->umma) { c->err = "tensor-core engine: " + uerr; return bail(RSLRL_ERR_UNSUPPORTED); }
        {
            bool okv = cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) == cudaSuccess &&
                       cudaEventCreateWithFlags(&c->ev_ready, cudaEventDisableTiming) == cudaSuccess &&
                       cudaEventCreateWithFlags(&c->ev_side_idle, cudaEventDisableTiming) == cudaSuccess;
            for (int b = 0; b < 2 && okv; ++b)
                okv = cudaEventCreateWithFlags(&c->ev_gathered[b], cudaEventDisableTiming) == cudaSuccess &&
                      cudaEventCreateWithFlags(&c->ev_consumed[b], cudaEventDisableTiming) == cudaSuccess;
            if (!okv) { c->err = "could not create the gather stream"; return bail(RSLRL_ERR_CUDA); }
            A_(c->perm[1], (size_t)B * p->epochs);
        }
    }
    // staging for the host-buffer variants
    A_(c->stage_obs_a, (size_t)N * m->actor_obs_dim);
    A_(c->stage_obs_c, (size_t)N * m->critic_obs_dim);
    A_(c->stage_act, (size_t)N * as); A_(c->stage_rew, N); A_(c->stage_done, N); A_(c->stage_to, N);
    A_(c->pack_dev, (size_t)N * 6);
    if (cudaMallocHost((void**)&c->pack_host, (size_t)N * 6) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->pack_sent, cudaEventDisableTiming) != cudaSuccess) {
        c->err = "could not allocate the pinned staging buffer"; return bail(RSLRL_ERR_CUDA);
    }
    if (p->sym_enable) {
        auto up_i = [&](const int32_t* h, int n, const int** d) -> rslrl_status {
            int* q; TRY(dev_alloc(c, &q, n));
            CU(c, cudaMemcpyAsync(q, h, n * sizeof(int), cudaMemcpyHostToDevice, c->stream)); *d = q; return RSLRL_OK; };
        auto up_f = [&](const float* h, int n, const float** d) -> rslrl_status {
            float* q; TRY(dev_alloc(c, &q, n));
            CU(c, cudaMemcpyAsync(q, h, n * sizeof(float), cudaMemcpyHostToDevice, c->stream)); *d = q; return RSLRL_OK; };
        if ((s = up_i(p->h_sym_obs_perm, m->actor_obs_dim, &c->sym.obs_perm)) != RSLRL_OK) return bail(s);
        if ((s = up_f(p->h_sym_obs_sign, m->actor_obs_dim, &c->sym.obs_sign)) != RSLRL_OK) return bail(s);
        if ((s = up_i(p->h_sym_act_perm, A, &c->sym.act_perm)) != RSLRL_OK) return bail(s);
        if ((s = up_f(p->h_sym_act_sign, A, &c->sym.act_sign)) != RSLRL_OK) return bail(s);
        if (m->shared_obs) { c->sym.cobs_perm = c->sym.obs_perm; c->sym.cobs_sign = c->sym.obs_sign; }
        else {
            if ((s = up_i(p->h_sym_cobs_perm, m->critic_obs_dim, &c->sym.cobs_perm)) != RSLRL_OK) return bail(s);
            if ((s = up_f(p->h_sym_cobs_sign, m->critic_obs_dim, &c->sym.cobs_sign)) != RSLRL_OK) return bail(s);
        }
    }
#undef A_
    const float lr2[2] = {p->lr, p->lr};
    if (cudaMemcpyAsync(c->lr_io, lr2, sizeof lr2, cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess) {
        c->err = std::string("create: ") + cudaGetErrorString(cudaGetLastError());
        return bail(RSLRL_ERR_CUDA);
    }
    *out = c;
    return RSLRL_OK;
}

rslrl_status rslrl_storage_view(rslrl_ctx* c, rslrl_storage* out) {
    if (!c || !out) return RSLRL_ERR_INVALID_ARG;
    *out = c->st; out->step = c->step;
    return RSLRL_OK;
}

rslrl_status rslrl_set_params(rslrl_ctx* c, const float* h, size_t n) {
    if (!c || !h) return RSLRL_ERR_INVALID_ARG;
    if (n != c->P_flat) return fail(c, RSLRL_ERR_SHAPE, "expected %zu parameters, got %zu", c->P_flat, n);
    std::vector<float> dev;
    flat_to_dev(c, h, dev);
    CU(c, cudaMemcpyAsync(c->param, dev.data(), dev.size() * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    if (c->umma) CU(c, umma_refresh_weights(c->umma));
    if (c->tf32) CU(c, tf32_refresh_weights(c->tf32));
    return RSLRL_OK;
}

static rslrl_status get_vec(rslrl_ctx* c, const float* d, float* h, size_t n) {
    if (!c || !h) return RSLRL_ERR_INVALID_ARG;
    if (n != c->P_flat) return fail(c, RSLRL_ERR_SHAPE, "expected %zu parameters, got %zu", c->P_flat, n);
    std::vector<float> dev(c->P_dev);
    CU(c, cudaMemcpyAsync(dev.data(), d, dev.size() * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    dev_to_flat(c, dev, h);
    return check_engine(c);
}
rslrl_status rslrl_get_params(rslrl_ctx* c, float* h, size_t n) { return c ? get_vec(c, c->param, h, n) : RSLRL_ERR_INVALID_ARG; }
rslrl_status rslrl_get_grads(rslrl_ctx* c, float* h, size_t n) { return c ? get_vec(c, c->grad, h, n) : RSLRL_ERR_INVALID_ARG; }
rslrl_status rslrl_get_adam(rslrl_ctx* c, float* hm, float* hv, size_t n) {
    if (!c) return RSLRL_ERR_INVALID_ARG;
    TRY(get_vec(c, c->adam_m, hm, n));
    return get_vec(c, c->adam_v, hv, n);
}
rslrl_status rslrl_set_adam(rslrl_ctx* c, const float* hm, const float* hv, size_t n) {
    if (!c || !hm || !hv) return RSLRL_ERR_INVALID_ARG;
    if (n != c->P_flat) return fail(c, RSLRL_ERR_SHAPE, "expected %zu parameters, got %zu", c->P_flat, n);
    std::vector<float> dev;
    flat_to_dev(c, hm, dev);
    CU(c, cudaMemcpyAsync(c->adam_m, dev.data(), dev.size() * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    flat_to_dev(c, hv, dev);
    CU(c, cudaMemcpyAsync(c->adam_v, dev.data(), dev.size() * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    return RSLRL_OK;
}

rslrl_status rslrl_get_counters(rslrl_ctx* c, rslrl_counters* out) {
    if (!c || !out) return RSLRL_ERR_INVALID_ARG;
    CU(c, cudaMemcpyAsync(&out->lr, c->lr_io + c->parity, sizeof(float), cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaMemcpyAsync(&out->adam_step, c->step_io + c->parity, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    out->global_step = c->global_step; out->iteration = c->iteration;
    return RSLRL_OK;
}

rslrl_status rslrl_set_counters(rslrl_ctx* c, const rslrl_counters* in) {
    if (!c || !in) return RSLRL_ERR_INVALID_ARG;
    if (!(in->lr > 0.f) || in->adam_step < 0) return fail(c, RSLRL_ERR_INVALID_ARG, "lr must be positive and adam_step non-negative");
    CU(c, cudaMemcpyAsync(c->lr_io + c->parity, &in->lr, sizeof(float), cudaMemcpyHostToDevice, c->stream));
    CU(c, cudaMemcpyAsync(c->step_io + c->parity, &in->adam_step, sizeof(int), cudaMemcpyHostToDevice, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    c->global_step = in->global_step; c->iteration = in->iteration;
    return RSLRL_OK;
}

// ----------------------------------------------------------------------------------- act
rslrl_status rslrl_act(rslrl_ctx* c, const float* d_actor_obs, const float* d_critic_obs, float* d_actions_out) {
    if (!c || !d_actor_obs) return RSLRL_ERR_INVALID_ARG;
    if (!c->mc.shared_obs && !d_critic_obs) return fail(c, RSLRL_ERR_INVALID_ARG, "critic observations are null");
    if (!aligned4(d_actor_obs) || !aligned4(d_critic_obs) || !aligned4(d_actions_out))
        return fail(c, RSLRL_ERR_ALIGNMENT, "float buffers must be 4-byte aligned");
    if (c->step >= c->st.T) return fail(c, RSLRL_ERR_STATE, "rollout already holds T = %d steps", c->st.T);
    if (c->act_pending) return fail(c, RSLRL_ERR_STATE, "rslrl_record_step must follow rslrl_act");
    const int N = c->st.N, t = c->step, sa = c->st.obs_a_stride, sc = c->st.obs_c_stride, as = c->st.act_stride;
    float* oa = c->st.obs_actor + (size_t)t * N * sa;
    float* oc = c->st.obs_critic + (size_t)t * N * sc;
    ActOut out;
    out.actions = c->st.actions + (size_t)t * N * as; out.mu = c->st.mu + (size_t)t * N * as;
    out.sigma = c->st.sigma + (size_t)t * as; out.logp = c->st.logp + (size_t)t * N;
    out.values = c->st.values + (size_t)t * N; out.actions_out = d_actions_out; out.act_stride = as;
    const HeadParams hp = head_params(c);
    if (c->prec != RSLRL_BF16) {
        CU(c, launch_pad_rows(d_actor_obs, c->mc.actor_obs_dim, oa, sa, nullptr, 0, N, c->stream));
        if (!c->mc.shared_obs) CU(c, launch_pad_rows(d_critic_obs, c->mc.critic_obs_dim, oc, sc, nullptr, 0, N, c->stream));
        if (c->tf32) CU(c, tf32_act_forward(c->tf32, t, true));
        else TRY(forward_hidden_fp32(c, true, true, oa, oc, N, c->act_h));
        CU(c, launch_act_head(c->act_h[0][c->actor.nl - 2], c->actor.hid_ld[c->actor.nl - 2],
                              c->act_h[1][c->critic.nl - 2], c->critic.hid_ld[c->critic.nl - 2], false, hp, out, N,
                              c->pc.seed, c->global_step, c->stream));
    } else {
        const void *ha, *hc; int ldha, ldhc;
        bool heads_done = false;
        CU(c, umma_act_forward(c->umma, d_actor_obs, c->mc.shared_obs ? nullptr : d_critic_obs, oa,
                               c->mc.shared_obs ? nullptr : oc, sa, sc, true, out, hp.log_std, c->pc.seed, c->global_step,
                               &heads_done, &ha, &ldha, &hc, &ldhc));
        if (!heads_done) CU(c, launch_act_head(ha, ldha, hc, ldhc, true, hp, out, N, c->pc.seed, c->global_step, c->stream));
    }
    c->global_step++;
    c->act_pending = true;
    return RSLRL_OK;
}

rslrl_status rslrl_record_step(rslrl_ctx* c, const float* d_rewards, const uint8_t* d_dones, const uint8_t* d_timeouts) {
    if (!c || !d_rewards || !d_dones || !d_timeouts) return RSLRL_ERR_INVALID_ARG;
    if (!aligned4(d_rewards)) return fail(c, RSLRL_ERR_ALIGNMENT, "float buffers must be 4-byte aligned");
    if (!c->act_pending) return fail(c, RSLRL_ERR_STATE, "rslrl_act must precede rslrl_record_step");
    const int N = c->st.N; const size_t o = (size_t)c->step * N;
    CU(c, launch_record_step(d_rewards, d_dones, d_timeouts, c->st.rewards + o, c->st.dones + o, c->st.timeouts + o, N, c->stream));
    c->act_pending = false;
    c->step++;
    return RSLRL_OK;
}

// ----------------------------------------------------------------------------------- gae
rslrl_status rslrl_gae(rslrl_ctx* c, const float* d_last_critic_obs) {
    if (!c || !d_last_critic_obs) return RSLRL_ERR_INVALID_ARG;
    if (!aligned4(d_last_critic_obs)) return fail(c, RSLRL_ERR_ALIGNMENT, "float buffers must be 4-byte aligned");
    if (c->step != c->st.T || c->act_pending) return fail(c, RSLRL_ERR_STATE, "rslrl_gae needs exactly T = %d recorded steps (have %d)", c->st.T, c->step);
    const int N = c->st.N, T = c->st.T;
    const HeadParams hp = head_params(c);
    if (c->prec != RSLRL_BF16) {
        CU(c, launch_pad_rows(d_last_critic_obs, c->mc.critic_obs_dim, c->last_obs_c, c->st.obs_c_stride, nullptr, 0, N, c->stream));
        if (c->tf32) CU(c, tf32_act_forward(c->tf32, 0, false));
        else TRY(forward_hidden_fp32(c, false, true, nullptr, c->last_obs_c, N, c->act_h));
        CU(c, launch_value_head(c->act_h[1][c->critic.nl - 2], c->critic.hid_ld[c->critic.nl - 2], false, hp, c->last_values, N, c->stream));
    } else {
        const void *ha, *hc; int ldha, ldhc;
        bool heads_done = false;
        ActOut vout{};
        vout.values = c->last_values; vout.act_stride = c->st.act_stride;
        CU(c, umma_act_forward(c->umma, nullptr, d_last_critic_obs, nullptr, nullptr, 0, 0, false, vout, hp.log_std, c->pc.seed,
                               c->global_step, &heads_done, &ha, &ldha, &hc, &ldhc));
        if (!heads_done) CU(c, launch_value_head(hc, ldhc, true, hp, c->last_values, N, c->stream));
    }
    CU(c, launch_gae(c->st.rewards, c->st.values, c->st.dones, c->st.timeouts, c->last_values, c->st.returns,
                     c->st.advantages, T, N, c->pc.gamma, c->pc.lam, c->pc.normalize_adv, c->pc.adv_std_unbiased,
                     c->pc.adv_eps, c->gae_scratch, c->stream));
    c->gae_done = true;
    return RSLRL_OK;
}

// -------------------------------------------------------------------------------- update
// The epoch x minibatch loop.  d_expert == nullptr: the PPO update.  Otherwise the distillation step: the
// gathered "actions" are the expert's, the head/loss kernel regresses the policy mean on them, the critic
// and log_std get no gradient and the learning rate is not adapted.
static rslrl_status update_impl(rslrl_ctx* c, int32_t max_steps, rslrl_update_stats* h_stats, const float* d_expert) {
    const bool distill = d_expert != nullptr;
    const rslrl_ppo_cfg& pc = c->pc;
    const int N = c->st.N, T = c->st.T, A = c->mc.num_actions;
    const int total_steps = pc.epochs * pc.minibatches;
    const int nsteps = max_steps > 0 ? std::min(max_steps, total_steps) : total_steps;
    const HeadParams hp_base = head_params(c);
    const Layer& ha = c->actor.L[c->actor.nl - 1];
    const Layer& hc = c->critic.L[c->critic.nl - 1];
    // Minibatch `step` gathered into input set `buf` on stream `st`.
    auto enqueue_gather = [&](int step, int buf, cudaStream_t st) -> rslrl_status {
        const int e = step / pc.minibatches, k = step % pc.minibatches;
        GatherArgs g{};
        g.obs_a = c->st.obs_actor; g.obs_c = c->st.obs_critic; g.actions = distill ? d_expert : c->st.actions; g.mu = c->st.mu;
        g.sigma = c->st.sigma; g.logp = c->st.logp; g.values = c->st.values; g.returns = c->st.returns;
        g.adv = c->st.advantages;
        g.N = N; g.B = T * N; g.sa = c->st.obs_a_stride; g.sc = c->st.obs_c_stride; g.as = c->st.act_stride;
        g.Da = c->mc.actor_obs_dim; g.Dc = c->mc.critic_obs_dim; g.A = A; g.shared_obs = c->mc.shared_obs;
        g.x_a = c->x_a; g.x_c = c->x_c; g.ldxa = c->actor.in_ld; g.ldxc = c->critic.in_ld;
        if (c->umma) umma_gather_targets(c->umma, &g, buf);
        g.act_mb = c->act_mb[buf]; g.mu_old = c->mu_old[buf]; g.sigma_old = c->sigma_old[buf];
        g.logp_old = c->logp_old[buf]; g.v_old = c->v_old[buf]; g.ret = c->ret_mb[buf]; g.adv_mb = c->adv_mb[buf];
        g.rows = c->perm[c->perm_cur] + (size_t)e * T * N + (size_t)k * c->Bmb; g.Bmb = c->Bmb; g.sym = pc.sym_enable; g.st = c->sym;
        CU(c, launch_gather(g, st, step == 0 && st == c->side));
        return RSLRL_OK;
    };
    // With a gather stream, minibatch s+1 is gathered into the other input set while minibatch s is
    // worked on: the gather waits for the kernels that read that set two steps ago, the step for its gather.
    if (distill && c->umma) CU(c, umma_zero_critic_gradients(c->umma));
    const bool overlap = c->side != nullptr;
    if (overlap) {
        CU(c, cudaEventRecord(c->ev_ready, c->stream));           // advantages and returns are in storage
        CU(c, cudaStreamWaitEvent(c->side, c->ev_ready, 0));
    }
    // the shuffles of all epochs of this iteration, resolved in one launch (with a gather stream the update
    // before has already resolved them into the other set, beside its own kernels)
    if (c->perm_iteration[c->perm_cur] != c->iteration) {
        CU(c, launch_perm_epochs(pc.seed, c->iteration, pc.epochs, (uint32_t)(T * N), c->perm[c->perm_cur], overlap ? c->side : c->stream));
        c->perm_iteration[c->perm_cur] = c->iteration;
    }
    if (overlap) {
        TRY(enqueue_gather(0, 0, c->side));
        CU(c, cudaEventRecord(c->ev_gathered[0], c->side));
        // the next iteration's shuffles depend on the seed and the iteration number only: they go into the
        // other set now, behind the first gather and beside this update's kernels
        CU(c, launch_perm_epochs(pc.seed, c->iteration + 1, pc.epochs, (uint32_t)(T * N), c->perm[c->perm_cur ^ 1], c->side));
        c->perm_iteration[c->perm_cur ^ 1] = c->iteration + 1;
    }
    int done_steps = 0;
    for (int e = 0; e < pc.epochs && done_steps < nsteps; ++e) {
        for (int k = 0; k < pc.minibatches && done_steps < nsteps; ++k, ++done_steps) {
            // ---- gather -----------------------------------------------------------------
            const int buf = overlap ? (done_steps & 1) : 0;
            if (overlap) {
                if (done_steps + 1 < nsteps) {
                    if (done_steps >= 1) CU(c, cudaStreamWaitEvent(c->side, c->ev_consumed[buf ^ 1], 0));
                    TRY(enqueue_gather(done_steps + 1, buf ^ 1, c->side));
                    CU(c, cudaEventRecord(c->ev_gathered[buf ^ 1], c->side));
                }
                // the step's own input set: waited for here only at the first step; later steps wait right behind
                // the backward pass of the step before (below), so that a step's launches follow one another
                // without a stream operation in between
                if (done_steps == 0) CU(c, cudaStreamWaitEvent(c->stream, c->ev_gathered[buf], 0));
            } else {
                TRY(enqueue_gather(done_steps, 0, c->stream));
            }
            // ---- forward, heads, loss, backward ----------------------------------------------
            HeadLossArgs hl{};
            if (c->prec != RSLRL_BF16) {
                if (c->tf32) CU(c, tf32_update_forward(c->tf32));
                else TRY(forward_hidden_fp32(c, true, true, c->x_a, c->mc.shared_obs ? c->x_a : c->x_c, c->R, c->up_h));
                hl.Ha = c->up_h[0][c->actor.nl - 2]; hl.ldha = c->actor.hid_ld[c->actor.nl - 2];
                hl.Hc = c->up_h[1][c->critic.nl - 2]; hl.ldhc = c->critic.hid_ld[c->critic.nl - 2];
                hl.bf16_act = 0;
                hl.dZa = c->up_dz[0][c->actor.nl - 2]; hl.lddza = hl.ldha;
                hl.dZc = c->up_dz[1][c->critic.nl - 2]; hl.lddzc = hl.ldhc;
            } else {
                CU(c, umma_update_forward(c->umma, buf, distill));
                umma_head_loss_targets(c->umma, &hl);
            }
            hl.hp = hp_base;
            hl.act_mb = c->act_mb[buf]; hl.mu_old = c->mu_old[buf]; hl.sigma_old = c->sigma_old[buf]; hl.as = c->st.act_stride;
            hl.logp_old = c->logp_old[buf]; hl.v_old = c->v_old[buf]; hl.ret = c->ret_mb[buf]; hl.adv = c->adv_mb[buf];
            hl.act_sign = c->sym.act_sign; hl.act_perm = c->sym.act_perm;
            hl.Bmb = c->Bmb; hl.sym = pc.sym_enable; hl.distill = distill ? 1 : 0;
            hl.h.clip = pc.clip; hl.h.value_clip = pc.value_clip; hl.h.value_coef = pc.value_coef;
            hl.h.entropy_coef = pc.entropy_coef; hl.h.sym_coef = pc.sym_coef; hl.h.alpha = c->mc.elu_alpha;
            hl.h.use_clipped_value_loss = pc.use_clipped_value_loss;
            hl.dmu = c->dmu; hl.lddmu = c->lddmu; hl.dv = c->dv;
            hl.block_partials = c->block_partials; hl.mu_out = nullptr; hl.v_out = nullptr;
            CU(c, launch_head_loss(hl, c->stream));
            // ---- backward ---------------------------------------------------------------
            if (c->prec != RSLRL_BF16) TRY(backward_fp32(c));
            else CU(c, umma_update_backward(c->umma, hl.colsum_written != 0, buf, distill));
            if (overlap) {
                CU(c, cudaEventRecord(c->ev_consumed[buf], c->stream));   // this input set may be refilled
                if (done_steps + 1 < nsteps) CU(c, cudaStreamWaitEvent(c->stream, c->ev_gathered[buf ^ 1], 0));   // the next step's inputs
            }
            // ---- reduce, clip, adaptive lr, Adam ------------------------------------------
            ReduceArgs r{};
            r.partials = c->partials; r.splits = c->splits; r.split_stride = c->P_dev;
            r.grad = c->grad; r.P = c->P_dev; r.sumsq_partials = c->sumsq_partials;
            r.block_partials = c->block_partials; r.nblocks = hl.nblocks_used;
            r.off_ba = (int)ha.b_off; r.off_logstd = (int)c->logstd_off; r.off_bc = (int)hc.b_off; r.A = A;
            r.entropy_coef = distill ? 0.f : pc.entropy_coef; r.log_std = c->param + c->logstd_off; r.loss_sums = c->loss_sums;
            if (c->umma) umma_fill_bias_sources(c->umma, &r, hl);
            CU(c, launch_reduce(r, c->stream));
            AdamArgs ad{};
            ad.param = c->param; ad.m = c->adam_m; ad.v = c->adam_v; ad.grad = c->grad; ad.P = c->P_dev;
            ad.sumsq_partials = c->sumsq_partials; ad.nsumsq = reduce_blocks(c->P_dev); ad.loss_sums = c->loss_sums;
            ad.inv_rows_all = 1.0f / (float)c->R; ad.inv_rows_orig = 1.0f / (float)c->Bmb;
            ad.inv_sym = 1.0f / ((float)c->Bmb * (float)A);
            ad.lr_io = c->lr_io; ad.step_io = c->step_io; ad.parity = c->parity;
            ad.lr_min = pc.lr_min; ad.lr_max = pc.lr_max; ad.lr_factor = pc.lr_factor; ad.desired_kl = pc.desired_kl;
            ad.adaptive = distill ? 0 : pc.adaptive_lr; ad.max_norm = pc.max_grad_norm;
            ad.b1 = pc.adam_b1; ad.b2 = pc.adam_b2; ad.eps = pc.adam_eps;
            ad.stats_row = c->stats_dev + (size_t)done_steps * 8;
            if (c->umma) umma_fill_cvt(c->umma, &ad);
            CU(c, launch_adam(ad, c->stream));
            if (c->tf32) CU(c, tf32_refresh_weights(c->tf32));
            c->parity ^= 1;
        }
    }
    c->iteration++;
    c->step = 0; c->gae_done = false; c->act_pending = false;
    if (overlap) {
        // join: whatever the gather stream still holds (the next iteration's shuffles when the update was cut
        // short) completes before anything the caller enqueues after this call
        c->perm_cur ^= 1;
        CU(c, cudaEventRecord(c->ev_side_idle, c->side));
        CU(c, cudaStreamWaitEvent(c->stream, c->ev_side_idle, 0));
    }
    if (h_stats) {
        CU(c, cudaMemcpyAsync(c->stats_host, c->stats_dev, (size_t)nsteps * 8 * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
        CU(c, cudaStreamSynchronize(c->stream));
        TRY(check_engine(c));
        rslrl_update_stats s{};
        const float* r0 = c->stats_host;
        for (int i = 0; i < nsteps; ++i) {
            const float* r = c->stats_host + (size_t)i * 8;
            s.surrogate += r[0]; s.value_loss += r[1]; s.entropy += r[2]; s.sym_loss += r[3]; s.kl += r[4];
            if (r[7] != 0.f) s.nonfinite = 1;
        }
        const float inv = 1.0f / (float)nsteps;
        s.surrogate *= inv; s.value_loss *= inv; s.entropy *= inv; s.sym_loss *= inv; s.kl *= inv;
        s.first_surrogate = r0[0]; s.first_value_loss = r0[1]; s.first_sym_loss = r0[3]; s.first_kl = r0[4];
        s.first_grad_norm = r0[5];
        s.last_grad_norm = c->stats_host[(size_t)(nsteps - 1) * 8 + 5];
        s.lr = c->stats_host[(size_t)(nsteps - 1) * 8 + 6];
        s.steps = nsteps;
        *h_stats = s;
        if (s.nonfinite) return fail(c, RSLRL_ERR_NONFINITE, "a loss or gradient norm was not finite; that step was skipped");
    }
    return RSLRL_OK;
}

rslrl_status rslrl_ppo_update_steps(rslrl_ctx* c, int32_t max_steps, rslrl_update_stats* h_stats) {
    if (!c) return RSLRL_ERR_INVALID_ARG;
    if (!c->gae_done) return fail(c, RSLRL_ERR_STATE, "rslrl_gae must precede rslrl_ppo_update");
    return update_impl(c, max_steps, h_stats, nullptr);
}

rslrl_status rslrl_ppo_update(rslrl_ctx* c, rslrl_update_stats* h_stats) { return rslrl_ppo_update_steps(c, 0, h_stats); }

rslrl_status rslrl_distill_update_steps(rslrl_ctx* c, const float* d_expert_actions, int32_t max_steps, rslrl_update_stats* h_stats) {
    if (!c || !d_expert_actions) return RSLRL_ERR_INVALID_ARG;
    if (!aligned4(d_expert_actions)) return fail(c, RSLRL_ERR_ALIGNMENT, "float buffers must be 4-byte aligned");
    if (c->pc.sym_enable) return fail(c, RSLRL_ERR_UNSUPPORTED, "distillation with symmetry augmentation is not available");
    if (c->step != c->st.T || c->act_pending)
        return fail(c, RSLRL_ERR_STATE, "rslrl_distill_update needs exactly T = %d recorded steps (have %d)", c->st.T, c->step);
    return update_impl(c, max_steps, h_stats, d_expert_actions);
}

rslrl_status rslrl_distill_update(rslrl_ctx* c, const float* d_expert_actions, rslrl_update_stats* h_stats) {
    return rslrl_distill_update_steps(c, d_expert_actions, 0, h_stats);
}

// ------------------------------------------------------------------------ host variants
rslrl_status rslrl_act_host(rslrl_ctx* c, const float* h_actor_obs, const float* h_critic_obs, float* h_actions_out) {
    if (!c || !h_actor_obs) return RSLRL_ERR_INVALID_ARG;
    if (!c->mc.shared_obs && !h_critic_obs) return fail(c, RSLRL_ERR_INVALID_ARG, "critic observations are null");
    const int N = c->st.N, A = c->mc.num_actions, as = c->st.act_stride;
    CU(c, cudaMemcpyAsync(c->stage_obs_a, h_actor_obs, (size_t)N * c->mc.actor_obs_dim * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    if (!c->mc.shared_obs)
        CU(c, cudaMemcpyAsync(c->stage_obs_c, h_critic_obs, (size_t)N * c->mc.critic_obs_dim * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    TRY(rslrl_act(c, c->stage_obs_a, c->mc.shared_obs ? nullptr : c->stage_obs_c, h_actions_out ? c->stage_act : nullptr));
    if (h_actions_out) {
        if (A == as)
            CU(c, cudaMemcpyAsync(h_actions_out, c->stage_act, (size_t)N * A * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
        else
            CU(c, cudaMemcpy2DAsync(h_actions_out, (size_t)A * sizeof(float), c->stage_act, (size_t)as * sizeof(float),
                                    (size_t)A * sizeof(float), N, cudaMemcpyDeviceToHost, c->stream));
        CU(c, cudaStreamSynchronize(c->stream));
    }
    return RSLRL_OK;
}

rslrl_status rslrl_record_step_host(rslrl_ctx* c, const float* h_rewards, const uint8_t* h_dones, const uint8_t* h_timeouts) {
    if (!c || !h_rewards || !h_dones || !h_timeouts) return RSLRL_ERR_INVALID_ARG;
    const int N = c->st.N;
    // one transfer instead of three: the three arrays are packed into the pinned buffer first (it is free
    // again once the transfer of the step before has left it)
    if (c->pack_in_flight) CU(c, cudaEventSynchronize(c->pack_sent));
    memcpy(c->pack_host, h_rewards, (size_t)N * sizeof(float));
    memcpy(c->pack_host + (size_t)N * 4, h_dones, (size_t)N);
    memcpy(c->pack_host + (size_t)N * 5, h_timeouts, (size_t)N);
    CU(c, cudaMemcpyAsync(c->pack_dev, c->pack_host, (size_t)N * 6, cudaMemcpyHostToDevice, c->stream));
    CU(c, cudaEventRecord(c->pack_sent, c->stream));
    c->pack_in_flight = true;
    return rslrl_record_step(c, reinterpret_cast<const float*>(c->pack_dev), c->pack_dev + (size_t)N * 4, c->pack_dev + (size_t)N * 5);
}

rslrl_status rslrl_gae_host(rslrl_ctx* c, const float* h_last_critic_obs) {
    if (!c || !h_last_critic_obs) return RSLRL_ERR_INVALID_ARG;
    CU(c, cudaMemcpyAsync(c->stage_obs_c, h_last_critic_obs, (size_t)c->st.N * c->mc.critic_obs_dim * sizeof(float),
                          cudaMemcpyHostToDevice, c->stream));
    return rslrl_gae(c, c->stage_obs_c);
}

// ------------------------------------------------------------------------ stand-alone
size_t rslrl_gae_scratch_bytes(int32_t T, int32_t N) {
    (void)T;
    return N > 0 ? (size_t)3 * gae_scan_blocks(N) * sizeof(float) : 0;
}

rslrl_status rslrl_gae_scan(const float* d_rewards, const float* d_values, const uint8_t* d_dones,
                            const uint8_t* d_timeouts, const float* d_last_values, float* d_returns,
                            float* d_advantages, int32_t T, int32_t N, float gamma, float lam, int32_t normalize,
                            int32_t unbiased, float adv_eps, void* d_scratch, void* stream) {
    if (T < 0 || N < 0) return RSLRL_ERR_INVALID_ARG;
    if (T == 0 || N == 0) return RSLRL_OK;
    if (!d_rewards || !d_values || !d_dones || !d_timeouts || !d_last_values || !d_returns || !d_advantages || !d_scratch)
        return RSLRL_ERR_INVALID_ARG;
    if ((long long)T * N >= (1ll << 31)) return RSLRL_ERR_UNSUPPORTED;
    if (!aligned16(d_advantages) || !aligned16(d_scratch)) return RSLRL_ERR_ALIGNMENT;
    cudaError_t e = launch_gae(d_rewards, d_values, d_dones, d_timeouts, d_last_values, d_returns, d_advantages, T, N,
                               gamma, lam, normalize, unbiased, adv_eps, (float*)d_scratch, (cudaStream_t)stream);
    return e == cudaSuccess ? RSLRL_OK : RSLRL_ERR_CUDA;
}

rslrl_status rslrl_minibatch_indices(uint64_t seed, uint32_t iteration, uint32_t epoch, int32_t batch,
                                     int32_t minibatches, int32_t k, int32_t* d_rows_out, void* stream) {
    if (batch < 0 || minibatches <= 0 || k < 0 || k >= minibatches) return RSLRL_ERR_INVALID_ARG;
    if (batch % minibatches) return RSLRL_ERR_SHAPE;
    if (batch == 0) return RSLRL_OK;
    if (!d_rows_out) return RSLRL_ERR_INVALID_ARG;
    const int rows = batch / minibatches;
    cudaError_t e = launch_perm_rows(seed, iteration, epoch, (uint32_t)batch, (uint32_t)k * (uint32_t)rows, rows,
                                     d_rows_out, (cudaStream_t)stream);
    return e == cudaSuccess ? RSLRL_OK : RSLRL_ERR_CUDA;
}

}  // extern "C"
