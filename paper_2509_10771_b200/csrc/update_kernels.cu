// Update-side kernels: keyed-permutation minibatch gather (with mirrored copies), the fused
// head + PPO loss + loss-gradient kernel, the deterministic gradient reduction, and the
// single-pass grad-norm / KL-adaptive learning rate / Adam kernel.
#include "common.cuh"
#include "kernels.h"
#include <algorithm>

namespace rslrl {

namespace {

constexpr float kHalfLog2Pi = 0.91893853320467274178f;

// =======================================================================================
// Gather.  One warp per minibatch row: the warp resolves the source transition through the
// Feistel shuffle, then streams the row (float4 per lane) into the minibatch buffers.
// =======================================================================================
template <bool BF16>
__device__ __forceinline__ void copy_obs_row(const float* __restrict__ src, int dim, int ld_src,
                                             float* __restrict__ dst, __nv_bfloat16* __restrict__ dst16,
                                             int ld_dst, const int* __restrict__ perm,
                                             const float* __restrict__ sign, int lane) {
    // ld_dst may exceed ld_src (the bf16 rows are padded further); pad columns are zero.
    if (perm == nullptr) {
        for (int c = lane * 4; c < ld_dst; c += 128) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c < ld_src) v = *reinterpret_cast<const float4*>(src + c);   // storage pad is zero
            if (BF16) {
                __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&lo);
                pk.y = *reinterpret_cast<uint32_t*>(&hi);
                *reinterpret_cast<uint2*>(dst16 + c) = pk;
            } else {
                *reinterpret_cast<float4*>(dst + c) = v;
            }
        }
    } else {
        for (int c = lane; c < ld_dst; c += 32) {
            const float v = c < dim ? sign[c] * src[perm[c]] : 0.f;
            if (BF16) dst16[c] = __float2bfloat16_rn(v);
            else dst[c] = v;
        }
    }
}

template <bool BF16>
__global__ void __launch_bounds__(256) gather_kernel(const GatherArgs a) {
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    PermKey pk{a.seed_lo, a.seed_hi, a.iteration, a.epoch, a.batch, feistel_half_bits(a.batch)};
    for (int j = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; j < a.Bmb; j += warps) {
        const uint32_t src = feistel_permute(pk, a.first + (uint32_t)j);
        const int t = (int)(src / (uint32_t)a.N);
        if (lane == 0) {
            if (a.rows_out) a.rows_out[j] = (int)src;
            a.logp_old[j] = a.logp[src];
            a.v_old[j] = a.values[src];
            a.ret[j] = a.returns[src];
            a.adv_mb[j] = a.adv[src];
        }
        const float* oa = a.obs_a + (size_t)src * a.sa;
        const int ldxa = BF16 ? a.ldxa16 : a.ldxa;
        copy_obs_row<BF16>(oa, a.Da, a.sa, a.x_a ? a.x_a + (size_t)j * ldxa : nullptr,
                           a.x_a16 ? a.x_a16 + (size_t)j * ldxa : nullptr, ldxa, nullptr, nullptr, lane);
        if (a.sym)
            copy_obs_row<BF16>(oa, a.Da, a.sa, a.x_a ? a.x_a + (size_t)(j + a.Bmb) * ldxa : nullptr,
                               a.x_a16 ? a.x_a16 + (size_t)(j + a.Bmb) * ldxa : nullptr, ldxa,
                               a.st.obs_perm, a.st.obs_sign, lane);
        if (!a.shared_obs) {
            const float* oc = a.obs_c + (size_t)src * a.sc;
            const int ldxc = BF16 ? a.ldxc16 : a.ldxc;
            copy_obs_row<BF16>(oc, a.Dc, a.sc, a.x_c ? a.x_c + (size_t)j * ldxc : nullptr,
                               a.x_c16 ? a.x_c16 + (size_t)j * ldxc : nullptr, ldxc, nullptr, nullptr, lane);
            if (a.sym)
                copy_obs_row<BF16>(oc, a.Dc, a.sc, a.x_c ? a.x_c + (size_t)(j + a.Bmb) * ldxc : nullptr,
                                   a.x_c16 ? a.x_c16 + (size_t)(j + a.Bmb) * ldxc : nullptr, ldxc,
                                   a.st.cobs_perm, a.st.cobs_sign, lane);
        }
        const float* act = a.actions + (size_t)src * a.as;
        for (int c = lane; c < a.as; c += 32) {
            a.act_mb[(size_t)j * a.as + c] = act[c];
            a.mu_old[(size_t)j * a.as + c] = a.mu[(size_t)src * a.as + c];
            a.sigma_old[(size_t)j * a.as + c] = a.sigma[(size_t)t * a.as + c];
            if (a.sym)
                a.act_mb[(size_t)(j + a.Bmb) * a.as + c] =
                    c < a.A ? a.st.act_sign[c] * act[a.st.act_perm[c]] : 0.f;
        }
    }
}

__global__ void perm_rows_kernel(PermKey pk, uint32_t first, int count, int* __restrict__ rows_out) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < count) rows_out[j] = (int)feistel_permute(pk, first + (uint32_t)j);
}

// =======================================================================================
// Head + loss.  One warp per minibatch row (and its mirrored twin).  Lane i owns action i
// (and i + 32): policy mean, log-density terms, dL/dmu.  The hidden row is read coalesced.
// =======================================================================================
constexpr int kHLThreads = 256;
constexpr int kHLWarps = kHLThreads / 32;
constexpr int kPartialStride = 8 + 2 * kMaxActions;   // [0..3] loss sums, [4] db_critic, [8..) db_actor, dlog_std

template <typename T>
__device__ __forceinline__ void head_fwd(const T* __restrict__ h, int n, const float* __restrict__ Ws,
                                         int ldws, const float* __restrict__ bias, int nout,
                                         float& out_lo, float& out_hi) {
    const int lane = threadIdx.x & 31;
    out_lo = 0.f; out_hi = 0.f;
    for (int o0 = 0; o0 < nout; o0 += 8) {
        float acc[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[q] = 0.f;
        for (int k = lane; k < n; k += 32) {
            const float hv = to_float(h[k]);
            const float* w = Ws + k * ldws + o0;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (o0 + q < nout) acc[q] = fmaf(hv, w[q], acc[q]);
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int o = o0 + q;
            if (o < nout) {
                const float val = warp_sum(acc[q]) + bias[o];
                if (lane == (o & 31)) { if (o < 32) out_lo = val; else out_hi = val; }
            }
        }
    }
}

// dZ[k] = ELU'(h[k]) * sum_i d_i W[k][i] for the lane's k = lane, lane+32, ...
template <typename T>
__device__ __forceinline__ void head_bwd(const T* __restrict__ h, int n, const float* __restrict__ Ws,
                                         int ldws, int nout, float d_lo, float d_hi, float alpha,
                                         T* __restrict__ dz, int ld_out_pad) {
    const int lane = threadIdx.x & 31;
    for (int k0 = 0; k0 < ld_out_pad; k0 += 128) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int i = 0; i < nout; ++i) {
            const float d = __shfl_sync(0xffffffffu, i < 32 ? d_lo : d_hi, i & 31);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int k = k0 + lane + 32 * q;
                if (k < n) acc[q] = fmaf(d, Ws[k * ldws + i], acc[q]);
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int k = k0 + lane + 32 * q;
            if (k < ld_out_pad) {
                float v = 0.f;
                if (k < n) v = acc[q] * elu_grad_from_h(to_float(h[k]), alpha);
                dz[k] = from_float<T>(v);
            }
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kHLThreads) head_loss_kernel(const HeadLossArgs a) {
    extern __shared__ float smem[];
    const HeadParams& hp = a.hp;
    const int ldwa_s = hp.ldwa + 1, ldwc_s = 2;       // odd / tiny strides: no bank conflicts
    float* Wa_s = smem;                                // [n_a][ldwa_s]
    float* Wc_s = Wa_s + hp.n_a * ldwa_s;              // [n_c][2]
    float* red = Wc_s + hp.n_c * ldwc_s;               // [kHLWarps][kPartialStride]
    for (int e = threadIdx.x; e < hp.n_a * hp.ldwa; e += kHLThreads) {
        const int k = e / hp.ldwa, i = e % hp.ldwa;
        Wa_s[k * ldwa_s + i] = hp.Wa[e];
    }
    for (int k = threadIdx.x; k < hp.n_c; k += kHLThreads) Wc_s[k * ldwc_s] = hp.Wc[(size_t)k * hp.ldwc];
    __syncthreads();

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int A = hp.A;
    const int R = a.sym ? 2 * a.Bmb : a.Bmb;
    const float inv_R = 1.0f / (float)R;
    const float inv_sym = 1.0f / ((float)a.Bmb * (float)A);
    // per-lane constants of actions i = lane, lane + 32
    float ls[2], inv_var[2];
    int aperm[2]; float asign[2];
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        const int i = lane + 32 * hf;
        ls[hf] = i < A ? hp.log_std[i] : 0.f;
        const float sg = expf(ls[hf]);
        inv_var[hf] = 1.0f / (sg * sg);
        aperm[hf] = (a.sym && i < A) ? a.act_perm[i] : i;
        asign[hf] = (a.sym && i < A) ? a.act_sign[i] : 1.f;
    }
    float s_surr = 0.f, s_val = 0.f, s_kl = 0.f, s_sym = 0.f, s_dbc = 0.f;
    float s_dba[2] = {0.f, 0.f}, s_dls[2] = {0.f, 0.f};

    const int warps_total = gridDim.x * kHLWarps;
    for (int j = blockIdx.x * kHLWarps + warp; j < a.Bmb; j += warps_total) {
        const float logp_old = a.logp_old[j], v_old = a.v_old[j], ret = a.ret[j], adv = a.adv[j];
        float mu_orig[2] = {0.f, 0.f};
        for (int copy = 0; copy < (a.sym ? 2 : 1); ++copy) {
            const int r = j + copy * a.Bmb;
            const T* ha = reinterpret_cast<const T*>(a.Ha) + (size_t)r * a.ldha;
            const T* hc = reinterpret_cast<const T*>(a.Hc) + (size_t)r * a.ldhc;
            float mu[2], v, unused;
            head_fwd(ha, hp.n_a, Wa_s, ldwa_s, hp.ba, A, mu[0], mu[1]);
            head_fwd(hc, hp.n_c, Wc_s, ldwc_s, hp.bc, 1, v, unused);
            v = __shfl_sync(0xffffffffu, v, 0);
            // ---- log-density, KL -------------------------------------------------------
            float act[2], lp = 0.f, kl = 0.f;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int i = lane + 32 * hf;
                act[hf] = 0.f;
                if (i < A) {
                    act[hf] = a.act_mb[(size_t)r * a.as + i];
                    const float d = act[hf] - mu[hf];
                    lp += -(d * d) * 0.5f * inv_var[hf] - ls[hf] - kHalfLog2Pi;
                    if (copy == 0) {
                        const float so = a.sigma_old[(size_t)j * a.as + i];
                        const float dm = a.mu_old[(size_t)j * a.as + i] - mu[hf];
                        kl += (ls[hf] - logf(so)) + (so * so + dm * dm) * 0.5f * inv_var[hf] - 0.5f;
                    }
                }
            }
            lp = warp_sum(lp);
            if (copy == 0) s_kl += warp_sum(kl);
            // ---- surrogate ------------------------------------------------------------
            const float ratio = expf(lp - logp_old);
            const float s1 = -adv * ratio;
            const float s2 = -adv * fminf(fmaxf(ratio, 1.0f - a.h.clip), 1.0f + a.h.clip);
            s_surr += fmaxf(s1, s2);
            const bool inside = ratio >= 1.0f - a.h.clip && ratio <= 1.0f + a.h.clip;
            const float dlogp = (inside || s1 > s2) ? s1 * inv_R : 0.f;
            // ---- value ----------------------------------------------------------------
            float dv;
            const float e1 = (v - ret) * (v - ret);
            if (a.h.use_clipped_value_loss) {
                const float vc = v_old + fminf(fmaxf(v - v_old, -a.h.value_clip), a.h.value_clip);
                const float e2 = (vc - ret) * (vc - ret);
                s_val += fmaxf(e1, e2);
                const bool vin = fabsf(v - v_old) <= a.h.value_clip;
                dv = (vin || e1 > e2) ? 2.0f * (v - ret) : 0.f;
            } else {
                s_val += e1;
                dv = 2.0f * (v - ret);
            }
            dv *= a.h.value_coef * inv_R;
            // ---- dL/dmu, dL/dlog_std, symmetry -----------------------------------------
            float dmu[2];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int i = lane + 32 * hf;
                dmu[hf] = 0.f;
                float tgt_src = 0.f;
                if (copy == 1) {
                    // target_i = sign_i * mu_orig[perm_i]; every lane takes part in the shuffle
                    const int p = aperm[hf];
                    const float lo = __shfl_sync(0xffffffffu, mu_orig[0], p & 31);
                    const float hi = __shfl_sync(0xffffffffu, mu_orig[1], p & 31);
                    tgt_src = p < 32 ? lo : hi;
                }
                if (i < A) {
                    const float d = act[hf] - mu[hf];
                    dmu[hf] = dlogp * d * inv_var[hf];
                    s_dls[hf] += dlogp * (d * d * inv_var[hf] - 1.0f);
                    if (copy == 1) {
                        const float diff = mu[hf] - asign[hf] * tgt_src;
                        s_sym += diff * diff;            // summed over lanes at the end
                        dmu[hf] += a.h.sym_coef * 2.0f * diff * inv_sym;
                    }
                    s_dba[hf] += dmu[hf];
                }
            }
            if (copy == 0) { mu_orig[0] = mu[0]; mu_orig[1] = mu[1]; }
            s_dbc += dv;
            // ---- outputs ---------------------------------------------------------------
            for (int hf = 0; hf < 2; ++hf) {
                const int i = lane + 32 * hf;
                if (i < a.lddmu) a.dmu[(size_t)r * a.lddmu + i] = dmu[hf];
                if (a.dmu16 && i < a.lddmu16) a.dmu16[(size_t)r * a.lddmu16 + i] = __float2bfloat16_rn(dmu[hf]);
                if (a.mu_out && i < a.as) a.mu_out[(size_t)r * a.as + i] = mu[hf];
            }
            if (lane < 4) a.dv[(size_t)r * 4 + lane] = lane == 0 ? dv : 0.f;
            if (a.dv16 && lane < a.lddv16) a.dv16[(size_t)r * a.lddv16 + lane] = __float2bfloat16_rn(lane == 0 ? dv : 0.f);
            if (a.v_out && lane == 0) a.v_out[r] = v;
            head_bwd(ha, hp.n_a, Wa_s, ldwa_s, A, dmu[0], dmu[1], a.h.alpha,
                     reinterpret_cast<T*>(a.dZa) + (size_t)r * a.lddza, a.lddza);
            head_bwd(hc, hp.n_c, Wc_s, ldwc_s, 1, dv, 0.f, a.h.alpha,
                     reinterpret_cast<T*>(a.dZc) + (size_t)r * a.lddzc, a.lddzc);
        }
    }
    // ---- block partials (fixed order over the warps) --------------------------------------
    s_sym = warp_sum(s_sym);
    float* my = red + warp * kPartialStride;
    if (lane == 0) {
        my[LS_SURR] = s_surr; my[LS_VALUE] = s_val; my[LS_KL] = s_kl; my[LS_SYM] = s_sym;
        my[4] = s_dbc;
    }
    my[8 + lane] = s_dba[0]; my[8 + 32 + lane] = s_dba[1];
    my[8 + kMaxActions + lane] = s_dls[0]; my[8 + kMaxActions + 32 + lane] = s_dls[1];
    __syncthreads();
    for (int e = threadIdx.x; e < kPartialStride; e += kHLThreads) {
        if (e >= 5 && e < 8) continue;
        float s = 0.f;
        for (int w = 0; w < kHLWarps; ++w) s += red[w * kPartialStride + e];
        a.block_partials[(size_t)blockIdx.x * kPartialStride + e] = s;
    }
}

// =======================================================================================
// Head partial finalisation: sums the head_loss block partials in block order and drops the
// head-bias / log_std gradients into split 0 of the weight-gradient partials, the loss sums
// into loss_sums.  One block.
// =======================================================================================
__global__ void __launch_bounds__(256) head_finalize_kernel(const float* __restrict__ block_partials,
                                                            int nblocks, float* __restrict__ partials0,
                                                            int off_ba, int off_logstd, int off_bc,
                                                            int A, float entropy_coef,
                                                            const float* __restrict__ log_std,
                                                            float* __restrict__ loss_sums) {
    if (threadIdx.x == 0) {   // policy entropy of the parameters this step's forward used
        float ent = 0.f;
        for (int i = 0; i < A; ++i) ent += 0.5f + kHalfLog2Pi + log_std[i];
        loss_sums[LS_COUNT] = ent;
    }
    // one warp per entry: lane l adds blocks l, l+32, ... in order, then a fixed shuffle tree
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int e = warp; e < kPartialStride; e += nwarps) {
        if (e >= 5 && e < 8) continue;
        if (e >= 8 && e < 8 + kMaxActions && e - 8 >= A) continue;
        if (e >= 8 + kMaxActions && e - 8 - kMaxActions >= A) continue;
        float s = 0.f;
        for (int b = lane; b < nblocks; b += 32) s += block_partials[(size_t)b * kPartialStride + e];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
        if (lane != 0) continue;
        if (e < LS_COUNT) loss_sums[e] = s;
        else if (e == 4) partials0[off_bc] = s;
        else if (e < 8 + kMaxActions) partials0[off_ba + e - 8] = s;
        else partials0[off_logstd + e - 8 - kMaxActions] = s - entropy_coef;
    }
}

// =======================================================================================
// Gradient reduction: grad[p] = sum over splits (fixed order), plus a per-block sum of squares.
// =======================================================================================
constexpr int kRedThreads = 256;
constexpr int kRedPerThread = 4;

__global__ void __launch_bounds__(kRedThreads) reduce_kernel(const ReduceArgs a) {
    const int base = (blockIdx.x * kRedThreads + threadIdx.x) * kRedPerThread;   // P is a multiple of 4
    float sq = 0.f;
    if (base < a.P) {
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sp = 0; sp < a.splits; ++sp) {
            const float4 v = *reinterpret_cast<const float4*>(a.partials + (size_t)sp * a.split_stride + base);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        *reinterpret_cast<float4*>(a.grad + base) = s;
        sq = (s.x * s.x + s.y * s.y) + (s.z * s.z + s.w * s.w);
    }
    sq = warp_sum(sq);
    __shared__ float ws[kRedThreads / 32];
    if ((threadIdx.x & 31) == 0) ws[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < kRedThreads / 32; ++w) t += ws[w];
        a.sumsq_partials[blockIdx.x] = t;
    }
}

// =======================================================================================
// Grad-norm clip + KL-adaptive learning rate + Adam, one pass over the parameters.  Every
// block derives the same scalars (norm, KL, new lr, step) from the same inputs in the same
// order; lr and the step count are double-buffered so no block reads what another writes.
// =======================================================================================
constexpr int kAdamThreads = 256;

__global__ void __launch_bounds__(kAdamThreads) adam_kernel(const AdamArgs a) {
    __shared__ float s_scal[4];   // clip coefficient, lr, bias corrections
    __shared__ int s_skip;
    if (threadIdx.x < 32) {
        float sq = 0.f;
        for (int i = threadIdx.x; i < a.nsumsq; i += 32) sq += a.sumsq_partials[i];
        sq = warp_sum(sq);
        if (threadIdx.x == 0) {
            const float gnorm = sqrtf(sq);
            const float surr = a.loss_sums[LS_SURR] * a.inv_rows_all;
            const float val = a.loss_sums[LS_VALUE] * a.inv_rows_all;
            const float kl = a.loss_sums[LS_KL] * a.inv_rows_orig;
            const float sym = a.loss_sums[LS_SYM] * a.inv_sym;
            float lr = a.lr_io[a.parity];
            const int step = a.step_io[a.parity] + 1;
            const bool finite = isfinite(gnorm) && isfinite(surr) && isfinite(val) && isfinite(kl);
            if (a.adaptive && finite) {
                if (kl > 2.0f * a.desired_kl) lr = fmaxf(a.lr_min, lr / a.lr_factor);
                else if (kl < 0.5f * a.desired_kl) lr = fminf(a.lr_max, lr * a.lr_factor);
            }
            s_scal[0] = fminf(1.0f, a.max_norm / (gnorm + 1e-6f));
            s_scal[1] = lr;
            // 1 - b^step in double: exact enough for any step count, computed once per block
            s_scal[2] = (float)(1.0 / (1.0 - pow((double)a.b1, (double)step)));
            s_scal[3] = (float)(1.0 / (1.0 - pow((double)a.b2, (double)step)));
            s_skip = finite ? 0 : 1;
            if (blockIdx.x == 0) {
                a.lr_io[a.parity ^ 1] = lr;
                a.step_io[a.parity ^ 1] = finite ? step : step - 1;
                a.stats_row[0] = surr; a.stats_row[1] = val; a.stats_row[2] = a.loss_sums[LS_COUNT];
                a.stats_row[3] = sym;
                a.stats_row[4] = kl; a.stats_row[5] = gnorm; a.stats_row[6] = lr;
                a.stats_row[7] = finite ? 0.f : 1.f;
            }
        }
    }
    __syncthreads();
    if (s_skip) return;          // non-finite step: parameters and moments stay untouched
    const float coef = s_scal[0], lr = s_scal[1], c1 = s_scal[2], c2 = s_scal[3];
    const int n4 = a.P / 4;
    for (int i = blockIdx.x * kAdamThreads + threadIdx.x; i < n4; i += gridDim.x * kAdamThreads) {
        const float4 g4 = reinterpret_cast<const float4*>(a.grad)[i];
        float4 p4 = reinterpret_cast<float4*>(a.param)[i];
        float4 m4 = reinterpret_cast<float4*>(a.m)[i];
        float4 v4 = reinterpret_cast<float4*>(a.v)[i];
        float g[4] = {g4.x, g4.y, g4.z, g4.w};
        float p[4] = {p4.x, p4.y, p4.z, p4.w};
        float m[4] = {m4.x, m4.y, m4.z, m4.w};
        float v[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float gc = g[q] * coef;
            m[q] = a.b1 * m[q] + (1.0f - a.b1) * gc;
            v[q] = a.b2 * v[q] + (1.0f - a.b2) * gc * gc;
            p[q] = p[q] - lr * (m[q] * c1) / (sqrtf(v[q] * c2) + a.eps);
        }
        reinterpret_cast<float4*>(a.param)[i] = make_float4(p[0], p[1], p[2], p[3]);
        reinterpret_cast<float4*>(a.m)[i] = make_float4(m[0], m[1], m[2], m[3]);
        reinterpret_cast<float4*>(a.v)[i] = make_float4(v[0], v[1], v[2], v[3]);
    }
}

}  // namespace

cudaError_t launch_gather(const GatherArgs& a, cudaStream_t s) {
    if (a.Bmb <= 0) return cudaSuccess;
    const int blocks = std::min((a.Bmb + 7) / 8, 148 * 8);
    LaunchScope scope_("gather", s);
    if (a.x_a16) gather_kernel<true><<<blocks, 256, 0, s>>>(a);
    else gather_kernel<false><<<blocks, 256, 0, s>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_perm_rows(uint64_t seed, uint32_t iteration, uint32_t epoch, uint32_t batch,
                             uint32_t first, int count, int* rows_out, cudaStream_t s) {
    if (count <= 0) return cudaSuccess;
    PermKey pk{(uint32_t)seed, (uint32_t)(seed >> 32), iteration, epoch, batch, feistel_half_bits(batch)};
    LaunchScope scope_("perm_rows", s);
    perm_rows_kernel<<<(count + 255) / 256, 256, 0, s>>>(pk, first, count, rows_out);
    return cudaGetLastError();
}

int head_loss_blocks(int Bmb) { return std::max(1, std::min((Bmb + kHLWarps - 1) / kHLWarps, 148 * 4)); }
int head_partial_stride() { return kPartialStride; }

cudaError_t launch_head_loss(const HeadLossArgs& a, cudaStream_t s) {
    const int blocks = head_loss_blocks(a.Bmb);
    const size_t smem = sizeof(float) * ((size_t)a.hp.n_a * (a.hp.ldwa + 1) + (size_t)a.hp.n_c * 2 +
                                         (size_t)kHLWarps * kPartialStride);
    LaunchScope scope_("head_loss", s);
    cudaError_t e;
    if (a.bf16_act) {
        e = cudaFuncSetAttribute(head_loss_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        head_loss_kernel<__nv_bfloat16><<<blocks, kHLThreads, smem, s>>>(a);
    } else {
        e = cudaFuncSetAttribute(head_loss_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        head_loss_kernel<float><<<blocks, kHLThreads, smem, s>>>(a);
    }
    return cudaGetLastError();
}

cudaError_t launch_head_finalize(const float* block_partials, int nblocks, float* partials0, int off_ba,
                                 int off_logstd, int off_bc, int A, float entropy_coef,
                                 const float* log_std, float* loss_sums, cudaStream_t s) {
    LaunchScope scope_("head_finalize", s);
    head_finalize_kernel<<<1, 256, 0, s>>>(block_partials, nblocks, partials0, off_ba, off_logstd, off_bc, A,
                                           entropy_coef, log_std, loss_sums);
    return cudaGetLastError();
}

int reduce_blocks(int P) { return (P + kRedThreads * kRedPerThread - 1) / (kRedThreads * kRedPerThread); }

cudaError_t launch_reduce(const ReduceArgs& a, cudaStream_t s) {
    LaunchScope scope_("grad_reduce", s);
    reduce_kernel<<<reduce_blocks(a.P), kRedThreads, 0, s>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_adam(const AdamArgs& a, cudaStream_t s) {
    const int blocks = std::max(1, std::min((a.P / 4 + kAdamThreads - 1) / kAdamThreads, 148 * 4));
    LaunchScope scope_("adam", s);
    adam_kernel<<<blocks, kAdamThreads, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace rslrl
