// Head + loss for BF16 activations on the warp-level tensor-core path (mma.sync m16n8k16).
//
// The policy head is a [rows x n] x [n x A] product with A <= 64: far too thin for the tcgen05
// tiles, but on the FP32 pipes it costs thousands of FMAs and shared-memory reads per row.
// Here a warp owns 16 rows: the head is 2 mma per 16 hidden units, the loss terms are finished in
// the accumulator layout (a row's actions sit in the four lanes of a quad), and dL/dz of the
// last hidden layer is again a thin product, [16 x A] x [A x n], whose result meets the stored
// post-activations in the same layout for the ELU derivative.  The critic head has one output:
// its dot product runs on the same fragments without mma.
//
// Accumulator layout of m16n8k16 (g = lane / 4, t = lane % 4): c0,c1 = row g, columns 2t, 2t+1;
// c2,c3 = row g+8, same columns.  A fragment: a0 = (row g, k 2t..2t+1), a1 = (row g+8, same k),
// a2 = (row g, k 8+2t..), a3 = (row g+8, k 8+2t..).  B fragment: b0 = (k 2t..2t+1, column g),
// b1 = (k 8+2t.., column g).
#include "common.cuh"
#include "kernels.h"
#include <algorithm>

namespace rslrl {

namespace {

constexpr float kHalfLog2Pi = 0.91893853320467274178f;
constexpr int kWarps = 4;
constexpr int kThreads = 32 * kWarps;
constexpr int kPartialStride = 8 + 2 * kMaxActions;   // must match update_kernels.cu

__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h2);
}
__device__ __forceinline__ float2 unpack_bf16(uint32_t w) {
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w));
}
__device__ __forceinline__ float quad_sum(float v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    return v;
}

// NT = number of 8-wide action tiles (actions padded to 8 * NT, NT even).
// CS: also emit the block's column sums of dZa / dZc (partial bias gradients of the last hidden layers).
template <int NT, bool CS>
__global__ void __launch_bounds__(kThreads, NT <= 6 ? 3 : 2) head_loss_mma_kernel(const HeadLossArgs a) {
    constexpr int AP = 8 * NT;
    extern __shared__ __align__(16) uint8_t smem_raw[];
    chain_begin();
    const HeadParams& hp = a.hp;
    const int A = hp.A;
    const int ksa = (hp.n_a + 15) / 16, ksc = (hp.n_c + 15) / 16;        // 16-wide steps over the hidden units
    const int ldk = 16 * ksa + 8;                                        // row stride of Wt_s (bf16), conflict-free
    const int lda = AP + 8;                                              // row stride of Wn_s (bf16)
    __nv_bfloat16* Wt_s = reinterpret_cast<__nv_bfloat16*>(smem_raw);    // [AP][ldk]      head weights, action-major
    __nv_bfloat16* Wn_s = Wt_s + AP * ldk;                               // [16 ksa][lda]  head weights, hidden-major
    float* Wc_s = reinterpret_cast<float*>(Wn_s + 16 * ksa * lda);       // [16 ksc]
    float* mu_s = Wc_s + 16 * ksc;                                       // [warps][16][AP + 1]
    float* red = mu_s + kWarps * 16 * (AP + 1);                          // [warps][kPartialStride]
    // [warps][8][cs_ld]: lane (g, t) keeps the running sums of its own columns of dZa | dZc
    const int cs_ld = (16 * (ksa + ksc) + 31) / 32 * 32 + 8;              // = 8 (mod 32): conflict-free float2 accesses
    float* cs_s = red + kWarps * kPartialStride;
    if (CS)
        for (int e = threadIdx.x; e < kWarps * 8 * cs_ld; e += kThreads) cs_s[e] = 0.f;
    for (int e = threadIdx.x; e < AP * 16 * ksa; e += kThreads) {
        const int i = e / (16 * ksa), k = e % (16 * ksa);
        const float w = (i < A && k < hp.n_a) ? hp.Wa[(size_t)k * hp.ldwa + i] : 0.f;
        Wt_s[i * ldk + k] = __float2bfloat16_rn(w);
        Wn_s[k * lda + i] = __float2bfloat16_rn(w);
    }
    for (int k = threadIdx.x; k < 16 * ksc; k += kThreads) Wc_s[k] = k < hp.n_c ? hp.Wc[(size_t)k * hp.ldwc] : 0.f;
    __syncthreads();

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int R = a.sym ? 2 * a.Bmb : a.Bmb;
    const float inv_R = 1.0f / (float)R;
    const float inv_sym = 1.0f / ((float)a.Bmb * (float)A);
    // the activation rows that are read and the gradient rows that are written never overlap
    const __nv_bfloat16* __restrict__ Ha = reinterpret_cast<const __nv_bfloat16*>(a.Ha);
    const __nv_bfloat16* __restrict__ Hc = reinterpret_cast<const __nv_bfloat16*>(a.Hc);
    __nv_bfloat16* __restrict__ dZa = reinterpret_cast<__nv_bfloat16*>(a.dZa);
    __nv_bfloat16* __restrict__ dZc = reinterpret_cast<__nv_bfloat16*>(a.dZc);
    float* mu_w = mu_s + warp * 16 * (AP + 1);
    float* cs_mine = cs_s + (warp * 8 + g) * cs_ld;

    // per-thread constants of its action columns: tile j -> actions 8j + 2t, 8j + 2t + 1
    float ls[NT][2], ivar[NT][2], var[NT][2], bias_a[NT][2];
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const int i = 8 * j + 2 * t + c;
            ls[j][c] = i < A ? hp.log_std[i] : 0.f;
            ivar[j][c] = __expf(-2.0f * ls[j][c]);
            var[j][c] = __expf(2.0f * ls[j][c]);
            bias_a[j][c] = i < A ? hp.ba[i] : 0.f;
        }
    const float bias_c = hp.bc[0];

    float s_surr = 0.f, s_val = 0.f, s_kl = 0.f, s_sym = 0.f, s_dbc = 0.f;
    float s_dba[NT][2], s_dls[NT][2];
#pragma unroll
    for (int j = 0; j < NT; ++j) { s_dba[j][0] = s_dba[j][1] = 0.f; s_dls[j][0] = s_dls[j][1] = 0.f; }

    const int tiles = (a.Bmb + 15) / 16;
    for (int tile = blockIdx.x * kWarps + warp; tile < tiles; tile += gridDim.x * kWarps) {
        const int j0 = tile * 16 + g, j1 = j0 + 8;                       // this thread's two minibatch rows
        const bool live0 = j0 < a.Bmb, live1 = j1 < a.Bmb;
        const int jc0 = live0 ? j0 : a.Bmb - 1, jc1 = live1 ? j1 : a.Bmb - 1;   // clamped for loads
        const float logp_old[2] = {a.logp_old[jc0], a.logp_old[jc1]};
        const float v_old[2] = {a.v_old[jc0], a.v_old[jc1]};
        const float ret[2] = {a.ret[jc0], a.ret[jc1]};
        const float adv[2] = {a.adv[jc0], a.adv[jc1]};
        for (int copy = 0; copy < (a.sym ? 2 : 1); ++copy) {
            const size_t r0 = (size_t)jc0 + (size_t)copy * a.Bmb, r1 = (size_t)jc1 + (size_t)copy * a.Bmb;
            const __nv_bfloat16* __restrict__ ha0 = Ha + r0 * a.ldha; const __nv_bfloat16* __restrict__ ha1 = Ha + r1 * a.ldha;
            const __nv_bfloat16* __restrict__ hc0 = Hc + r0 * a.ldhc; const __nv_bfloat16* __restrict__ hc1 = Hc + r1 * a.ldhc;
            // the per-action inputs of the loss terms, requested before the products so that they arrive meanwhile
            float act_in[NT][4], so_in[NT][4], mo_in[NT][4];
#pragma unroll
            for (int j = 0; j < NT; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i = 8 * j + 2 * t + (e & 1);
                    act_in[j][e] = so_in[j][e] = mo_in[j][e] = 0.f;
                    if (i < A) {
                        act_in[j][e] = a.act_mb[((e >> 1) ? r1 : r0) * a.as + i];
                        if (copy == 0 && !a.distill) {
                            const int jj = (e >> 1) ? jc1 : jc0;
                            so_in[j][e] = a.sigma_old[(size_t)jj * a.as + i];
                            mo_in[j][e] = a.mu_old[(size_t)jj * a.as + i];
                        }
                    }
                }
            // ---- heads ------------------------------------------------------------------------
            float mu[NT][4];
#pragma unroll
            for (int j = 0; j < NT; ++j) { mu[j][0] = mu[j][2] = bias_a[j][0]; mu[j][1] = mu[j][3] = bias_a[j][1]; }
#pragma unroll 8
            for (int ks = 0; ks < ksa; ++ks) {
                uint32_t af[4];
                af[0] = *reinterpret_cast<const uint32_t*>(ha0 + 16 * ks + 2 * t);
                af[1] = *reinterpret_cast<const uint32_t*>(ha1 + 16 * ks + 2 * t);
                af[2] = *reinterpret_cast<const uint32_t*>(ha0 + 16 * ks + 8 + 2 * t);
                af[3] = *reinterpret_cast<const uint32_t*>(ha1 + 16 * ks + 8 + 2 * t);
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    const __nv_bfloat16* wp = Wt_s + (8 * j + g) * ldk + 16 * ks + 2 * t;
                    mma_bf16(mu[j], af, *reinterpret_cast<const uint32_t*>(wp), *reinterpret_cast<const uint32_t*>(wp + 8));
                }
            }
            float v[2] = {0.f, 0.f};
#pragma unroll 8
            for (int ks = 0; ks < ksc; ++ks) {
                const float2 w01 = *reinterpret_cast<const float2*>(Wc_s + 16 * ks + 2 * t);
                const float2 w89 = *reinterpret_cast<const float2*>(Wc_s + 16 * ks + 8 + 2 * t);
                const float2 x0 = unpack_bf16(*reinterpret_cast<const uint32_t*>(hc0 + 16 * ks + 2 * t));
                const float2 x1 = unpack_bf16(*reinterpret_cast<const uint32_t*>(hc1 + 16 * ks + 2 * t));
                const float2 y0 = unpack_bf16(*reinterpret_cast<const uint32_t*>(hc0 + 16 * ks + 8 + 2 * t));
                const float2 y1 = unpack_bf16(*reinterpret_cast<const uint32_t*>(hc1 + 16 * ks + 8 + 2 * t));
                v[0] += x0.x * w01.x + x0.y * w01.y + y0.x * w89.x + y0.y * w89.y;
                v[1] += x1.x * w01.x + x1.y * w01.y + y1.x * w89.x + y1.y * w89.y;
            }
            v[0] = quad_sum(v[0]) + bias_c;
            v[1] = quad_sum(v[1]) + bias_c;
            // ---- per-row loss terms (h = 0: row g, h = 1: row g + 8) ----------------------------
            float dmu[NT][4];
            float lp[2] = {0.f, 0.f}, kl[2] = {0.f, 0.f}, sq[2] = {0.f, 0.f};
#pragma unroll
            for (int j = 0; j < NT; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int h = e >> 1, c = e & 1;
                    const int i = 8 * j + 2 * t + c;
                    dmu[j][e] = 0.f;
                    if (i < A) {
                        const float d = act_in[j][e] - mu[j][e];
                        if (a.distill) { sq[h] += d * d; dmu[j][e] = d; continue; }      // (a* - mu_i)^2
                        lp[h] += -(d * d) * 0.5f * ivar[j][c] - ls[j][c] - kHalfLog2Pi;
                        dmu[j][e] = d * ivar[j][c];                       // d logp / d mu_i
                        if (copy == 0) {
                            const float so = so_in[j][e];
                            const float dm = mo_in[j][e] - mu[j][e];
                            kl[h] += (ls[j][c] - logf(so)) + (so * so + dm * dm) * 0.5f * ivar[j][c] - 0.5f;
                        }
                    }
                }
            float dlogp[2], dv[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const bool live = h ? live1 : live0;
                const bool lead = t == 0 && live;                        // accounts the row once
                lp[h] = quad_sum(lp[h]);
                kl[h] = quad_sum(kl[h]);
                if (copy == 0 && lead) s_kl += kl[h];
                sq[h] = quad_sum(sq[h]);
                if (a.distill && lead) s_surr += sq[h] / (float)A;      // the row's mean squared error
                const float ratio = expf(lp[h] - logp_old[h]);
                const float s1 = -adv[h] * ratio;
                const float s2 = -adv[h] * fminf(fmaxf(ratio, 1.0f - a.h.clip), 1.0f + a.h.clip);
                if (lead && !a.distill) s_surr += fmaxf(s1, s2);
                const bool inside = ratio >= 1.0f - a.h.clip && ratio <= 1.0f + a.h.clip;
                dlogp[h] = (live && (inside || s1 > s2)) ? s1 * inv_R : 0.f;
                const float e1 = (v[h] - ret[h]) * (v[h] - ret[h]);
                float d;
                if (a.h.use_clipped_value_loss) {
                    const float vc = v_old[h] + fminf(fmaxf(v[h] - v_old[h], -a.h.value_clip), a.h.value_clip);
                    const float e2 = (vc - ret[h]) * (vc - ret[h]);
                    if (lead && !a.distill) s_val += fmaxf(e1, e2);
                    const bool vin = fabsf(v[h] - v_old[h]) <= a.h.value_clip;
                    d = (vin || e1 > e2) ? 2.0f * (v[h] - ret[h]) : 0.f;
                } else {
                    if (lead && !a.distill) s_val += e1;
                    d = 2.0f * (v[h] - ret[h]);
                }
                dv[h] = (live && !a.distill) ? d * a.h.value_coef * inv_R : 0.f;      // no critic term when distilling
                if (lead) s_dbc += dv[h];
            }
            // ---- dL/dmu, dL/dlog_std, symmetry ------------------------------------------------
            if (copy == 1) __syncwarp();                                  // mu of the original rows is in mu_w
#pragma unroll
            for (int j = 0; j < NT; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int h = e >> 1, c = e & 1;
                    const int i = 8 * j + 2 * t + c;
                    const bool live = h ? live1 : live0;
                    float gmu = 0.f;
                    if (i < A && live) {
                        const float dlp = dmu[j][e];
                        if (!a.distill) s_dls[j][c] += dlogp[h] * (dlp * dlp * var[j][c] - 1.0f);
                        gmu = a.distill ? -2.0f * dlp * inv_R / (float)A : dlogp[h] * dlp;
                        if (copy == 1) {
                            const float diff = mu[j][e] - a.act_sign[i] * mu_w[(g + 8 * h) * (AP + 1) + a.act_perm[i]];
                            s_sym += diff * diff;
                            gmu += a.h.sym_coef * 2.0f * diff * inv_sym;
                        }
                        s_dba[j][c] += gmu;
                    }
                    dmu[j][e] = gmu;
                }
            if (copy == 0 && a.sym) {
#pragma unroll
                for (int j = 0; j < NT; ++j)
#pragma unroll
                    for (int e = 0; e < 4; ++e) mu_w[(g + 8 * (e >> 1)) * (AP + 1) + 8 * j + 2 * t + (e & 1)] = mu[j][e];
            }
            // ---- row outputs ----------------------------------------------------------------------
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (!(h ? live1 : live0)) continue;
                const size_t r = h ? r1 : r0;
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    const int c0 = 8 * j + 2 * t;
                    if (c0 < a.lddmu) *reinterpret_cast<float2*>(a.dmu + r * a.lddmu + c0) = make_float2(dmu[j][2 * h], dmu[j][2 * h + 1]);
                    if (a.dmu16 && c0 < a.lddmu16)
                        *reinterpret_cast<uint32_t*>(a.dmu16 + r * a.lddmu16 + c0) = pack_bf16(dmu[j][2 * h], dmu[j][2 * h + 1]);
                    if (a.mu_out && c0 < a.as) *reinterpret_cast<float2*>(a.mu_out + r * a.as + c0) = make_float2(mu[j][2 * h], mu[j][2 * h + 1]);
                }
                if (t == 0) {
                    *reinterpret_cast<float4*>(a.dv + r * 4) = make_float4(dv[h], 0.f, 0.f, 0.f);
                    if (a.dv16) *reinterpret_cast<uint4*>(a.dv16 + r * a.lddv16) = make_uint4(pack_bf16(dv[h], 0.f), 0u, 0u, 0u);
                    if (a.v_out) a.v_out[r] = v[h];
                }
            }
            // ---- dL/dz of the actor's last hidden layer: [16 x AP] x [AP x n] --------------------------
            uint32_t df[NT / 2][4];                                       // dL/dmu as A fragments, one per 16 actions
#pragma unroll
            for (int ka = 0; ka < NT / 2; ++ka) {
                df[ka][0] = pack_bf16(dmu[2 * ka][0], dmu[2 * ka][1]);
                df[ka][1] = pack_bf16(dmu[2 * ka][2], dmu[2 * ka][3]);
                df[ka][2] = pack_bf16(dmu[2 * ka + 1][0], dmu[2 * ka + 1][1]);
                df[ka][3] = pack_bf16(dmu[2 * ka + 1][2], dmu[2 * ka + 1][3]);
            }
            __nv_bfloat16* __restrict__ dza0 = dZa + r0 * a.lddza; __nv_bfloat16* __restrict__ dza1 = dZa + r1 * a.lddza;
#pragma unroll 8
            for (int jn = 0; jn < 2 * ksa; ++jn) {                        // 8 hidden units per step
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ka = 0; ka < NT / 2; ++ka) {
                    const __nv_bfloat16* wp = Wn_s + (8 * jn + g) * lda + 16 * ka + 2 * t;
                    mma_bf16(acc, df[ka], *reinterpret_cast<const uint32_t*>(wp), *reinterpret_cast<const uint32_t*>(wp + 8));
                }
                const int col = 8 * jn + 2 * t;
                const float2 h0 = unpack_bf16(*reinterpret_cast<const uint32_t*>(ha0 + col));
                const float2 h1 = unpack_bf16(*reinterpret_cast<const uint32_t*>(ha1 + col));
                const float z00 = acc[0] * elu_grad_from_h(h0.x, a.h.alpha), z01 = acc[1] * elu_grad_from_h(h0.y, a.h.alpha);
                const float z10 = acc[2] * elu_grad_from_h(h1.x, a.h.alpha), z11 = acc[3] * elu_grad_from_h(h1.y, a.h.alpha);
                if (live0) *reinterpret_cast<uint32_t*>(dza0 + col) = pack_bf16(z00, z01);
                if (live1) *reinterpret_cast<uint32_t*>(dza1 + col) = pack_bf16(z10, z11);
                if (CS) {                                                 // rows that are not live carry dL/dmu = 0
                    float2* cs = reinterpret_cast<float2*>(cs_mine + col);
                    const float2 o = *cs;
                    *cs = make_float2(o.x + (z00 + z10), o.y + (z01 + z11));
                }
            }
            // ---- critic: dz = dV * Wc * ELU'(h), element-wise on the same column pairs ------------------
            __nv_bfloat16* __restrict__ dzc0 = dZc + r0 * a.lddzc; __nv_bfloat16* __restrict__ dzc1 = dZc + r1 * a.lddzc;
#pragma unroll 8
            for (int jn = 0; jn < 2 * ksc; ++jn) {
                const int col = 8 * jn + 2 * t;
                const float2 w = *reinterpret_cast<const float2*>(Wc_s + col);
                const float2 h0 = unpack_bf16(*reinterpret_cast<const uint32_t*>(hc0 + col));
                const float2 h1 = unpack_bf16(*reinterpret_cast<const uint32_t*>(hc1 + col));
                const float z00 = dv[0] * w.x * elu_grad_from_h(h0.x, a.h.alpha), z01 = dv[0] * w.y * elu_grad_from_h(h0.y, a.h.alpha);
                const float z10 = dv[1] * w.x * elu_grad_from_h(h1.x, a.h.alpha), z11 = dv[1] * w.y * elu_grad_from_h(h1.y, a.h.alpha);
                if (live0) *reinterpret_cast<uint32_t*>(dzc0 + col) = pack_bf16(z00, z01);
                if (live1) *reinterpret_cast<uint32_t*>(dzc1 + col) = pack_bf16(z10, z11);
                if (CS) {                                                 // rows that are not live carry dV = 0
                    float2* cs = reinterpret_cast<float2*>(cs_mine + 16 * ksa + col);
                    const float2 o = *cs;
                    *cs = make_float2(o.x + (z00 + z10), o.y + (z01 + z11));
                }
            }
            if (a.sym) __syncwarp();                                      // mu_w is rewritten by the next original rows
        }
    }
    // ---- block partials: lanes of equal t hold the same columns -> sum over g, then over the warps ----------
    float* mine = red + warp * kPartialStride;
    auto over_rows = [](float v) {
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        return v;
    };
    s_surr = warp_sum(s_surr); s_val = warp_sum(s_val); s_kl = warp_sum(s_kl); s_sym = warp_sum(s_sym); s_dbc = warp_sum(s_dbc);
    if (lane == 0) { mine[LS_SURR] = s_surr; mine[LS_VALUE] = s_val; mine[LS_KL] = s_kl; mine[LS_SYM] = s_sym; mine[4] = s_dbc; }
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const float ba = over_rows(s_dba[j][c]), dl = over_rows(s_dls[j][c]);
            const int i = 8 * j + 2 * t + c;
            if (g == 0 && i < kMaxActions) { mine[8 + i] = ba; mine[8 + kMaxActions + i] = dl; }
        }
    __syncthreads();
    for (int e = threadIdx.x; e < kPartialStride; e += kThreads) {
        if (e >= 5 && e < 8) continue;
        if (e >= 8 && ((e - 8) % kMaxActions) >= AP) continue;
        float s = 0.f;
        for (int w = 0; w < kWarps; ++w) s += red[w * kPartialStride + e];
        a.block_partials[(size_t)blockIdx.x * kPartialStride + e] = s;
    }
    if (CS) {
        // column sums of the block: the 8 row slots of each warp in order, then the warps in order
        for (int c = threadIdx.x; c < 16 * (ksa + ksc); c += kThreads) {
            float s = 0.f;
            for (int w = 0; w < kWarps * 8; ++w) s += cs_s[w * cs_ld + c];
            if (c < 16 * ksa) a.colsum_a[(size_t)blockIdx.x * a.lddza + c] = s;
            else a.colsum_c[(size_t)blockIdx.x * a.lddzc + (c - 16 * ksa)] = s;
        }
    }
}

constexpr size_t kMaxColsumSmem = 96 * 1024;   // above this the column sums are left to their own kernel

template <int NT>
cudaError_t launch_nt(HeadLossArgs& a, cudaStream_t s) {
    const int AP = 8 * NT;
    const int ksa = (a.hp.n_a + 15) / 16, ksc = (a.hp.n_c + 15) / 16;
    size_t smem = 2 * ((size_t)AP * (16 * ksa + 8) + (size_t)16 * ksa * (AP + 8)) +
                  4 * ((size_t)16 * ksc + (size_t)kWarps * 16 * (AP + 1) + (size_t)kWarps * kPartialStride);
    const size_t cs_bytes = 4 * (size_t)kWarps * 8 * ((16 * (ksa + ksc) + 31) / 32 * 32 + 8);
    const bool cs = a.colsum_a && a.colsum_c && cs_bytes <= kMaxColsumSmem;
    if (cs) smem += cs_bytes;
    a.colsum_written = cs ? 1 : 0;
    auto kernel = cs ? head_loss_mma_kernel<NT, true> : head_loss_mma_kernel<NT, false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int tiles = (a.Bmb + 15) / 16;
    const int blocks = std::max(1, std::min((tiles + kWarps - 1) / kWarps, 148 * 4));
    a.nblocks_used = blocks;
    LaunchScope scope_("head_loss", s);
    return launch_chained(kernel, blocks, kThreads, smem, s, a);
}

}  // namespace

bool head_loss_mma_applicable(const HeadLossArgs& a) {
    // BF16 activations whose rows cover the 16-wide steps the fragments read
    const int ksa = (a.hp.n_a + 15) / 16, ksc = (a.hp.n_c + 15) / 16;
    return a.bf16_act && a.hp.A <= kMaxActions && 16 * ksa <= a.ldha && 16 * ksc <= a.ldhc &&
           16 * ksa <= a.lddza && 16 * ksc <= a.lddzc && (a.ldha % 2) == 0 && (a.ldhc % 2) == 0 &&
           (a.lddmu % 2) == 0 && (a.as % 2) == 0 && 16 * ksa <= 1024;
}

cudaError_t launch_head_loss_mma(HeadLossArgs& a, cudaStream_t s) {
    const int nt = 2 * ((a.hp.A + 15) / 16);
    if (nt == 2) return launch_nt<2>(a, s);
    if (nt == 4) return launch_nt<4>(a, s);
    if (nt == 6) return launch_nt<6>(a, s);
    return launch_nt<8>(a, s);
}

}  // namespace rslrl
