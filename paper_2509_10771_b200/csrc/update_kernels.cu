// Update-side kernels: keyed-permutation minibatch gather (with mirrored copies), the fused
// head + PPO loss + loss-gradient kernel, the deterministic gradient reduction, and the
// single-pass grad-norm / KL-adaptive learning rate / Adam kernel.
#define RSLRL_INDEX_CHECKS
#include "guard.h"
#include "common.cuh"
#include "kernels.h"
#include <algorithm>

namespace rslrl {

namespace {

constexpr float kHalfLog2Pi = 0.91893853320467274178f;

// =======================================================================================
// Gather.  The epoch's shuffle is resolved once by perm_rows_kernel (one thread per index);
// here one warp per minibatch row reads its source index and streams the row (float4 per
// lane) into the minibatch buffers.
// =======================================================================================
// All loads of a row are issued before its first store: the destination arrays are plain
// pointers, so a store in between would order the loads behind it.
constexpr int kObsVec = 2;            // float4 pieces per lane held at once (32 lanes x 2 x 4 floats = 256 floats)

__device__ __forceinline__ void store_obs_piece(float* dst, __nv_bfloat16* dst16, int c, const float4 v) {
    if (dst16) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(dst16 + c) = pk;
    } else {
        *reinterpret_cast<float4*>(dst + c) = v;
    }
}

// Observation rows: a warp takes kGatherRows minibatch rows per pass and issues the loads of all of them before the
// first store; the row numbers of a pass are loaded during the pass before, and the rows of the next pass are
// prefetched into L2 meanwhile (one bulk prefetch per row and matrix, issued by one lane, no registers held).  The
// bandwidth of this kernel is the bytes it keeps in flight, so this loop carries nothing but the rows; the small
// per-row items are gathered by a second loop with one thread per row.  Storage is read through the read-only path
// (it does not change while an update runs).
// Two shapes of the kernel are launched.  The first gather of an update runs alone and, unless rows are mirrored, in
// the shape built for that: eight rows per pass, 256 threads, two blocks per SM.  The others run on a second stream beside the tensor-core
// kernels of the minibatch step before, whose CTAs hold an SM's shared memory and 55,296 of its 65,536
// registers: two rows per pass, 128 threads and at most 80 registers make a block that fits beside such a CTA
// (10,240 registers, no shared memory), so these gathers really run meanwhile instead of taking SMs in turn.
constexpr int kGatherRowsAlone = 8;
constexpr int kGatherRowsBeside = 2;

struct MirrorTables { int pc[kObsVec][4]; float sg[kObsVec][4]; };   // of one column block, the same for every row

__device__ __forceinline__ void load_mirror_tables(MirrorTables& t, const int* __restrict__ perm, const float* __restrict__ sign,
                                                   int dim, int c0, int lane) {
#pragma unroll
    for (int i = 0; i < kObsVec; ++i)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int c = c0 + 128 * i + lane * 4 + q;
            t.pc[i][q] = c < dim ? __ldg(perm + c) : 0;
            t.sg[i][q] = c < dim ? __ldg(sign + c) : 0.f;
        }
}

// float4 pieces of the column block at c0 of one storage row (pads of the storage row are zero)
__device__ __forceinline__ void load_obs_pieces(float4 (&v)[kObsVec], const float* __restrict__ row, int stride, int c0, int lane) {
#pragma unroll
    for (int i = 0; i < kObsVec; ++i) {
        const int c = c0 + 128 * i + lane * 4;
        v[i] = c < stride ? __ldg(reinterpret_cast<const float4*>(row + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

// Stores the pieces into minibatch row j and, when t is given, the mirror m[c] = sign[c] * row[perm[c]] into row
// j + Bmb (the row is read back through L1, where it has just landed); destination columns [dim, ld_dst) get zero.
__device__ __forceinline__ void store_obs_pieces(const float4 (&v)[kObsVec], const float* __restrict__ row, const MirrorTables* t,
                                                 float* x, __nv_bfloat16* x16, int ld_dst, size_t j, size_t Bmb, int c0, int lane) {
#pragma unroll
    for (int i = 0; i < kObsVec; ++i) {
        const int c = c0 + 128 * i + lane * 4;
        if (c >= ld_dst) continue;
        store_obs_piece(x16 ? nullptr : x + j * ld_dst, x16 ? x16 + j * ld_dst : nullptr, c, v[i]);
        if (t) {
            const float4 m = make_float4(t->sg[i][0] * __ldg(row + t->pc[i][0]), t->sg[i][1] * __ldg(row + t->pc[i][1]),
                                         t->sg[i][2] * __ldg(row + t->pc[i][2]), t->sg[i][3] * __ldg(row + t->pc[i][3]));
            store_obs_piece(x16 ? nullptr : x + (j + Bmb) * ld_dst, x16 ? x16 + (j + Bmb) * ld_dst : nullptr, c, m);
        }
    }
}

__device__ __forceinline__ void prefetch_row_l2(const float* row, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(row), "r"(bytes) : "memory");
}

template <int kGatherRows, int kBlockThreads, int kMinBlocks>
__global__ void __launch_bounds__(kBlockThreads, kMinBlocks) gather_kernel(const GatherArgs a) {
    chain_begin();
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const bool bf16 = a.x_a16 != nullptr;
    const int ldxa = bf16 ? a.ldxa16 : a.ldxa;
    const int first = ((blockIdx.x * blockDim.x + threadIdx.x) >> 5) * kGatherRows;
    // ---- observation rows: one sweep over the minibatch per matrix and block of 128 * kObsVec columns
    const int blocks_a = (ldxa + 128 * kObsVec - 1) / (128 * kObsVec);
    const int ldxc = bf16 ? a.ldxc16 : a.ldxc;
    const int sweeps = blocks_a + (a.shared_obs ? 0 : (ldxc + 128 * kObsVec - 1) / (128 * kObsVec));
    for (int sweep = 0; sweep < sweeps; ++sweep) {
        const bool critic = sweep >= blocks_a;
        const float* __restrict__ obs = critic ? a.obs_c : a.obs_a;
        const int stride = critic ? a.sc : a.sa, dim = critic ? a.Dc : a.Da, ld_dst = critic ? ldxc : ldxa;
        const int c0 = (critic ? sweep - blocks_a : sweep) * 128 * kObsVec;
        const int* perm = !a.sym ? nullptr : critic ? a.st.cobs_perm : a.st.obs_perm;
        float* x = critic ? a.x_c : a.x_a;
        __nv_bfloat16* x16 = critic ? a.x_c16 : a.x_a16;
        MirrorTables mt;
        if (perm) load_mirror_tables(mt, perm, critic ? a.st.cobs_sign : a.st.obs_sign, dim, c0, lane);
        uint32_t src[kGatherRows];
#pragma unroll
        for (int r = 0; r < kGatherRows; ++r)
            src[r] = first + r < a.Bmb ? checked_index((uint32_t)__ldg(a.rows + first + r), (uint32_t)a.B, 1) : 0u;
        for (int j0 = first; j0 < a.Bmb; j0 += warps * kGatherRows) {
            uint32_t nxt[kGatherRows];
#pragma unroll
            for (int r = 0; r < kGatherRows; ++r) {
                const int jn = j0 + warps * kGatherRows + r;
                nxt[r] = jn < a.Bmb ? (uint32_t)__ldg(a.rows + jn) : 0u;
            }
            float4 v[kGatherRows][kObsVec];
#pragma unroll
            for (int r = 0; r < kGatherRows; ++r) load_obs_pieces(v[r], obs + (size_t)src[r] * stride, stride, c0, lane);
            // the next pass's rows towards L2 (rows are 16-byte multiples at 16-byte aligned addresses)
            if (c0 == 0 && lane < kGatherRows && j0 + warps * kGatherRows + lane < a.Bmb) {
                uint32_t sn = nxt[0];
#pragma unroll
                for (int r = 1; r < kGatherRows; ++r) if (lane == r) sn = nxt[r];
                prefetch_row_l2(obs + (size_t)checked_index(sn, (uint32_t)a.B, 1) * stride, (uint32_t)stride * 4u);
            }
#pragma unroll
            for (int r = 0; r < kGatherRows; ++r)
                if (j0 + r < a.Bmb)
                    store_obs_pieces(v[r], obs + (size_t)src[r] * stride, perm ? &mt : nullptr, x, x16, ld_dst, (size_t)(j0 + r),
                                     (size_t)a.Bmb, c0, lane);
#pragma unroll
            for (int r = 0; r < kGatherRows; ++r) src[r] = checked_index(nxt[r], (uint32_t)a.B, 1);
        }
    }
    // ---- the small per-row items, one thread per minibatch row (action-sized rows are multiples of four floats)
    const int as4 = a.as >> 2;
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < a.Bmb; j += gridDim.x * blockDim.x) {
        const uint32_t s = checked_index((uint32_t)__ldg(a.rows + j), (uint32_t)a.B, 1);
        const int t = (int)(s / (uint32_t)a.N);
        const float lp = __ldg(a.logp + s), vl = __ldg(a.values + s), rt = __ldg(a.returns + s), ad = __ldg(a.adv + s);
        const float4* ac = reinterpret_cast<const float4*>(a.actions + (size_t)s * a.as);
        const float4* mu = reinterpret_cast<const float4*>(a.mu + (size_t)s * a.as);
        const float4* sg = reinterpret_cast<const float4*>(a.sigma + (size_t)t * a.as);
        float4* ac_o = reinterpret_cast<float4*>(a.act_mb + (size_t)j * a.as);
        float4* mu_o = reinterpret_cast<float4*>(a.mu_old + (size_t)j * a.as);
        float4* sg_o = reinterpret_cast<float4*>(a.sigma_old + (size_t)j * a.as);
        a.logp_old[j] = lp; a.v_old[j] = vl; a.ret[j] = rt; a.adv_mb[j] = ad;
        for (int q = 0; q < as4; ++q) {
            const float4 x = __ldg(ac + q), y = __ldg(mu + q), z = __ldg(sg + q);
            ac_o[q] = x; mu_o[q] = y; sg_o[q] = z;
        }
        if (a.sym) {
            float* am = a.act_mb + ((size_t)j + (size_t)a.Bmb) * a.as;
            const float* arow = a.actions + (size_t)s * a.as;
            for (int c = 0; c < a.as; ++c)
                am[c] = c < a.A ? __ldg(a.st.act_sign + c) * __ldg(arow + __ldg(a.st.act_perm + c)) : 0.f;
        }
    }
}

// rows_out[e * count + j] = shuffle of epoch (pk.epoch + e) at position first + j, e < epochs
__global__ void perm_rows_kernel(PermKey pk, uint32_t first, int count, int epochs, int* __restrict__ rows_out) {
    chain_begin();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= count) return;
    for (int e = blockIdx.y; e < epochs; e += gridDim.y) {
        PermKey k = pk;
        k.epoch = pk.epoch + (uint32_t)e;
        rows_out[(size_t)e * count + j] = (int)feistel_permute(k, first + (uint32_t)j);
    }
}

// =======================================================================================
// Head + loss.  Four threads per minibatch row (and its mirrored twin).  Thread q of the quad
// owns the actions 4q .. 4q+3 (+16 per further pass): all four walk the whole row of
// last-hidden activations in 16-byte pieces against head weights read from shared memory
// (the quad reads one contiguous 64-byte span, lanes of equal q broadcast), so the heads need
// no cross-lane traffic; the row's loss terms are finished with two shuffles; the backward walk
// ends in a transposing reduction that leaves every thread with one finished 16-byte piece
// of dL/dz to store.  NP = number of 16-action passes.
// =======================================================================================
constexpr int kHLThreads = 128;
constexpr int kHLRows = kHLThreads / 4;               // minibatch rows per block
constexpr int kPartialStride = 8 + 2 * kMaxActions;   // [0..3] loss sums, [4] db_critic, [8..) db_actor, dlog_std

__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&v)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
        w[e] = *reinterpret_cast<uint32_t*>(&h2);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}
__device__ __forceinline__ void store_piece(float* p, const float (&o)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(o[0], o[1], o[2], o[3]);
}
__device__ __forceinline__ void store_piece(__nv_bfloat16* p, const float (&o)[8]) { store8(p, o); }

// Four consecutive 16-byte pieces of an activation row, fetched with all loads in flight.
template <typename T>
struct RowBlock {
    static constexpr int EPV = 16 / (int)sizeof(T);     // elements per piece
    static constexpr int N = 4 * EPV;                   // elements per block
    uint4 v[4];
    __device__ __forceinline__ void load(const T* row, int k0, int ld) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            v[i] = k0 + i * EPV < ld ? *reinterpret_cast<const uint4*>(row + k0 + i * EPV) : make_uint4(0u, 0u, 0u, 0u);
    }
    __device__ __forceinline__ static void unpack(const uint4 x, float (&h)[EPV]) {
        if (sizeof(T) == 4) {
            h[0] = __uint_as_float(x.x); h[1] = __uint_as_float(x.y);
            h[2] = __uint_as_float(x.z); h[3] = __uint_as_float(x.w);
        } else {
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const __nv_bfloat162 h2 = *reinterpret_cast<const __nv_bfloat162*>(&w[e]);
                h[(2 * e) % EPV] = __low2float(h2); h[(2 * e + 1) % EPV] = __high2float(h2);
            }
        }
    }
    __device__ __forceinline__ uint4 pick(int q) const { return q == 0 ? v[0] : q == 1 ? v[1] : q == 2 ? v[2] : v[3]; }
};

// Block-wide sum in a fixed order: shuffle tree inside each warp, then the warps in order.
__device__ __forceinline__ float block_sum(float v, float* scratch /* [warps] */) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < kHLThreads / 32; ++w) t += scratch[w];
    return t;
}

template <typename T, int NP>
__global__ void __launch_bounds__(kHLThreads) head_loss_kernel(const HeadLossArgs a) {
    constexpr int AP = 16 * NP;                          // padded number of actions
    constexpr int AQ = 4 * NP;                           // actions per thread
    constexpr int EPV = RowBlock<T>::EPV;
    extern __shared__ float smem[];
    const HeadParams& hp = a.hp;
    const int A = hp.A;
    float* Wa_s = smem;                                  // [n_a][AP], zero padded
    float* Wc_s = Wa_s + hp.n_a * AP;                    // [n_c]
    float* mu_s = Wc_s + ((hp.n_c + 3) & ~3);            // [rows][AP + 1]  policy mean of the original row
    float* red = mu_s + kHLRows * (AP + 1);              // [warps]
    for (int e = threadIdx.x; e < hp.n_a * AP; e += kHLThreads) {
        const int k = e / AP, i = e % AP;
        Wa_s[e] = i < A ? hp.Wa[(size_t)k * hp.ldwa + i] : 0.f;
    }
    for (int k = threadIdx.x; k < hp.n_c; k += kHLThreads) Wc_s[k] = hp.Wc[(size_t)k * hp.ldwc];
    __syncthreads();

    const int qt = threadIdx.x & 3;                      // position in the quad
    const int row_local = threadIdx.x >> 2;
    const int j = blockIdx.x * kHLRows + row_local;
    const bool live = j < a.Bmb;
    const bool lead = qt == 0;                           // accounts the per-row scalars, writes dL/dV
    const unsigned qmask = 0xFu << (threadIdx.x & 28);   // the four lanes of this quad
    const int R = a.sym ? 2 * a.Bmb : a.Bmb;
    const float inv_R = 1.0f / (float)R;
    const float inv_sym = 1.0f / ((float)a.Bmb * (float)A);
    // slot s of this thread is action 16 (s / 4) + 4 qt + s % 4
    float ls[AQ], ivar[AQ];
#pragma unroll
    for (int s = 0; s < AQ; ++s) {
        const int i = 16 * (s >> 2) + 4 * qt + (s & 3);
        ls[s] = i < A ? hp.log_std[i] : 0.f;
        ivar[s] = __expf(-2.0f * ls[s]);                 // 1 / sigma^2
    }
    float s_surr = 0.f, s_val = 0.f, s_kl = 0.f, s_sym = 0.f, s_dbc = 0.f;
    float s_dba[AQ], s_dls[AQ];
#pragma unroll
    for (int s = 0; s < AQ; ++s) { s_dba[s] = 0.f; s_dls[s] = 0.f; }

    if (live) {
        const float logp_old = a.logp_old[j], v_old = a.v_old[j], ret = a.ret[j], adv = a.adv[j];
        float* mu_row = mu_s + row_local * (AP + 1);
        for (int copy = 0; copy < (a.sym ? 2 : 1); ++copy) {
            const int r = j + copy * a.Bmb;
            const T* ha = reinterpret_cast<const T*>(a.Ha) + (size_t)r * a.ldha;
            const T* hc = reinterpret_cast<const T*>(a.Hc) + (size_t)r * a.ldhc;
            RowBlock<T> blk;
            // ---- actor head: own actions over the whole row -------------------------------
            float mu[AQ];
#pragma unroll
            for (int s = 0; s < AQ; ++s) {
                const int i = 16 * (s >> 2) + 4 * qt + (s & 3);
                mu[s] = i < A ? hp.ba[i] : 0.f;
            }
            for (int k0 = 0; k0 < hp.n_a; k0 += RowBlock<T>::N) {     // row strides are multiples of 8
                blk.load(ha, k0, a.ldha);
#pragma unroll
                for (int pi = 0; pi < 4; ++pi) {
                    float h[EPV];
                    RowBlock<T>::unpack(blk.v[pi], h);
#pragma unroll
                    for (int kk = 0; kk < EPV; ++kk) {
                        const int k = k0 + pi * EPV + kk;
                        if (k < hp.n_a) {
#pragma unroll
                            for (int p = 0; p < NP; ++p) {
                                const float4 w = *reinterpret_cast<const float4*>(Wa_s + k * AP + 16 * p + 4 * qt);
                                mu[4 * p] = fmaf(h[kk], w.x, mu[4 * p]); mu[4 * p + 1] = fmaf(h[kk], w.y, mu[4 * p + 1]);
                                mu[4 * p + 2] = fmaf(h[kk], w.z, mu[4 * p + 2]); mu[4 * p + 3] = fmaf(h[kk], w.w, mu[4 * p + 3]);
                            }
                        }
                    }
                }
            }
            // ---- critic head: the quad splits the row, piece pi goes to thread pi -------------
            float v = 0.f;
            for (int k0 = 0; k0 < hp.n_c; k0 += RowBlock<T>::N) {
                const int kp = k0 + qt * EPV;
                if (kp < hp.n_c) {
                    float h[EPV];
                    RowBlock<T>::unpack(*reinterpret_cast<const uint4*>(hc + kp), h);
#pragma unroll
                    for (int kk = 0; kk < EPV; ++kk)
                        if (kp + kk < hp.n_c) v = fmaf(h[kk], Wc_s[kp + kk], v);
                }
            }
            v += __shfl_xor_sync(qmask, v, 1);
            v += __shfl_xor_sync(qmask, v, 2);
            v += hp.bc[0];
            // ---- log-density, KL (own actions, then two shuffles) --------------------------------
            float dmu[AQ];
            float lp = 0.f, kl = 0.f, sq = 0.f;
#pragma unroll
            for (int s = 0; s < AQ; ++s) {
                const int i = 16 * (s >> 2) + 4 * qt + (s & 3);
                dmu[s] = 0.f;
                if (i < A) {
                    const float d = a.act_mb[(size_t)r * a.as + i] - mu[s];
                    if (a.distill) {
                        sq += d * d;                                    // (a* - mu_i)^2
                        dmu[s] = d;
                        continue;
                    }
                    lp += -(d * d) * 0.5f * ivar[s] - ls[s] - kHalfLog2Pi;
                    dmu[s] = d * ivar[s];                               // d logp / d mu_i
                    if (copy == 0) {
                        const float so = a.sigma_old[(size_t)j * a.as + i];
                        const float dm = a.mu_old[(size_t)j * a.as + i] - mu[s];
                        kl += (ls[s] - logf(so)) + (so * so + dm * dm) * 0.5f * ivar[s] - 0.5f;
                    }
                }
            }
            lp += __shfl_xor_sync(qmask, lp, 1); lp += __shfl_xor_sync(qmask, lp, 2);
            kl += __shfl_xor_sync(qmask, kl, 1); kl += __shfl_xor_sync(qmask, kl, 2);
            if (copy == 0 && lead) s_kl += kl;
            if (a.distill) {
                sq += __shfl_xor_sync(qmask, sq, 1); sq += __shfl_xor_sync(qmask, sq, 2);
                if (lead) s_surr += sq / (float)A;                      // the row's mean squared error
            }
            // ---- surrogate ---------------------------------------------------------------
            const float ratio = expf(lp - logp_old);
            const float s1 = -adv * ratio;
            const float s2 = -adv * fminf(fmaxf(ratio, 1.0f - a.h.clip), 1.0f + a.h.clip);
            if (lead && !a.distill) s_surr += fmaxf(s1, s2);
            const bool inside = ratio >= 1.0f - a.h.clip && ratio <= 1.0f + a.h.clip;
            const float dlogp = (inside || s1 > s2) ? s1 * inv_R : 0.f;
            // ---- value -------------------------------------------------------------------
            float dv;
            const float e1 = (v - ret) * (v - ret);
            if (a.h.use_clipped_value_loss) {
                const float vc = v_old + fminf(fmaxf(v - v_old, -a.h.value_clip), a.h.value_clip);
                const float e2 = (vc - ret) * (vc - ret);
                if (lead && !a.distill) s_val += fmaxf(e1, e2);
                const bool vin = fabsf(v - v_old) <= a.h.value_clip;
                dv = (vin || e1 > e2) ? 2.0f * (v - ret) : 0.f;
            } else {
                if (lead && !a.distill) s_val += e1;
                dv = 2.0f * (v - ret);
            }
            dv *= a.h.value_coef * inv_R;
            if (a.distill) dv = 0.f;                                    // the critic takes no part
            if (lead) s_dbc += dv;
            // ---- dL/dmu, dL/dlog_std, symmetry -------------------------------------------
            if (copy == 1) __syncwarp(qmask);                           // mu of the original row is in mu_row
#pragma unroll
            for (int s = 0; s < AQ; ++s) {
                const int i = 16 * (s >> 2) + 4 * qt + (s & 3);
                if (i < A) {
                    const float dlp_dmu = dmu[s];                       // (a - mu) / sigma^2
                    if (!a.distill) s_dls[s] += dlogp * (dlp_dmu * dlp_dmu * __expf(2.0f * ls[s]) - 1.0f);
                    float g = a.distill ? -2.0f * dmu[s] * inv_R / (float)A : dlogp * dlp_dmu;
                    if (copy == 1) {
                        const float diff = mu[s] - a.act_sign[i] * mu_row[a.act_perm[i]];
                        s_sym += diff * diff;
                        g += a.h.sym_coef * 2.0f * diff * inv_sym;
                    }
                    dmu[s] = g;
                    s_dba[s] += g;
                }
            }
            if (copy == 0 && a.sym) {
#pragma unroll
                for (int s = 0; s < AQ; ++s) mu_row[16 * (s >> 2) + 4 * qt + (s & 3)] = mu[s];
            }
            // ---- row outputs -----------------------------------------------------------------
#pragma unroll
            for (int p = 0; p < NP; ++p) {
                const int c = 16 * p + 4 * qt;
                if (c < a.lddmu)
                    *reinterpret_cast<float4*>(a.dmu + (size_t)r * a.lddmu + c) =
                        make_float4(dmu[4 * p], dmu[4 * p + 1], dmu[4 * p + 2], dmu[4 * p + 3]);
                if (a.dmu16 && c < a.lddmu16) {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(dmu[4 * p], dmu[4 * p + 1]);
                    __nv_bfloat162 hi = __floats2bfloat162_rn(dmu[4 * p + 2], dmu[4 * p + 3]);
                    uint2 pk;
                    pk.x = *reinterpret_cast<uint32_t*>(&lo); pk.y = *reinterpret_cast<uint32_t*>(&hi);
                    *reinterpret_cast<uint2*>(a.dmu16 + (size_t)r * a.lddmu16 + c) = pk;
                }
                if (a.mu_out && c < a.as)
                    *reinterpret_cast<float4*>(a.mu_out + (size_t)r * a.as + c) =
                        make_float4(mu[4 * p], mu[4 * p + 1], mu[4 * p + 2], mu[4 * p + 3]);
            }
            if (lead) {
                *reinterpret_cast<float4*>(a.dv + (size_t)r * 4) = make_float4(dv, 0.f, 0.f, 0.f);
                if (a.dv16) {
                    const float d8[8] = {dv, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                    store8(a.dv16 + (size_t)r * a.lddv16, d8);
                }
                if (a.v_out) a.v_out[r] = v;
            }
            // ---- dL/dz of the actor's last hidden layer --------------------------------------------
            // every thread forms its actions' share of four pieces, then a transposing reduction
            // (exchange two pieces with lane^2, one with lane^1) leaves thread q with piece q
            T* dza = reinterpret_cast<T*>(a.dZa) + (size_t)r * a.lddza;
            for (int k0 = 0; k0 < a.lddza; k0 += RowBlock<T>::N) {
                blk.load(ha, k0, min(a.ldha, a.lddza));
                float part[4][EPV];
#pragma unroll
                for (int pi = 0; pi < 4; ++pi) {
#pragma unroll
                    for (int kk = 0; kk < EPV; ++kk) {
                        const int k = k0 + pi * EPV + kk;
                        float acc = 0.f;
                        if (k < hp.n_a) {
#pragma unroll
                            for (int p = 0; p < NP; ++p) {
                                const float4 w = *reinterpret_cast<const float4*>(Wa_s + k * AP + 16 * p + 4 * qt);
                                acc = fmaf(dmu[4 * p], w.x, acc); acc = fmaf(dmu[4 * p + 1], w.y, acc);
                                acc = fmaf(dmu[4 * p + 2], w.z, acc); acc = fmaf(dmu[4 * p + 3], w.w, acc);
                            }
                        }
                        part[pi][kk] = acc;
                    }
                }
                float half[2][EPV], tot[EPV];
#pragma unroll
                for (int pp = 0; pp < 2; ++pp) {
#pragma unroll
                    for (int kk = 0; kk < EPV; ++kk) {
                        const float send = (qt & 2) ? part[pp][kk] : part[pp + 2][kk];
                        const float keep = (qt & 2) ? part[pp + 2][kk] : part[pp][kk];
                        half[pp][kk] = keep + __shfl_xor_sync(qmask, send, 2);
                    }
                }
#pragma unroll
                for (int kk = 0; kk < EPV; ++kk) {
                    const float send = (qt & 1) ? half[0][kk] : half[1][kk];
                    const float keep = (qt & 1) ? half[1][kk] : half[0][kk];
                    tot[kk] = keep + __shfl_xor_sync(qmask, send, 1);
                }
                const int kp = k0 + qt * EPV;                            // thread q finishes piece q
                if (kp < a.lddza) {
                    float h[EPV], o[EPV];
                    RowBlock<T>::unpack(blk.pick(qt), h);
#pragma unroll
                    for (int kk = 0; kk < EPV; ++kk)
                        o[kk] = kp + kk < hp.n_a ? tot[kk] * elu_grad_from_h(h[kk], a.h.alpha) : 0.f;
                    store_piece(dza + kp, o);
                }
            }
            // ---- critic: thread q handles piece q of every block -------------------------------------
            T* dzc = reinterpret_cast<T*>(a.dZc) + (size_t)r * a.lddzc;
            for (int k0 = 0; k0 < a.lddzc; k0 += RowBlock<T>::N) {
                const int kp = k0 + qt * EPV;
                if (kp < a.lddzc) {
                    float h[EPV], o[EPV];
                    RowBlock<T>::unpack(kp < a.ldhc ? *reinterpret_cast<const uint4*>(hc + kp) : make_uint4(0u, 0u, 0u, 0u), h);
#pragma unroll
                    for (int kk = 0; kk < EPV; ++kk)
                        o[kk] = kp + kk < hp.n_c ? dv * Wc_s[kp + kk] * elu_grad_from_h(h[kk], a.h.alpha) : 0.f;
                    store_piece(dzc + kp, o);
                }
            }
        }
    }
    // ---- block partials (fixed order) ----------------------------------------------------------
    float* out = a.block_partials + (size_t)blockIdx.x * kPartialStride;
    float t;
    t = block_sum(s_surr, red); if (threadIdx.x == 0) out[LS_SURR] = t;
    t = block_sum(s_val, red);  if (threadIdx.x == 0) out[LS_VALUE] = t;
    t = block_sum(s_kl, red);   if (threadIdx.x == 0) out[LS_KL] = t;
    t = block_sum(s_sym, red);  if (threadIdx.x == 0) out[LS_SYM] = t;
    t = block_sum(s_dbc, red);  if (threadIdx.x == 0) out[4] = t;
#pragma unroll
    for (int i = 0; i < AP; ++i) {
        if (i < A) {                                    // uniform across the block
            const bool mine = qt == ((i & 15) >> 2);    // the quad member that owns action i
            constexpr int unused = 0; (void)unused;
            const int s = 4 * (i >> 4) + (i & 3);
            t = block_sum(mine ? s_dba[s] : 0.f, red); if (threadIdx.x == 0) out[8 + i] = t;
            t = block_sum(mine ? s_dls[s] : 0.f, red); if (threadIdx.x == 0) out[8 + kMaxActions + i] = t;
        }
    }
}

// =======================================================================================
// Gradient reduction: grad[p] = sum over splits (fixed order), plus a per-block sum of squares.
// The head-bias and log_std entries come from the head_loss block partials instead (summed in
// block order), and block 0 also finishes the loss sums and the policy entropy.
// =======================================================================================
constexpr int kRedThreads = 256;
constexpr int kRedPerThread = 4;

__device__ __forceinline__ bool head_entry(const ReduceArgs& a, int p) {
    return (p >= a.off_ba && p < a.off_ba + a.A) || (p >= a.off_logstd && p < a.off_logstd + a.A) || p == a.off_bc;
}
__device__ __forceinline__ bool bias_entry(const ReduceArgs& a, int p) {
    for (int b = 0; b < a.n_bias; ++b)
        if (p >= a.bias[b].p_off && p < a.bias[b].p_off + a.bias[b].n) return true;
    return false;
}
constexpr int kRedExtraBlocks = 96;     // blocks that finish the entries coming from partial rows: a warp per four columns

// grid = reduce_blocks(P) blocks over the parameter vector + one extra block for the entries
// that come from the head/loss kernel and for the loss sums.
__global__ void __launch_bounds__(kRedThreads) reduce_kernel(const ReduceArgs a) {
    chain_begin();
    __shared__ float ws[kRedThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float sq = 0.f;
    if (blockIdx.x + kRedExtraBlocks < gridDim.x) {
        const int base = (blockIdx.x * kRedThreads + threadIdx.x) * kRedPerThread;   // P is a multiple of 4
        if (base < a.P) {
            float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int sp = 0; sp < a.splits; ++sp) {
                const float4 v = *reinterpret_cast<const float4*>(a.partials + (size_t)sp * a.split_stride + base);
                s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
            }
            bool special = (base + 3 >= a.off_ba && base < a.off_logstd + a.A) || (base <= a.off_bc && base + 3 >= a.off_bc);
            for (int b = 0; b < a.n_bias; ++b)
                special = special || (base + 3 >= a.bias[b].p_off && base < a.bias[b].p_off + a.bias[b].n);
            if (special) {
                // a group that touches entries finished by the extra blocks: those are written (and squared) there
                const float g[4] = {s.x, s.y, s.z, s.w};
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (!head_entry(a, base + q) && !bias_entry(a, base + q)) { a.grad[base + q] = g[q]; sq += g[q] * g[q]; }
            } else {
                *reinterpret_cast<float4*>(a.grad + base) = s;
                sq = (s.x * s.x + s.y * s.y) + (s.z * s.z + s.w * s.w);
            }
        }
    } else {
        // one warp per entry: lane l adds partial rows l, l+32, ... in order, then a fixed shuffle tree
        const int xwarp = (blockIdx.x - (gridDim.x - kRedExtraBlocks)) * (kRedThreads / 32) + warp;
        const int xwarps = kRedExtraBlocks * (kRedThreads / 32);
        // bias sources: a warp takes 4 consecutive columns (one float4) and spreads the partial rows over
        // its 32 lanes; every lane walks its rows in order, then a fixed butterfly
        int total_units = 0;
        for (int b = 0; b < a.n_bias; ++b) total_units += (a.bias[b].n + 3) / 4;
        for (int u = xwarp; u < total_units; u += xwarps) {
            int b = 0, ul = u;
            while (ul >= (a.bias[b].n + 3) / 4) { ul -= (a.bias[b].n + 3) / 4; ++b; }
            const BiasSource& src = a.bias[b];
            const int c = 4 * ul;                                       // < ld: the rows are padded to 64 columns
            const float* __restrict__ base = src.slots + c;
            const size_t ld = (size_t)src.ld;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            int r = lane;
            for (; r + 32 * 7 < src.nslots; r += 32 * 8) {
                float4 v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = __ldg(reinterpret_cast<const float4*>(base + (size_t)(r + 32 * i) * ld));
#pragma unroll
                for (int i = 0; i < 8; ++i) { acc.x += v[i].x; acc.y += v[i].y; acc.z += v[i].z; acc.w += v[i].w; }
            }
            for (; r < src.nslots; r += 32) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(base + (size_t)r * ld));
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o);
                acc.z += __shfl_xor_sync(0xffffffffu, acc.z, o); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, o);
            }
            if (lane == 0) {
                const float g[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (c + q < src.n) { a.grad[src.p_off + c + q] = g[q]; sq += g[q] * g[q]; }
            }
        }
        const int entries = 2 * a.A + 1 + LS_COUNT;
        for (int e = xwarp; e < entries; e += xwarps) {
            int slot, p = -1; float shift = 0.f;
            if (e < a.A) { slot = 8 + e; p = a.off_ba + e; }
            else if (e < 2 * a.A) { slot = 8 + kMaxActions + e - a.A; p = a.off_logstd + e - a.A; shift = -a.entropy_coef; }
            else if (e == 2 * a.A) { slot = 4; p = a.off_bc; }
            else slot = e - 2 * a.A - 1;                                   // loss sums
            float s = 0.f;
            for (int b = lane; b < a.nblocks; b += 32) s += a.block_partials[(size_t)b * kPartialStride + slot];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
            if (lane == 0) {
                if (p >= 0) { s += shift; a.grad[p] = s; sq += s * s; }
                else a.loss_sums[slot] = s;
            }
        }
        if (threadIdx.x == 0 && blockIdx.x + 1 == gridDim.x) {   // entropy of the policy this step's forward used
            float ent = 0.f;
            for (int i = 0; i < a.A; ++i) ent += 0.5f + kHalfLog2Pi + a.log_std[i];
            a.loss_sums[LS_COUNT] = ent;
        }
    }
    sq = warp_sum(sq);
    if (lane == 0) ws[warp] = sq;
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
    chain_begin();
    // The first group of every thread is loaded before the block derives its scalars: those loads need none of them,
    // and the sums below are a chain of dependent loads of their own.
    // BF16 mode, hidden-layer weights: a thread takes four consecutive ROWS of one column instead of four
    // consecutive columns of one row, so that its entries of the transposed operand copy Wt[out][in] are
    // one 8-byte store (neighbouring threads: neighbouring columns, every FP32 access still coalesced).
    // Those groups cover the rows below the last multiple of four, the same elements as before in another
    // assignment; the remaining rows, biases and everything else take the plain path.
    struct Group { float g[4], p[4], m[4], v[4]; size_t base; int e, r4, o; bool rows; };
    auto fetch = [&](int i, Group& G) {
        const int idx0 = 4 * i;
        int e = 0;
        while (e < a.n_cvt && !(idx0 >= a.cvt[e].w_off && idx0 < a.cvt[e].w_off + a.cvt[e].in * a.cvt[e].out_p)) ++e;
        G.rows = false;
        if (e < a.n_cvt) {
            const CvtRange& c = a.cvt[e];
            const int lg = (idx0 - c.w_off) >> 2;
            if (lg < (c.in >> 2) * c.out_p) {
                G.rows = true; G.e = e;
                G.r4 = lg / c.out_p; G.o = lg - G.r4 * c.out_p;
                G.base = (size_t)c.w_off + (size_t)(4 * G.r4) * c.out_p + G.o;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const size_t at = G.base + (size_t)q * c.out_p;
                    G.g[q] = a.grad[at]; G.p[q] = a.param[at]; G.m[q] = a.m[at]; G.v[q] = a.v[at];
                }
                return;
            }
        }
        const float4 g4 = reinterpret_cast<const float4*>(a.grad)[i];
        const float4 p4 = reinterpret_cast<const float4*>(a.param)[i];
        const float4 m4 = reinterpret_cast<const float4*>(a.m)[i];
        const float4 v4 = reinterpret_cast<const float4*>(a.v)[i];
        G.g[0] = g4.x; G.g[1] = g4.y; G.g[2] = g4.z; G.g[3] = g4.w;
        G.p[0] = p4.x; G.p[1] = p4.y; G.p[2] = p4.z; G.p[3] = p4.w;
        G.m[0] = m4.x; G.m[1] = m4.y; G.m[2] = m4.z; G.m[3] = m4.w;
        G.v[0] = v4.x; G.v[1] = v4.y; G.v[2] = v4.z; G.v[3] = v4.w;
    };
    const int n4 = a.P / 4;
    int i = blockIdx.x * kAdamThreads + threadIdx.x;
    Group G;
    if (i < n4) fetch(i, G);
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
    } else if (threadIdx.x == 32 || threadIdx.x == 64) {
        // 1 - b^step in double: exact enough for any step count; one thread of two other warps each, so that
        // the two powers run beside the norm instead of after it
        const int step = a.step_io[a.parity] + 1;
        const double b = threadIdx.x == 32 ? (double)a.b1 : (double)a.b2;
        s_scal[threadIdx.x == 32 ? 2 : 3] = (float)(1.0 / (1.0 - pow(b, (double)step)));
    }
    __syncthreads();
    if (s_skip) return;          // non-finite step: parameters and moments stay untouched
    const float coef = s_scal[0], lr = s_scal[1], c1 = s_scal[2], c2 = s_scal[3];
    while (i < n4) {
        float* g = G.g; float* p = G.p; float* m = G.m; float* v = G.v;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float gc = g[q] * coef;
            m[q] = a.b1 * m[q] + (1.0f - a.b1) * gc;
            v[q] = a.b2 * v[q] + (1.0f - a.b2) * gc * gc;
            p[q] = p[q] - lr * (m[q] * c1) / (sqrtf(v[q] * c2) + a.eps);
        }
        if (G.rows) {
            const CvtRange& c = a.cvt[G.e];
            const int r4 = G.r4, o = G.o;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const size_t at = G.base + (size_t)q * c.out_p;
                a.param[at] = p[q]; a.m[at] = m[q]; a.v[at] = v[q];
            }
            if (o < c.out) {
                __nv_bfloat16 w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    w[q] = __float2bfloat16_rn(p[q]);
                    if (c.wn) c.wn[(size_t)(4 * r4 + q) * c.ld_wn + o] = w[q];
                }
                __nv_bfloat162 lo2 = __halves2bfloat162(w[0], w[1]), hi2 = __halves2bfloat162(w[2], w[3]);
                *reinterpret_cast<uint2*>(c.wt + (size_t)o * c.ld_wt + 4 * r4) =
                    make_uint2(*reinterpret_cast<uint32_t*>(&lo2), *reinterpret_cast<uint32_t*>(&hi2));
                if (c.wt_lo) {
                    __nv_bfloat162 l0 = __floats2bfloat162_rn(p[0] - __bfloat162float(w[0]), p[1] - __bfloat162float(w[1]));
                    __nv_bfloat162 l1 = __floats2bfloat162_rn(p[2] - __bfloat162float(w[2]), p[3] - __bfloat162float(w[3]));
                    *reinterpret_cast<uint2*>(c.wt_lo + (size_t)o * c.ld_wt + 4 * r4) =
                        make_uint2(*reinterpret_cast<uint32_t*>(&l0), *reinterpret_cast<uint32_t*>(&l1));
                }
            }
        } else {
            reinterpret_cast<float4*>(a.param)[i] = make_float4(p[0], p[1], p[2], p[3]);
            reinterpret_cast<float4*>(a.m)[i] = make_float4(m[0], m[1], m[2], m[3]);
            reinterpret_cast<float4*>(a.v)[i] = make_float4(v[0], v[1], v[2], v[3]);
            // BF16 mode: refresh the operand copies of the hidden-layer weights and biases in place.
            // A group of four parameters lies in one row of one layer (rows are padded to 4).
            const int idx = 4 * i;
            for (int e = 0; e < a.n_cvt; ++e) {
                const CvtRange& c = a.cvt[e];
                if (idx >= c.w_off && idx < c.w_off + c.in * c.out_p) {
                    const int rel = idx - c.w_off, row = rel / c.out_p, o = rel - row * c.out_p;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (o + q < c.out) {
                            const __nv_bfloat16 w = __float2bfloat16_rn(p[q]);
                            c.wt[(size_t)(o + q) * c.ld_wt + row] = w;
                            if (c.wn) c.wn[(size_t)row * c.ld_wn + o + q] = w;
                            if (c.wt_lo) c.wt_lo[(size_t)(o + q) * c.ld_wt + row] = __float2bfloat16_rn(p[q] - __bfloat162float(w));
                        }
                    }
                    break;
                }
                if (idx >= c.b_off && idx < c.b_off + c.out_p) {
                    const int o = idx - c.b_off;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (o + q < c.out) c.bias_pad[o + q] = p[q];
                    break;
                }
            }
        }
        i += gridDim.x * kAdamThreads;
        if (i < n4) fetch(i, G);
    }
}

}  // namespace

cudaError_t launch_gather(const GatherArgs& a, cudaStream_t s, bool alone) {
    if (a.Bmb <= 0) return cudaSuccess;
    // (accounting only) the first gather of an update runs while the caller's stream waits for it, the others beside
    // the kernels of the minibatch step before
    LaunchScope scope_(alone ? "gather_alone" : "gather", s);
    // (with mirrored copies the small shape is also the faster one alone: 73.7 against 78.9 us at 131,072 rows, its
    // 24 warps per SM cover the mirror's reads through L1 better than 16 warps with more rows each)
    if (alone && !a.sym) {
        const int blocks = std::min((a.Bmb + 8 * kGatherRowsAlone - 1) / (8 * kGatherRowsAlone), 148 * 2);   // one resident wave
        return launch_chained(gather_kernel<kGatherRowsAlone, 256, 2>, blocks, 256, 0, s, a);
    }
    const int blocks = std::min((a.Bmb + 4 * kGatherRowsBeside - 1) / (4 * kGatherRowsBeside), 148 * 4);
    return launch_chained(gather_kernel<kGatherRowsBeside, 128, 6>, blocks, 128, 0, s, a);
}

cudaError_t launch_perm_rows(uint64_t seed, uint32_t iteration, uint32_t epoch, uint32_t batch,
                             uint32_t first, int count, int* rows_out, cudaStream_t s) {
    if (count <= 0) return cudaSuccess;
    PermKey pk{(uint32_t)seed, (uint32_t)(seed >> 32), iteration, epoch, batch, feistel_half_bits(batch)};
    LaunchScope scope_("perm_rows", s);
    return launch_chained(perm_rows_kernel, (count + 255) / 256, 256, 0, s, pk, first, count, 1, rows_out);
}

cudaError_t launch_perm_epochs(uint64_t seed, uint32_t iteration, int epochs, uint32_t batch, int* rows_out, cudaStream_t s) {
    if (batch == 0 || epochs <= 0) return cudaSuccess;
    PermKey pk{(uint32_t)seed, (uint32_t)(seed >> 32), iteration, 0u, batch, feistel_half_bits(batch)};
    LaunchScope scope_("perm_rows", s);
    return launch_chained(perm_rows_kernel, dim3((batch + 255) / 256, std::min(epochs, 65535)), 256, 0, s, pk, 0u, (int)batch, epochs, rows_out);
}

int head_loss_blocks(int Bmb) { return std::max(1, (Bmb + kHLRows - 1) / kHLRows); }
int head_partial_stride() { return kPartialStride; }

namespace {
template <typename T, int NP>
cudaError_t launch_head_loss_t(HeadLossArgs& a, cudaStream_t s) {
    const int AP = 16 * NP;
    const size_t smem = sizeof(float) * ((size_t)a.hp.n_a * AP + ((a.hp.n_c + 3) & ~3) + (size_t)kHLRows * (AP + 1) +
                                         kHLThreads / 32);
    cudaError_t e = cudaFuncSetAttribute(head_loss_kernel<T, NP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    a.nblocks_used = head_loss_blocks(a.Bmb);
    LaunchScope scope_("head_loss", s);
    head_loss_kernel<T, NP><<<head_loss_blocks(a.Bmb), kHLThreads, smem, s>>>(a);
    return cudaGetLastError();
}
template <typename T>
cudaError_t launch_head_loss_np(HeadLossArgs& a, cudaStream_t s) {
    const int np = (a.hp.A + 15) / 16;
    if (np == 1) return launch_head_loss_t<T, 1>(a, s);
    if (np == 2) return launch_head_loss_t<T, 2>(a, s);
    if (np == 3) return launch_head_loss_t<T, 3>(a, s);
    return launch_head_loss_t<T, 4>(a, s);
}
}  // namespace

cudaError_t launch_head_loss(HeadLossArgs& a, cudaStream_t s) {
    a.colsum_written = 0;
    if (head_loss_mma_applicable(a)) return launch_head_loss_mma(a, s);
    // row strides of the hidden activations must allow 16-byte pieces
    if ((a.ldha % 8) || (a.ldhc % 8) || (a.lddza % 8) || (a.lddzc % 8)) return cudaErrorInvalidValue;
    return a.bf16_act ? launch_head_loss_np<__nv_bfloat16>(a, s) : launch_head_loss_np<float>(a, s);
}

int reduce_blocks(int P) { return (P + kRedThreads * kRedPerThread - 1) / (kRedThreads * kRedPerThread) + kRedExtraBlocks; }

cudaError_t launch_reduce(const ReduceArgs& a, cudaStream_t s) {
    LaunchScope scope_("grad_reduce", s);
    return launch_chained(reduce_kernel, reduce_blocks(a.P), kRedThreads, 0, s, a);
}

cudaError_t launch_adam(const AdamArgs& a, cudaStream_t s) {
    const int blocks = std::max(1, std::min((a.P / 4 + kAdamThreads - 1) / kAdamThreads, 148 * 4));
    LaunchScope scope_("adam", s);
    return launch_chained(adam_kernel, blocks, kAdamThreads, 0, s, a);
}

}  // namespace rslrl
