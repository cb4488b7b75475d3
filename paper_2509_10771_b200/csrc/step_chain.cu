// Row-local part of a minibatch step in one persistent kernel (see step_chain.h).
//
// A work item is (128-row tile, net).  The CTA runs the item's program, compiled by the host from
// the layer widths: MMA jobs, each a run of k-blocks into one accumulator of up to 256 tensor-
// memory columns, and epilogues, each turning one accumulator into the next operand:
//   forward epilogue      z + b -> ELU -> BF16 activations, kept in shared memory as the A operand
//                         of the next layer and stored to global memory for the weight gradients
//   head epilogue         head outputs -> PPO loss terms of the row and dL/d(head output), which
//                         becomes the A operand of the first data-gradient job
//   data-gradient epil.   (dZ_next W^T) * ELU'(h) -> BF16 dZ, again the next A operand; h comes
//                         from shared memory (last hidden layer) or is read back, by the warp that
//                         stored it, from the copy the forward epilogue wrote to global memory
// Only weights (and the observations of the first layer) stream through the operand ring.
//
// Warp roles (576 threads): warp 0 = TMA producer, warp 1 = MMA issuer and owner of the tensor
// memory, warps 2..17 = epilogue (warp = 4 * column group + accumulator-lane quarter).
// Every wait is bounded in time; on expiry the CTA raises an error flag and winds down.
#include "step_chain.h"
#include "tc_ptx.cuh"

#include <algorithm>
#include <cstring>
#include <vector>

namespace rslrl {

using namespace tc;

namespace {

constexpr int kSlots = 8;
constexpr uint32_t kSlotBytes = 16384;
constexpr uint32_t kActBytes = BLOCK_M * kMaxBN * 2;     // 64 KiB = four [128 rows][64] blocks
constexpr uint32_t kHeadBytes = BLOCK_M * 64 * 2;        // 16 KiB: dL/d(head output), [128 rows][64]
constexpr int kLayers = kStepChainLayers;
constexpr int kJobs = 12, kEpis = 12, kWmaps = 10;
constexpr int kBiasFloats = 2 * (512 + (kLayers - 1) * 256);
constexpr int kHeadFloats = 256;                         // head bias[64], log_std[64], 1/sigma^2[64], critic head bias
constexpr int kPartialStride = 8 + 2 * kMaxActions;      // layout of a block_partials row (see update_kernels.cu)
constexpr size_t kSmem = 1024 + (size_t)kSlots * kSlotBytes + kActBytes + kHeadBytes + kBiasFloats * 4 +
                         kHeadFloats * 4 + 4 * kPartialStride * 4 + 512;
constexpr int kPrevItem = 16;            // added to an epilogue index: that epilogue of the CTA's previous item
constexpr float kHalfLog2Pi = 0.91893853320467274178f;

enum { EK_FWD = 0, EK_HEAD = 1, EK_DGRAD_ACT = 2, EK_DGRAD_GLB = 3 };
enum { SRC_ACT = 0, SRC_RING = 1, SRC_HEAD = 2 };

struct Job {
    int wmap;            // tensor map of the B operand
    int n0, bn;          // rows [n0, n0 + bn) of the B operand = output columns
    int kb0, nkb;        // k-blocks [kb0, kb0 + nkb) of the B operand's contraction
    int a_src;           // SRC_ACT: block i of the activation buffer for the job's i-th k-block;
                         // SRC_RING: observations through the ring; SRC_HEAD: the head-gradient tile
    int tmem_col;        // accumulator columns [tmem_col, tmem_col + bn)
    int accumulate;      // 1: adds to what the accumulator holds
    int wait_epi;        // epilogue that must be done before the first MMA (-1: none; + kPrevItem: of the previous item)
};
struct Epi {
    int kind, layer;
    int n0, ncols, tmem_col;   // columns [n0, n0 + ncols) of `layer` from these accumulator columns
    int wait_job;        // the job that completes the accumulator
    int write_job;       // a later job that still reads the activation buffer this epilogue rewrites (-1: none)
};

struct Net {
    int nlayers, njobs, nepis;
    int is_actor, A;
    Job job[kJobs];
    Epi epi[kEpis];
    const float* bias[kLayers]; int bias_n[kLayers], bias_off[kLayers];
    const float* head_bias;
    float* colsum[kLayers]; int ld[kLayers];
    const __nv_bfloat16* h[kLayers];     // stored post-activations, row stride ld[l]
};

struct Params {
    CUtensorMap tmX[2];                // observations, boxes of 64 x 128 rows
    CUtensorMap tmW[2][kWmaps];        // weight operands, boxes of 64 x (rows per job)
    CUtensorMap tmH[2][kLayers];       // post-activations, boxes of 64 columns x 32 rows (stores)
    CUtensorMap tmDz[2][kLayers];      // dL/dz, same boxes (stores)
    CUtensorMap tmDhead[2];            // head gradient, boxes of 64 x 32 rows (stores)
    Net net[2];
    int nnets, rows, total_items;
    float alpha;
    int* error;
    const float* act_mb; const float* mu_old; const float* sigma_old; int as;
    const float* logp_old; const float* v_old; const float* ret; const float* adv;
    const float* log_std;
    float clip, value_clip, value_coef; int use_clipped_value_loss;
    float* block_partials;
};

__host__ __device__ constexpr int slots_of(int a_ring, int bn) {
    return a_ring + (bn * BLOCK_K * 2 + (int)kSlotBytes - 1) / (int)kSlotBytes;
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h2);
}

// acc (32 columns) * ELU'(h) for one 16-byte piece (8 columns) of stored post-activations
__device__ __forceinline__ uint4 dgrad_piece(const uint4 hv, const uint32_t* acc8, float alpha) {
    const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w};
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 h2 = *reinterpret_cast<const __nv_bfloat162*>(&hw[e]);
        const float h0 = __low2float(h2), h1 = __high2float(h2);
        const float v0 = __uint_as_float(acc8[2 * e]) * (h0 > 0.f ? 1.0f : h0 + alpha);
        const float v1 = __uint_as_float(acc8[2 * e + 1]) * (h1 > 0.f ? 1.0f : h1 + alpha);
        o[e] = pack2(v0, v1);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// Column sums of a [32 rows][64 columns] BF16 tile kept with the 128-byte swizzle: lane l adds
// columns 2l, 2l+1 (the 32 words of a row sit in 32 different banks).
__device__ __forceinline__ float2 tile_colsum(const uint8_t* tile, int lane) {
    float s0 = 0.f, s1 = 0.f;
    const uint8_t* mine = tile + ((lane & 3) << 2);
#pragma unroll
    for (int r = 0; r < 32; ++r) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(mine + r * 128 + ((((lane >> 2) ^ (r & 7))) << 4));
        const __nv_bfloat162 v2 = *reinterpret_cast<const __nv_bfloat162*>(&w);
        s0 += __low2float(v2); s1 += __high2float(v2);
    }
    return make_float2(s0, s1);
}

__global__ void __launch_bounds__(kThreads, 1) step_chain_kernel(const __grid_constant__ Params P) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sRing = smem;
    uint8_t* sAct = sRing + kSlots * kSlotBytes;
    uint8_t* sDhead = sAct + kActBytes;
    float* sBias = reinterpret_cast<float*>(sDhead + kHeadBytes);
    float* sHead = sBias + kBiasFloats;
    float* sLoss = sHead + kHeadFloats;                     // [4][kPartialStride]
    uint64_t* full = reinterpret_cast<uint64_t*>(sLoss + 4 * kPartialStride);
    uint64_t* empty = full + kSlots;
    uint64_t* job_done = empty + kSlots;       // one completion per item each
    uint64_t* epi_done = job_done + kJobs;
    uint64_t* drain = epi_done + kEpis;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kSlots; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int j = 0; j < kJobs; ++j) mbar_init(&job_done[j], 1);
        for (int e = 0; e < kEpis; ++e) mbar_init(&epi_done[e], kEpiWarps);
        mbar_init(drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    if (warp == 0 && lane == 0)
        for (int n = 0; n < P.nnets; ++n) {
            tma_prefetch_desc(&P.tmX[n]); tma_prefetch_desc(&P.tmDhead[n]);
            for (int l = 0; l < P.net[n].nlayers; ++l) {
                tma_prefetch_desc(&P.tmW[n][l]); tma_prefetch_desc(&P.tmH[n][l]); tma_prefetch_desc(&P.tmDz[n][l]);
            }
        }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    chain_wait();
    // constants the epilogues read between two MMA jobs: keep them close
    for (int n = 0; n < P.nnets; ++n) {
        const Net& N = P.net[n];
        for (int l = 0; l < N.nlayers; ++l)
            for (int i = threadIdx.x; i < N.bias_n[l]; i += kThreads) sBias[N.bias_off[l] + i] = N.bias[l][i];
        if (N.is_actor) {
            for (int i = threadIdx.x; i < 64; i += kThreads) {
                const float ls = i < N.A ? P.log_std[i] : 0.f;
                sHead[i] = N.head_bias[i];
                sHead[64 + i] = ls;
                sHead[128 + i] = __expf(-2.0f * ls);
            }
        } else if (threadIdx.x == 0) {
            sHead[192] = N.head_bias[0];
        }
    }
    for (int i = threadIdx.x; i < 4 * kPartialStride; i += kThreads) sLoss[i] = 0.f;
    __syncthreads();

    if (warp == 0) {
        // ================================ TMA producer =================================
        if (lane == 0) {
            int pos = 0;
            uint32_t full_bits = 0, empty_bits = 0;     // parity of the next use of each slot's barriers
            uint32_t issued_mask = 0, issued_parity = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x) {
                const int ni = item % P.nnets, m0 = (item / P.nnets) * BLOCK_M;
                const Net& N = P.net[ni];
                for (int j = 0; ok && j < N.njobs; ++j) {
                    const Job& J = N.job[j];
                    const int a_ring = J.a_src == SRC_RING ? 1 : 0;
                    const int need = slots_of(a_ring, J.bn);
                    const uint32_t bytes = (uint32_t)J.bn * BLOCK_K * 2 + (a_ring ? kSlotBytes : 0u);
                    for (int kb = J.kb0; ok && kb < J.kb0 + J.nkb; ++kb) {
                        if (pos + need > kSlots) pos = 0;
                        for (int s = pos; s < pos + need; ++s)
                            if (!mbar_wait(&empty[s], ((empty_bits >> s) & 1u) ^ 1u, abort_flag, P.error, 11)) { ok = false; break; }
                        if (!ok) break;
                        mbar_expect_tx(&full[pos], bytes);
                        uint8_t* dst = sRing + pos * kSlotBytes;
                        if (a_ring) { tma_load_2d(dst, &P.tmX[ni], kb * BLOCK_K, m0, &full[pos]); dst += kSlotBytes; }
                        tma_load_2d(dst, &P.tmW[ni][J.wmap], kb * BLOCK_K, J.n0, &full[pos]);
                        issued_mask |= 1u << pos;
                        issued_parity = (issued_parity & ~(1u << pos)) | (((full_bits >> pos) & 1u) << pos);
                        full_bits ^= 1u << pos;
                        empty_bits ^= ((1u << need) - 1u) << pos;
                        pos += need;
                    }
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA's shared memory goes away
                for (int s = 0; s < kSlots; ++s) {
                    if (!(issued_mask & (1u << s))) continue;
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(&full[s], (issued_parity >> s) & 1u) && global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer ===================================
        if (lane == 0) {
            int pos = 0;
            uint32_t full_bits = 0;
            bool ok = true;
            uint32_t t = 0;                          // items this CTA has started
            for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++t) {
                const Net& N = P.net[item % P.nnets];
                for (int j = 0; ok && j < N.njobs; ++j) {
                    const Job& J = N.job[j];
                    if (J.wait_epi >= kPrevItem) {
                        if (t > 0 && !mbar_wait(&epi_done[J.wait_epi - kPrevItem], (t - 1) & 1u, abort_flag, P.error, 12)) { ok = false; break; }
                    } else if (J.wait_epi >= 0) {
                        if (!mbar_wait(&epi_done[J.wait_epi], t & 1u, abort_flag, P.error, 12)) { ok = false; break; }
                    }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)J.tmem_col;
                    const uint32_t idesc = instr_desc(J.bn, 0, 0);
                    const int a_ring = J.a_src == SRC_RING ? 1 : 0;
                    const int need = slots_of(a_ring, J.bn);
                    for (int i = 0; i < J.nkb; ++i) {
                        if (pos + need > kSlots) pos = 0;
                        if (!mbar_wait(&full[pos], (full_bits >> pos) & 1u, abort_flag, P.error, 13)) { ok = false; break; }
                        full_bits ^= 1u << pos;
                        tc_fence_after();
                        const uint32_t ring_addr = smem_u32(sRing + pos * kSlotBytes);
                        const uint32_t a_addr = a_ring ? ring_addr
                                              : J.a_src == SRC_HEAD ? smem_u32(sDhead) : smem_u32(sAct + i * kStageA);
                        const uint32_t b_addr = ring_addr + (a_ring ? kSlotBytes : 0u);
#pragma unroll
                        for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                            umma_bf16(d_tmem, smem_desc(a_addr + k * (UMMA_K * 2), 16, 1024),
                                      smem_desc(b_addr + k * (UMMA_K * 2), 16, 1024), idesc,
                                      (J.accumulate || i > 0 || k > 0) ? 1u : 0u);
                        for (int s2 = pos; s2 < pos + need; ++s2) umma_commit(&empty[s2]);   // frees the slots once these MMAs have read them
                        pos += need;
                    }
                    if (ok) umma_commit(&job_done[j]);
                }
            }
            // all products of this CTA are issued: the next kernel of the stream may be scheduled
            chain_release();
            if (!ok) {
                umma_commit(drain);
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(drain, 0) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else {
        // ================================ epilogue =====================================
        const int q = warp & 3;                    // accumulator lanes (= tile rows) 32q .. 32q+31
        const int g = (warp - 2) >> 2;             // columns [64 g, 64 g + 64) of the epilogue's output
        // block g of the activation buffer, rows 32q..: lane r owns row r (128 bytes = eight 16-byte
        // pieces), piece j is kept at j ^ (r & 7), the 128-byte swizzle the MMA and the copies expect
        uint8_t* tile = sAct + g * kStageA + q * (32 * 128);
        uint8_t* tile_row = tile + lane * 128;
        const int sw = lane & 7;
        const uint32_t lane_base = tmem_base + ((uint32_t)(32 * q) << 16);
        float* my_loss = sLoss + q * kPartialStride;
        bool ok = true;
        uint32_t t = 0;
        const float inv_R = 1.0f / (float)P.rows;
        for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++t) {
            const int ni = item % P.nnets, m0 = (item / P.nnets) * BLOCK_M;
            const Net& N = P.net[ni];
            const int row0 = m0 + 32 * q;
            for (int e = 0; ok && e < N.nepis; ++e) {
                const Epi& E = N.epi[e];
                const bool active = 64 * g < E.ncols;          // uniform across the warp
                uint4 hv[8];                                   // data gradient: this lane's 64 stored post-activations
                if (E.kind == EK_DGRAD_GLB && active) {
                    // read back what this warp stored in the forward pass (complete since the head epilogue),
                    // past the L1 cache, while the products still run; rows beyond the extent read row 0
                    const int r = row0 + lane < P.rows ? row0 + lane : 0;
                    const uint4* src = reinterpret_cast<const uint4*>(N.h[E.layer] + (size_t)r * N.ld[E.layer] + E.n0 + 64 * g);
#pragma unroll
                    for (int p8 = 0; p8 < 8; ++p8) hv[p8] = __ldcg(src + p8);
                }
                if (!mbar_wait(&job_done[E.wait_job], t & 1u, abort_flag, P.error, 14)) { ok = false; break; }
                tc_fence_after();
                if (E.kind == EK_FWD) {
                    uint4 outv[8];
                    if (active) {
                        const float* bias = sBias + N.bias_off[E.layer] + E.n0 + 64 * g;
#pragma unroll
                        for (int ci = 0; ci < 2; ++ci) {
                            uint32_t acc[32];
                            tmem_ld32(lane_base + (uint32_t)(E.tmem_col + 64 * g + 32 * ci), acc);
                            const float4* b4 = reinterpret_cast<const float4*>(bias + 32 * ci);
#pragma unroll
                            for (int gg = 0; gg < 4; ++gg) {
                                const float4 ba = b4[2 * gg], bb = b4[2 * gg + 1];
                                const float bv[8] = {ba.x, ba.y, ba.z, ba.w, bb.x, bb.y, bb.z, bb.w};
                                uint32_t o[4];
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    o[k] = pack2(elu_fast(__uint_as_float(acc[8 * gg + 2 * k]) + bv[2 * k], P.alpha),
                                                 elu_fast(__uint_as_float(acc[8 * gg + 2 * k + 1]) + bv[2 * k + 1], P.alpha));
                                outv[4 * ci + gg] = make_uint4(o[0], o[1], o[2], o[3]);
                            }
                        }
                    }
                    // the accumulator is in registers; the buffer may still feed a job that runs meanwhile
                    if (E.write_job >= 0 && !mbar_wait(&job_done[E.write_job], t & 1u, abort_flag, P.error, 15)) { ok = false; break; }
                    if (active) {
                        if (lane == 0) tma_store_wait_read();       // this warp's last store has read the rows
                        __syncwarp();
#pragma unroll
                        for (int p8 = 0; p8 < 8; ++p8) *reinterpret_cast<uint4*>(tile_row + ((p8 ^ sw) << 4)) = outv[p8];
                        fence_async_smem();                         // rows -> visible to the MMA and the copy engine
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        // rows at or beyond the tensor's extent are clipped by the store itself
                        if (active && row0 < P.rows) tma_store_2d(&P.tmH[ni][E.layer], tile, E.n0 + 64 * g, row0);
                        mbar_arrive(&epi_done[e]);
                    }
                } else if (E.kind == EK_HEAD) {
                    if (g == 0) {
                        // one thread per row of the tile: loss terms and dL/d(head output)
                        const int j = row0 + lane;
                        const bool live = j < P.rows;
                        const int jc = live ? j : P.rows - 1;
                        const uint32_t taddr = lane_base + (uint32_t)E.tmem_col;
                        uint8_t* hrow = sDhead + (32 * q + lane) * 128;
                        if (N.is_actor) {
                            // actions in chunks of 16: one accumulator read and four 16-byte loads per array
                            const int A = N.A, nch = (A + 15) / 16;
                            const float* arow = P.act_mb + (size_t)jc * P.as;
                            const float* mrow = P.mu_old + (size_t)jc * P.as;
                            const float* srow = P.sigma_old + (size_t)jc * P.as;
                            const float logp_old = P.logp_old[jc], adv = P.adv[jc];
                            float lp = 0.f, kl = 0.f;
                            for (int ch = 0; ch < nch; ++ch) {
                                uint32_t acc[16];
                                tmem_ld16(taddr + (uint32_t)(16 * ch), acc);
                                float aa[16], mm[16], ss[16];
#pragma unroll
                                for (int v = 0; v < 4; ++v) {
                                    const int c = 16 * ch + 4 * v;
                                    float4 av = make_float4(0.f, 0.f, 0.f, 0.f), mv = av, sv = make_float4(1.f, 1.f, 1.f, 1.f);
                                    if (c < P.as) {
                                        av = *reinterpret_cast<const float4*>(arow + c);
                                        mv = *reinterpret_cast<const float4*>(mrow + c);
                                        sv = *reinterpret_cast<const float4*>(srow + c);
                                    }
                                    aa[4 * v] = av.x; aa[4 * v + 1] = av.y; aa[4 * v + 2] = av.z; aa[4 * v + 3] = av.w;
                                    mm[4 * v] = mv.x; mm[4 * v + 1] = mv.y; mm[4 * v + 2] = mv.z; mm[4 * v + 3] = mv.w;
                                    ss[4 * v] = sv.x; ss[4 * v + 1] = sv.y; ss[4 * v + 2] = sv.z; ss[4 * v + 3] = sv.w;
                                }
#pragma unroll
                                for (int k = 0; k < 16; ++k) {
                                    const int i = 16 * ch + k;
                                    if (i < A) {
                                        const float mu = __uint_as_float(acc[k]) + sHead[i];
                                        const float ls = sHead[64 + i], ivar = sHead[128 + i];
                                        const float d = aa[k] - mu;
                                        lp += -(d * d) * 0.5f * ivar - ls - kHalfLog2Pi;
                                        const float dm = mm[k] - mu;
                                        kl += (ls - logf(ss[k])) + (ss[k] * ss[k] + dm * dm) * 0.5f * ivar - 0.5f;
                                    }
                                }
                            }
                            const float ratio = expf(lp - logp_old);
                            const float s1 = -adv * ratio;
                            const float s2 = -adv * fminf(fmaxf(ratio, 1.0f - P.clip), 1.0f + P.clip);
                            const bool inside = ratio >= 1.0f - P.clip && ratio <= 1.0f + P.clip;
                            const float dlogp = (live && (inside || s1 > s2)) ? s1 * inv_R : 0.f;
                            const float surr = warp_sum(live ? fmaxf(s1, s2) : 0.f);
                            const float klw = warp_sum(live ? kl : 0.f);
                            if (lane == 0) { my_loss[LS_SURR] += surr; my_loss[LS_KL] += klw; }
                            for (int ch = 0; ch < 4; ++ch) {
                                // v[0..16): dL/dmu of the chunk's actions, v[16..32): their dL/dlog_std terms
                                float v[32];
#pragma unroll
                                for (int k = 0; k < 32; ++k) v[k] = 0.f;
                                if (ch < nch) {
                                    uint32_t acc[16];
                                    tmem_ld16(taddr + (uint32_t)(16 * ch), acc);
                                    float aa[16];
#pragma unroll
                                    for (int w4 = 0; w4 < 4; ++w4) {
                                        const int c = 16 * ch + 4 * w4;
                                        float4 av = make_float4(0.f, 0.f, 0.f, 0.f);
                                        if (c < P.as) av = *reinterpret_cast<const float4*>(arow + c);
                                        aa[4 * w4] = av.x; aa[4 * w4 + 1] = av.y; aa[4 * w4 + 2] = av.z; aa[4 * w4 + 3] = av.w;
                                    }
#pragma unroll
                                    for (int k = 0; k < 16; ++k) {
                                        const int i = 16 * ch + k;
                                        if (i < A) {
                                            const float mu = __uint_as_float(acc[k]) + sHead[i];
                                            const float ivar = sHead[128 + i];
                                            const float d = aa[k] - mu;
                                            v[k] = dlogp * d * ivar;
                                            v[16 + k] = dlogp * (d * d * ivar - 1.0f);
                                        }
                                    }
                                }
                                // the chunk's 32 bytes of the head-gradient row (zeros beyond the actions)
#pragma unroll
                                for (int hh = 0; hh < 2; ++hh)
                                    *reinterpret_cast<uint4*>(hrow + (((2 * ch + hh) ^ sw) << 4)) =
                                        make_uint4(pack2(v[8 * hh], v[8 * hh + 1]), pack2(v[8 * hh + 2], v[8 * hh + 3]),
                                                   pack2(v[8 * hh + 4], v[8 * hh + 5]), pack2(v[8 * hh + 6], v[8 * hh + 7]));
                                if (ch < nch) {
                                    // sums over the warp's 32 rows of all 32 values at once: every exchange halves
                                    // what a lane holds, and lane l ends with the total of v[l]
#pragma unroll
                                    for (int off = 16; off >= 1; off >>= 1) {
                                        const bool up = (lane & off) != 0;
#pragma unroll
                                        for (int k = 0; k < off; ++k) {
                                            const float send = up ? v[k] : v[k + off];
                                            const float keep = up ? v[k + off] : v[k];
                                            v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                                        }
                                    }
                                    const int i = 16 * ch + (lane & 15);
                                    if (i < A) my_loss[8 + (lane < 16 ? 0 : kMaxActions) + i] += v[0];
                                }
                            }
                        } else {
                            uint32_t a4[4];
                            tmem_ld4(taddr, a4);
                            const float v = __uint_as_float(a4[0]) + sHead[192];
                            const float v_old = P.v_old[jc], ret = P.ret[jc];
                            float dv, lossv;
                            const float e1 = (v - ret) * (v - ret);
                            if (P.use_clipped_value_loss) {
                                const float vc = v_old + fminf(fmaxf(v - v_old, -P.value_clip), P.value_clip);
                                const float e2 = (vc - ret) * (vc - ret);
                                lossv = fmaxf(e1, e2);
                                const bool vin = fabsf(v - v_old) <= P.value_clip;
                                dv = (vin || e1 > e2) ? 2.0f * (v - ret) : 0.f;
                            } else {
                                lossv = e1;
                                dv = 2.0f * (v - ret);
                            }
                            dv = live ? dv * P.value_coef * inv_R : 0.f;
                            const float vsum = warp_sum(live ? lossv : 0.f);
                            const float dsum = warp_sum(dv);
                            if (lane == 0) { my_loss[LS_VALUE] += vsum; my_loss[4] += dsum; }
#pragma unroll
                            for (int p8 = 0; p8 < 8; ++p8)
                                *reinterpret_cast<uint4*>(hrow + ((p8 ^ sw) << 4)) = make_uint4(p8 == 0 ? pack2(dv, 0.f) : 0u, 0u, 0u, 0u);
                        }
                        fence_async_smem();                         // rows -> visible to the MMA and the copy engine
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (g == 0 && row0 < P.rows) tma_store_2d(&P.tmDhead[ni], sDhead + q * (32 * 128), 0, row0);
                        // every store of the forward pass is complete from here on: the producer may fetch
                        // the stored activations back, and the tiles they left from may be rewritten
                        tma_store_wait_all();
                        mbar_arrive(&epi_done[e]);
                    }
                } else if (E.kind == EK_DGRAD_ACT) {
                    // the stored post-activations of this layer are still in the activation buffer
                    if (active) {
#pragma unroll
                        for (int ci = 0; ci < 2; ++ci) {
                            uint32_t acc[32];
                            tmem_ld32(lane_base + (uint32_t)(E.tmem_col + 64 * g + 32 * ci), acc);
#pragma unroll
                            for (int gg = 0; gg < 4; ++gg) {
                                uint4* piece = reinterpret_cast<uint4*>(tile_row + (((4 * ci + gg) ^ sw) << 4));
                                *piece = dgrad_piece(*piece, &acc[8 * gg], P.alpha);
                            }
                        }
                        fence_async_smem();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (active) {
                        if (lane == 0 && row0 < P.rows) tma_store_2d(&P.tmDz[ni][E.layer], tile, E.n0 + 64 * g, row0);
                        const float2 cs = tile_colsum(tile, lane);
                        *reinterpret_cast<float2*>(N.colsum[E.layer] + (size_t)(m0 / BLOCK_M * 4 + q) * N.ld[E.layer] + E.n0 + 64 * g + 2 * lane) = cs;
                    }
                    if (lane == 0) mbar_arrive(&epi_done[e]);
                } else {
                    // EK_DGRAD_GLB: the stored post-activations are in hv; the result replaces them there
                    if (active) {
#pragma unroll
                        for (int ci = 0; ci < 2; ++ci) {
                            uint32_t acc[32];
                            tmem_ld32(lane_base + (uint32_t)(E.tmem_col + 64 * g + 32 * ci), acc);
#pragma unroll
                            for (int gg = 0; gg < 4; ++gg) hv[4 * ci + gg] = dgrad_piece(hv[4 * ci + gg], &acc[8 * gg], P.alpha);
                        }
                    }
                    // the accumulator is in registers; the buffer may still feed a job that runs meanwhile
                    if (E.write_job >= 0 && !mbar_wait(&job_done[E.write_job], t & 1u, abort_flag, P.error, 15)) { ok = false; break; }
                    if (active) {
                        if (lane == 0) tma_store_wait_read();       // this warp's last store has read the rows
                        __syncwarp();
#pragma unroll
                        for (int p8 = 0; p8 < 8; ++p8) *reinterpret_cast<uint4*>(tile_row + ((p8 ^ sw) << 4)) = hv[p8];
                        fence_async_smem();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (active) {
                        if (lane == 0 && row0 < P.rows) tma_store_2d(&P.tmDz[ni][E.layer], tile, E.n0 + 64 * g, row0);
                        const float2 cs = tile_colsum(tile, lane);
                        *reinterpret_cast<float2*>(N.colsum[E.layer] + (size_t)(m0 / BLOCK_M * 4 + q) * N.ld[E.layer] + E.n0 + 64 * g + 2 * lane) = cs;
                    }
                    if (lane == 0) mbar_arrive(&epi_done[e]);
                }
            }
        }
        if (lane == 0) tma_store_wait_all();        // stores done before the CTA retires
    }
    tc_fence_before();
    __syncthreads();
    // loss sums and head-bias / log_std gradients of this CTA's rows, in a fixed order
    for (int k = threadIdx.x; k < kPartialStride; k += kThreads)
        P.block_partials[(size_t)blockIdx.x * kPartialStride + k] =
            (sLoss[k] + sLoss[kPartialStride + k]) + (sLoss[2 * kPartialStride + k] + sLoss[3 * kPartialStride + k]);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

// ------------------------------------------------------------------------------- host side
struct StepChain {
    Params P;
    int grid;
};

namespace {

// Builds the program of one net.  Accumulators alternate between the two halves of tensor memory;
// a job waits for the epilogue that produced its A operand and for the one that drained its half.
struct Builder {
    Net& N;
    int nj = 0, ne = 0;
    int drain_epi[2] = {-1, -1};       // epilogue that last drained each half in this item
    std::vector<int> first_use[2];     // jobs that overwrite a half before any epilogue of the item drained it
    bool overflow = false;
    explicit Builder(Net& n) : N(n) {}
    int job(int wmap, int n0, int bn, int kb0, int nkb, int a_src, int half, int accumulate, int ready_epi) {
        if (nj == kJobs) { overflow = true; return 0; }
        int wait = ready_epi;
        if (!accumulate) {
            if (drain_epi[half] >= 0) wait = std::max(wait, drain_epi[half]);
            else first_use[half].push_back(nj);
        }
        N.job[nj] = Job{wmap, n0, bn, kb0, nkb, a_src, half * 256, accumulate, wait};
        return nj++;
    }
    int epi(int kind, int layer, int n0, int ncols, int half, int wait_job, int write_job) {
        if (ne == kEpis) { overflow = true; return 0; }
        N.epi[ne] = Epi{kind, layer, n0, ncols, half * 256, wait_job, write_job};
        drain_epi[half] = ne;
        return ne++;
    }
    void finish() {
        // a half's first job of an item waits for the epilogue that drained it last in the item before
        for (int h = 0; h < 2; ++h)
            for (int j : first_use[h])
                if (drain_epi[h] >= 0 && N.job[j].wait_epi < 0) N.job[j].wait_epi = kPrevItem + drain_epi[h];
        N.njobs = nj; N.nepis = ne;
    }
};

// Widths the kernel takes: first hidden layer <= 512 (a multiple of 128 beyond 256), the others <= 256.
bool compile(Net& N, const StepChainNet& s, int* bn_w /* box rows of every weight map */) {
    const int nh = s.nh;
    if (nh < 1 || nh > kLayers || s.pw[0] > 512 || (s.pw[0] > 256 && (s.pw[0] % 128 != 0 || nh < 2))) return false;
    for (int l = 1; l < nh; ++l)
        if (s.pw[l] > 256) return false;
    if (s.A < 1 || s.A > 64) return false;
    Builder B(N);
    const int kb_in = s.kp / BLOCK_K;
    const int WHT = nh, WHN = nh + 1;
    auto WN = [&](int l) { return nh + 1 + l; };       // data-gradient operand of layer l >= 1
    int half = 0, prev_e;
    // ---- forward ---------------------------------------------------------------------------
    if (s.pw[0] > 256) {
        const int hw = s.pw[0] / 2, hk = hw / BLOCK_K;
        bn_w[0] = hw;
        const int j0 = B.job(0, 0, hw, 0, kb_in, SRC_RING, 0, 0, -1);
        const int j1 = B.job(0, hw, hw, 0, kb_in, SRC_RING, 1, 0, -1);
        const int e0 = B.epi(EK_FWD, 0, 0, hw, 0, j0, -1);
        const int j2 = B.job(1, 0, s.pw[1], 0, hk, SRC_ACT, 0, 0, e0);
        const int e1 = B.epi(EK_FWD, 0, hw, hw, 1, j1, j2);
        const int j3 = B.job(1, 0, s.pw[1], hk, hk, SRC_ACT, 0, 1, e1);
        prev_e = B.epi(EK_FWD, 1, 0, s.pw[1], 0, j3, -1);
        bn_w[1] = s.pw[1];
        half = 1;
        for (int l = 2; l < nh; ++l, half ^= 1) {
            bn_w[l] = s.pw[l];
            const int j = B.job(l, 0, s.pw[l], 0, s.pw[l - 1] / BLOCK_K, SRC_ACT, half, 0, prev_e);
            prev_e = B.epi(EK_FWD, l, 0, s.pw[l], half, j, -1);
        }
    } else {
        prev_e = -1;
        for (int l = 0; l < nh; ++l, half ^= 1) {
            bn_w[l] = s.pw[l];
            const int j = l == 0 ? B.job(0, 0, s.pw[0], 0, kb_in, SRC_RING, half, 0, -1)
                                 : B.job(l, 0, s.pw[l], 0, s.pw[l - 1] / BLOCK_K, SRC_ACT, half, 0, prev_e);
            prev_e = B.epi(EK_FWD, l, 0, s.pw[l], half, j, -1);
        }
    }
    // ---- head and loss -----------------------------------------------------------------------
    const int last = nh - 1;
    const int nhead = (s.A + 15) / 16 * 16;
    bn_w[WHT] = nhead;
    {
        const int j = B.job(WHT, 0, nhead, 0, s.pw[last] / BLOCK_K, SRC_ACT, half, 0, prev_e);
        prev_e = B.epi(EK_HEAD, last, 0, nhead, half, j, -1);
        half ^= 1;
    }
    // ---- data gradients ------------------------------------------------------------------------
    bn_w[WHN] = s.pw[last];
    {
        const int j = B.job(WHN, 0, s.pw[last], 0, 1, SRC_HEAD, half, 0, prev_e);
        prev_e = B.epi(EK_DGRAD_ACT, last, 0, s.pw[last], half, j, -1);
        half ^= 1;
    }
    for (int l = last - 1; l >= 0; --l) {
        const int nkb = s.pw[l + 1] / BLOCK_K;
        if (s.pw[l] <= 256) {
            bn_w[WN(l + 1)] = s.pw[l];
            const int j = B.job(WN(l + 1), 0, s.pw[l], 0, nkb, SRC_ACT, half, 0, prev_e);
            prev_e = B.epi(EK_DGRAD_GLB, l, 0, s.pw[l], half, j, -1);
            half ^= 1;
        } else {
            const int hw = s.pw[l] / 2;
            bn_w[WN(l + 1)] = hw;
            // both halves read the activation buffer: the first epilogue holds its result until the second job is done
            const int ja = B.job(WN(l + 1), 0, hw, 0, nkb, SRC_ACT, half, 0, prev_e);
            const int jb = B.job(WN(l + 1), hw, hw, 0, nkb, SRC_ACT, half ^ 1, 0, prev_e);
            B.epi(EK_DGRAD_GLB, l, 0, hw, half, ja, jb);
            prev_e = B.epi(EK_DGRAD_GLB, l, hw, hw, half ^ 1, jb, -1);
        }
    }
    B.finish();
    N.nlayers = nh;
    N.is_actor = s.is_actor; N.A = s.A;
    return !B.overflow;
}

}  // namespace

int step_chain_colsum_rows(int rows) { return 4 * ((rows + BLOCK_M - 1) / BLOCK_M); }
int step_chain_blocks(const StepChain* c) { return c->grid; }

StepChain* step_chain_create(const StepChainSetup& s, std::string* err) {
    auto fail = [&](const char* m) { if (err) *err = m; return (StepChain*)nullptr; };
    if (err) err->clear();
    if (cudaFuncSetAttribute(step_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem) != cudaSuccess)
        return fail("could not reserve shared memory for the fused step kernel");
    StepChain* c = new StepChain();
    Params& P = c->P;
    memset(&P, 0, sizeof P);
    int bias_floats = 0;
    for (int n = 0; n < 2; ++n) {
        const StepChainNet& sn = s.net[n];
        Net& N = P.net[n];
        int bn_w[kWmaps] = {};
        if (!compile(N, sn, bn_w)) { delete c; return nullptr; }     // not applicable
        const int nh = sn.nh, last = nh - 1;
        bool okm = make_tmap(&P.tmX[n], sn.x16, s.rows, sn.kp, sn.kp, BLOCK_K, BLOCK_M);
        for (int l = 0; l < nh && okm; ++l) {
            const int kin = l == 0 ? sn.kp : sn.pw[l - 1];
            okm = make_tmap(&P.tmW[n][l], sn.wt[l], sn.pw[l], kin, kin, BLOCK_K, bn_w[l]) &&
                  make_tmap(&P.tmH[n][l], sn.h[l], s.rows, sn.pw[l], sn.pw[l], 64, 32) &&
                  make_tmap(&P.tmDz[n][l], sn.dz[l], s.rows, sn.pw[l], sn.pw[l], 64, 32);
            if (l >= 1 && okm)
                okm = make_tmap(&P.tmW[n][nh + 1 + l], sn.wn[l], sn.pw[l - 1], sn.pw[l], sn.pw[l], BLOCK_K, bn_w[nh + 1 + l]);
            N.bias[l] = sn.bias_pad[l]; N.bias_n[l] = sn.pw[l]; N.bias_off[l] = bias_floats;
            bias_floats += sn.pw[l];
            N.colsum[l] = sn.colsum[l]; N.ld[l] = sn.pw[l]; N.h[l] = sn.h[l];
        }
        okm = okm && make_tmap(&P.tmW[n][nh], sn.wht, 64, sn.pw[last], sn.pw[last], BLOCK_K, bn_w[nh]) &&
              make_tmap(&P.tmW[n][nh + 1], sn.whn, sn.pw[last], 64, 64, BLOCK_K, bn_w[nh + 1]) &&
              make_tmap(&P.tmDhead[n], sn.dhead16, s.rows, 64, 64, 64, 32);
        if (!okm) { delete c; return fail("tensor map encoding failed"); }
        N.head_bias = sn.head_bias;
    }
    if (bias_floats > kBiasFloats) { delete c; return nullptr; }
    P.nnets = 2; P.rows = s.rows;
    P.total_items = 2 * ((s.rows + BLOCK_M - 1) / BLOCK_M);
    P.alpha = s.alpha; P.error = s.error; P.log_std = s.log_std;
    c->grid = std::min(P.total_items, s.num_sms);
    return c;
}

void step_chain_destroy(StepChain* c) { delete c; }

cudaError_t step_chain_launch(StepChain* c, const StepChainLoss& L, cudaStream_t stream) {
    Params& P = c->P;
    P.act_mb = L.act_mb; P.mu_old = L.mu_old; P.sigma_old = L.sigma_old; P.as = L.as;
    P.logp_old = L.logp_old; P.v_old = L.v_old; P.ret = L.ret; P.adv = L.adv;
    P.clip = L.clip; P.value_clip = L.value_clip; P.value_coef = L.value_coef;
    P.use_clipped_value_loss = L.use_clipped_value_loss;
    P.block_partials = L.block_partials;
    LaunchScope scope_("step_chain", stream);
    return launch_chained(step_chain_kernel, c->grid, kThreads, kSmem, stream, P);
}

}  // namespace rslrl
