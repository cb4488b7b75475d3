// Tensor-core engine: the hidden-layer products of act, forward and backward as grouped,
// persistent tcgen05 GEMM kernels.  Operands are BF16 tiles staged in shared memory by TMA
// (128-byte swizzle), accumulators are FP32 in tensor memory (two buffers, so the epilogue of
// one tile overlaps the main loop of the next), and the epilogues fuse bias+ELU (forward),
// the ELU derivative (data gradient) or the split-partial store (weight gradient).  Forward and
// data gradient keep the weight operand of a CTA resident in shared memory and stream the rows.
//
// Warp roles in a CTA of 576 threads: warp 0 = TMA producer, warp 1 = MMA issuer and owner of
// the tensor-memory allocation, warps 2..17 = epilogue (each reads its quarter of the 128
// accumulator lanes and every fourth 32-column chunk of the tile).
//
// Every wait on an mbarrier is bounded in time; on expiry the CTA raises an error flag that
// the host reads, drains its own asynchronous work, frees its tensor memory and returns.
#include "guard.h"
#include "umma.h"
#include "tc_ptx.cuh"

#include <cuda.h>
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <vector>

namespace rslrl {

using namespace tc;

namespace {

// Weight gradient (long contraction, FP32 results stored from registers): 4 pipeline stages of A + B.
constexpr int kWgradStages = 4;
constexpr uint32_t kStageB = kMaxBN * BLOCK_K * 2;       // 32 KiB
constexpr int kMaxProblems = 8;
constexpr size_t kWgradSmem = 1024 + (size_t)kWgradStages * (kStageA + kStageB) + 512;

enum TcMode { TC_FWD = 0, TC_DGRAD = 1, TC_WGRAD = 2 };

struct TcProblem {
    int m_extent, n_extent;        // rows / columns of D that exist (stores are clipped to them)
    int m_tiles, n_tiles, bn;
    int kblocks;                   // k-blocks of 64 along the contraction
    int splits, kb_per_split;      // weight gradient: the contraction is cut into splits
    int item_begin;
    const float* bias; int bias_n;
    __nv_bfloat16* out16; int ld_out;
    const __nv_bfloat16* aux16; int ld_aux;
    float* out32; int ld_out32; long long split_stride;
    float* colsum; int ld_colsum;  // data gradient: column sums of each 32-row slice, [4 m_tiles][ld_colsum] (may be null)
    int net_id, layer_id;          // host side: which net and layer the problem belongs to
};

// Forward and data gradient run "weight-stationary": a CTA is bound to one slab (a problem's column
// block of up to 256 output columns), keeps that slab of the weight operand in shared memory for the
// whole launch where it fits, and walks the row tiles rank, rank + ctas, ... of the slab, so that only
// the activations stream through the pipeline.
constexpr int kMaxSlabs = 64;
constexpr int kMaxCtas = 160;
struct WsSlab {
    int prob, n0;                  // problem and first output column
    int cta_begin, cta_count;      // CTAs [cta_begin, cta_begin + cta_count) work on this slab
    int resident;                  // 1: all k-blocks of the weight slab stay in shared memory
    int stages;                    // pipeline stages (of A alone when resident, of A + B otherwise)
};
struct WsPlan {
    WsSlab slab[kMaxSlabs];
    int nslabs, grid, num_sms, mode;
    int b_early;                   // 1: the weight operand was not written by the kernel launched just before this one, so a
                                   // resident slab may be fetched before the wait for that kernel (during its tail)
    unsigned char cta_slab[kMaxCtas];
};

struct TcParams {
    CUtensorMap tmA[kMaxProblems];
    CUtensorMap tmB[kMaxProblems];
    CUtensorMap tmOut[kMaxProblems];   // BF16 output, boxes of 32 columns x 32 rows, 64-byte swizzle
    CUtensorMap tmAux[kMaxProblems];   // data gradient: stored post-activations, same boxes
    TcProblem p[kMaxProblems];
    int count, total_items;
    float alpha;
    int* error;
    WsPlan ws;                         // forward / data gradient only
};

struct Item { int prob, m0, n0, kb0, kb1, split; };

__device__ __forceinline__ Item decode_item(const TcParams& P, int item) {
    int pi = 0;
#pragma unroll 1
    for (int i = 1; i < P.count; ++i)
        if (item >= P.p[i].item_begin) pi = i;
    const TcProblem& p = P.p[pi];
    const int local = item - p.item_begin;
    const int per_split = p.m_tiles * p.n_tiles;
    Item it;
    it.prob = pi;
    it.split = local / per_split;
    const int rem = local - it.split * per_split;
    it.m0 = (rem / p.n_tiles) * BLOCK_M;
    it.n0 = (rem % p.n_tiles) * p.bn;
    it.kb0 = it.split * p.kb_per_split;
    it.kb1 = min(p.kblocks, it.kb0 + p.kb_per_split);
    return it;
}

// Weight gradient: D[features_in x features_out] = A^T B over the minibatch rows, both operands as stored
// ([row][feature], the contraction index outermost: MN-major tiles).  A work item is a 128 x (<= 256) tile of one
// problem over one split of the row range; its FP32 result is a partial that the gradient reduction sums.
__global__ void __launch_bounds__(kThreads, 1) wgrad_gemm_kernel(const __grid_constant__ TcParams P) {
    constexpr int kStages = kWgradStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = smem + kStages * kStageA;
    uint64_t* full = reinterpret_cast<uint64_t*>(sB + kStages * kStageB);
    uint64_t* empty = full + kStages;
    uint64_t* tfull = empty + kStages;
    uint64_t* tempty = tfull + 2;
    uint64_t* drain = tempty + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // the set-up below touches only shared memory, tensor memory and the kernel parameters: it may
    // overlap the tail of the preceding kernel; global memory is first touched after the wait
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&tfull[b], 1); mbar_init(&tempty[b], kEpiWarps); }
        mbar_init(drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    if (warp == 0 && lane == 0)
        for (int i = 0; i < P.count; ++i) { tma_prefetch_desc(&P.tmA[i]); tma_prefetch_desc(&P.tmB[i]); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    chain_wait();

    if (warp == 0) {
        // ================================ TMA producer =================================
        // a k-block is six boxes of 64 features x 64 rows (two of A, up to four of B), one 8 KiB block per 64
        // features: lane l issues box l, so that the whole k-block goes out in one pass of the loop
        int stage = 0; uint32_t phase = 0;
        uint32_t issued_mask = 0, issued_parity = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x) {
            const Item it = decode_item(P, item);
            const TcProblem& p = P.p[it.prob];
            const uint32_t bytes = (uint32_t)(BLOCK_M + p.bn) * BLOCK_K * 2;
            const bool mine = lane < 2 + p.bn / 64;
            const CUtensorMap* tm = lane < 2 ? &P.tmA[it.prob] : &P.tmB[it.prob];
            const int x = lane < 2 ? it.m0 + 64 * lane : it.n0 + 64 * (lane - 2);
            uint8_t* base = lane < 2 ? sA + (uint32_t)lane * 8192u : sB + (uint32_t)(lane - 2) * 8192u;
            const uint32_t per_stage = lane < 2 ? kStageA : kStageB;
            for (int kb = it.kb0; kb < it.kb1; ++kb) {
                int good = 1;
                if (lane == 0) {
                    good = mbar_wait(&empty[stage], phase ^ 1u, abort_flag, P.error, 1) ? 1 : 0;
                    if (good) mbar_expect_tx(&full[stage], bytes);
                }
                good = __shfl_sync(0xffffffffu, good, 0);
                if (!good) { ok = false; break; }
                if (mine) tma_load_2d(base + (uint32_t)stage * per_stage, tm, x, kb * BLOCK_K, &full[stage]);
                issued_mask |= 1u << stage;
                issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok && lane == 0) {
            // let the copies already issued land before the CTA's shared memory goes away
            for (int s = 0; s < kStages; ++s) {
                if (!(issued_mask & (1u << s))) continue;
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(&full[s], (issued_parity >> s) & 1u) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer ===================================
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            int local = 0;
            // descriptors differ only in their address field (16-byte units): one add per stage and k-step
            const uint64_t a_desc0 = smem_desc(smem_u32(sA), 8192, 1024);
            const uint64_t b_desc0 = smem_desc(smem_u32(sB), 8192, 1024);
            constexpr uint32_t kstep = (UMMA_K * 128) >> 4;
            for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++local) {
                const Item it = decode_item(P, item);
                const TcProblem& p = P.p[it.prob];
                const int buf = local & 1;
                const uint32_t use = (uint32_t)(local >> 1);
                if (!mbar_wait(&tempty[buf], (use & 1u) ^ 1u, abort_flag, P.error, 2)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * kMaxBN;
                const uint32_t idesc = instr_desc(p.bn, 1, 1);
                for (int kb = it.kb0; kb < it.kb1; ++kb) {
                    if (!mbar_wait(&full[stage], phase, abort_flag, P.error, 3)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t da = a_desc0 + (uint64_t)((uint32_t)stage * (kStageA >> 4));
                    const uint64_t db = b_desc0 + (uint64_t)((uint32_t)stage * (kStageB >> 4));
                    umma_bf16(d_tmem, da, db, idesc, kb > it.kb0 ? 1u : 0u);
                    umma_bf16(d_tmem, da + kstep, db + kstep, idesc, 1u);
                    umma_bf16(d_tmem, da + 2 * kstep, db + 2 * kstep, idesc, 1u);
                    umma_bf16(d_tmem, da + 3 * kstep, db + 3 * kstep, idesc, 1u);
                    umma_commit(&empty[stage]);       // frees the stage once these MMAs have read it
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(&tfull[buf]);     // accumulator complete
            }
            // all products of this CTA are issued: the next kernel of the stream may be scheduled and set
            // itself up while the last accumulators drain (it waits for this grid before it reads)
            chain_release();
            if (!ok) {
                umma_commit(drain);
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(drain, 0) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else {
        // ================================ epilogue =====================================
        const int q = warp & 3;                    // accumulator lanes 32q .. 32q+31
        const int group = (warp - 2) >> 2;         // handles the 64 columns [64 group, 64 group + 64) of the tile
        bool ok = true;
        int local = 0;
        for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++local) {
            const Item it = decode_item(P, item);
            const TcProblem& p = P.p[it.prob];
            const int buf = local & 1;
            const uint32_t use = (uint32_t)(local >> 1);
            const int row = it.m0 + 32 * q + lane;
            const int chunks = p.bn / 32;
            const bool active = 2 * group < chunks && it.n0 + 64 * group < p.n_extent;   // uniform across the warp
            if (!mbar_wait(&tfull[buf], use & 1u, abort_flag, P.error, 4)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int ci = 0; ci < 2; ++ci) {
                if (!active) break;
                const int c = 2 * group + ci;
                uint32_t acc[32];
                tmem_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * kMaxBN + 32 * c), acc);
                const int col = it.n0 + 32 * c;
                if (row < p.m_extent) {
                    float* dst = p.out32 + (size_t)it.split * p.split_stride + (size_t)row * p.ld_out32 + col;
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        if (col + 4 * g < p.n_extent)
                            *reinterpret_cast<float4*>(dst + 4 * g) =
                                make_float4(__uint_as_float(acc[4 * g]), __uint_as_float(acc[4 * g + 1]),
                                            __uint_as_float(acc[4 * g + 2]), __uint_as_float(acc[4 * g + 3]));
                }
            }
            // the accumulator has been read: hand the tensor-memory buffer back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty[buf]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------ weight-stationary GEMM
// Forward (MODE 0) and data gradient (MODE 1).  Shared memory: a 2 KiB result tile per epilogue warp
// (32 rows x 32 BF16, 64-byte swizzle, one TMA store per 32-column chunk), then the operands: the
// resident weight slab (k-blocks of bn rows x 128 bytes) followed by the A stages of 16 KiB, or, where
// the slab does not fit, stages of A + B.  Tensor memory: two accumulators of 256 columns, so that the
// epilogue of a row tile overlaps the products of the next.
constexpr int kWsMaxStages = 8;
constexpr uint32_t kWsStageOut = 32 * 32 * 2;
constexpr uint32_t kWsBarBytes = 512;
constexpr uint32_t kWsSmem = 231424;                                // 226 KiB: with the 1 KiB the system keeps per block, 1 KiB of
                                                                    // the SM is left for a block without shared memory (the gather)
constexpr uint32_t kWsAuxBox = 128 * 32 * 2;                         // 32 columns x 128 rows of stored post-activations
constexpr uint32_t kWsAuxTile = 4 * kWsAuxBox;                       // a row tile of up to 128 columns
// result tiles (one per epilogue warp) and, for the data gradient, two tiles of stored post-activations
__host__ __device__ constexpr uint32_t ws_staging(int mode) { return kEpiWarps * kWsStageOut + (mode == 1 ? 2u * kWsAuxTile : 0u); }
__host__ __device__ constexpr uint32_t ws_operand_bytes(int mode) { return (kWsSmem - 1024 - ws_staging(mode) - kWsBarBytes) / 1024 * 1024; }

template <int MODE>
__global__ void __launch_bounds__(kThreads, 1) ws_gemm_kernel(const __grid_constant__ TcParams P) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sOut = smem;                                   // a 2 KiB result tile per epilogue warp
    uint8_t* sAux = smem + kEpiWarps * kWsStageOut;          // data gradient: two tiles of stored post-activations
    uint8_t* sOp = smem + ws_staging(MODE);
    uint64_t* full = reinterpret_cast<uint64_t*>(sOp + ws_operand_bytes(MODE));
    uint64_t* empty = full + kWsMaxStages;
    uint64_t* tfull = empty + kWsMaxStages;
    uint64_t* tempty = tfull + 2;
    uint64_t* bfull = tempty + 2;
    uint64_t* drain = bfull + 1;
    uint64_t* auxfull = drain + 1;                           // data gradient: post-activations of a row tile have landed
    uint64_t* auxempty = auxfull + 2;                        // ... and have been read by every epilogue warp
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(auxempty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const WsSlab& S = P.ws.slab[P.ws.cta_slab[blockIdx.x]];
    const TcProblem& p = P.p[S.prob];
    const int rank = (int)blockIdx.x - S.cta_begin;
    const int nst = S.stages;
    const uint32_t b_kb_bytes = (uint32_t)p.bn * 128u;
    const uint32_t stage_bytes = S.resident ? kStageA : kStageA + b_kb_bytes;
    uint8_t* sB = sOp;
    uint8_t* sA = sOp + (S.resident ? (uint32_t)p.kblocks * b_kb_bytes : 0u);
    // set-up: shared memory, tensor memory and kernel parameters only (may overlap the preceding kernel's tail)
    if (threadIdx.x == 0) {
        for (int s = 0; s < kWsMaxStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&tfull[b], 1); mbar_init(&tempty[b], kEpiWarps); }
        mbar_init(bfull, 1); mbar_init(drain, 1);
        for (int b = 0; b < 2; ++b) { mbar_init(&auxfull[b], 1); mbar_init(&auxempty[b], kEpiWarps); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&P.tmA[S.prob]); tma_prefetch_desc(&P.tmB[S.prob]); tma_prefetch_desc(&P.tmOut[S.prob]);
        if (MODE == TC_DGRAD) tma_prefetch_desc(&P.tmAux[S.prob]);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    auto fetch_slab = [&]() {
        mbar_expect_tx(bfull, (uint32_t)p.kblocks * b_kb_bytes);
        for (int kb = 0; kb < p.kblocks; ++kb) tma_load_2d(sB + (uint32_t)kb * b_kb_bytes, &P.tmB[S.prob], kb * BLOCK_K, S.n0, bfull);
    };
    const bool slab_early = S.resident && P.ws.b_early && rank < p.m_tiles;
    if (slab_early && warp == 0 && lane == 0) fetch_slab();      // the weights are older than the kernel waited for below
    chain_wait();

    if (warp == 0) {
        // ================================ TMA producer =================================
        if (lane == 0) {
            const CUtensorMap* tmA = &P.tmA[S.prob];
            const CUtensorMap* tmB = &P.tmB[S.prob];
            if (S.resident && !slab_early) fetch_slab();
            int stage = 0; uint32_t phase = 0;
            uint32_t issued_mask = 0, issued_parity = 0, aux_issued = 0, aux_parity = 0;
            bool ok = true;
            int local = 0;
            const int nchunks = min(p.bn, p.n_extent - S.n0) / 32;     // 32-column chunks of the slab that exist
            for (int mt = rank; ok && mt < p.m_tiles; mt += S.cta_count, ++local) {
                const int m0 = mt * BLOCK_M;
                for (int kb = 0; kb < p.kblocks; ++kb) {
                    if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag, P.error, 1)) { ok = false; break; }
                    mbar_expect_tx(&full[stage], stage_bytes);
                    uint8_t* dst = sA + (uint32_t)stage * stage_bytes;
                    tma_load_2d(dst, tmA, kb * BLOCK_K, m0, &full[stage]);
                    if (!S.resident) tma_load_2d(dst + kStageA, tmB, kb * BLOCK_K, S.n0, &full[stage]);
                    issued_mask |= 1u << stage;
                    issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == nst) { stage = 0; phase ^= 1u; }
                }
                if (MODE == TC_DGRAD && ok) {
                    // stored post-activations of the row tile, one box of 32 columns x 128 rows per chunk, fetched
                    // behind the operands of the tile (the epilogue reads them after the products)
                    const int ab = local & 1;
                    if (!mbar_wait(&auxempty[ab], (((uint32_t)local >> 1) & 1u) ^ 1u, abort_flag, P.error, 7)) { ok = false; break; }
                    mbar_expect_tx(&auxfull[ab], (uint32_t)nchunks * kWsAuxBox);
                    for (int c = 0; c < nchunks; ++c)
                        tma_load_2d(sAux + (uint32_t)ab * kWsAuxTile + (uint32_t)c * kWsAuxBox, &P.tmAux[S.prob], S.n0 + 32 * c, m0, &auxfull[ab]);
                    aux_issued |= 1u << ab;
                    aux_parity = (aux_parity & ~(1u << ab)) | ((((uint32_t)local >> 1) & 1u) << ab);
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA's shared memory goes away
                for (int s = 0; s < nst; ++s) {
                    if (!(issued_mask & (1u << s))) continue;
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(&full[s], (issued_parity >> s) & 1u) && global_ns() - t0 < kWaitLimitNs) {}
                }
                if (S.resident) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bfull, 0) && global_ns() - t0 < kWaitLimitNs) {}
                }
                for (int ab = 0; ab < 2; ++ab) {
                    if (!(aux_issued & (1u << ab))) continue;
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(&auxfull[ab], (aux_parity >> ab) & 1u) && global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer ===================================
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            const uint32_t idesc = instr_desc(p.bn, 0, 0);
            // operand descriptors differ only in their address field (16-byte units, no carry out of it for
            // shared-memory addresses): one add per stage / k-block / k-step instead of a rebuild
            const uint64_t a_desc0 = smem_desc(smem_u32(sA), 16, 1024);
            const uint64_t b_desc0 = smem_desc(smem_u32(S.resident ? sB : sA + kStageA), 16, 1024);
            const uint64_t a_step = stage_bytes >> 4;
            const uint64_t b_step = S.resident ? (b_kb_bytes >> 4) : a_step;
            const int kblocks = p.kblocks;
            const bool resident = S.resident != 0;
            if (resident && !mbar_wait(bfull, 0, abort_flag, P.error, 6)) ok = false;
            uint64_t a_desc = a_desc0, b_desc_stream = b_desc0;
            int local = 0;
            for (int mt = rank; ok && mt < p.m_tiles; mt += S.cta_count, ++local) {
                const int buf = local & 1;
                const uint32_t use = (uint32_t)(local >> 1);
                if (!mbar_wait(&tempty[buf], (use & 1u) ^ 1u, abort_flag, P.error, 2)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * kMaxBN;
                uint64_t b_res = b_desc0;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&full[stage], phase, abort_flag, P.error, 3)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t db = resident ? b_res : b_desc_stream;
                    umma_bf16(d_tmem, a_desc, db, idesc, kb > 0 ? 1u : 0u);
                    umma_bf16(d_tmem, a_desc + 2, db + 2, idesc, 1u);
                    umma_bf16(d_tmem, a_desc + 4, db + 4, idesc, 1u);
                    umma_bf16(d_tmem, a_desc + 6, db + 6, idesc, 1u);
                    umma_commit(&empty[stage]);       // frees the stage once these MMAs have read it
                    b_res += b_step;
                    a_desc += a_step; b_desc_stream += a_step;
                    if (++stage == nst) { stage = 0; phase ^= 1u; a_desc = a_desc0; b_desc_stream = b_desc0; }
                }
                if (ok) umma_commit(&tfull[buf]);     // accumulator complete
            }
            // all products of this CTA are issued: the next kernel of the stream may be scheduled and set
            // itself up while the last accumulators drain (it waits for this grid before it reads)
            chain_release();
            if (!ok) {
                umma_commit(drain);
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(drain, 0) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else {
        // ================================ epilogue =====================================
        const int q = warp & 3;                    // accumulator lanes 32q .. 32q+31
        const int group = (warp - 2) >> 2;         // the 32-column chunks group and group + 4 of the tile
        // lane r owns row r of a 32 x 32 BF16 tile (64 bytes = four 16-byte pieces); piece j is kept at
        // j ^ ((r >> 1) & 3), the 64-byte swizzle of the tensor maps (conflict-free for the warp).
        // Data gradient: the stored post-activations of the row tile are read from the tile the producer fetched
        // (same layout, rows 32q.. of the chunk's box).
        uint8_t* tile = sOut + (warp - 2) * kWsStageOut;
        uint8_t* tile_row = tile + lane * 64;
        const int sw = (lane >> 1) & 3;
        bool ok = true;
        const int chunks = p.bn / 32;
        // this warp's chunks that exist (uniform across the warp): with up to 128 columns every warp has at most one
        int nact = 0;
        for (int ci = 0; ci < 2; ++ci)
            if (group + 4 * ci < chunks && S.n0 + 32 * (group + 4 * ci) < p.n_extent) nact = ci + 1;
        const CUtensorMap* tmOut = &P.tmOut[S.prob];
        int local = 0;
        for (int mt = rank; ok && mt < p.m_tiles; mt += S.cta_count, ++local) {
            const int m0 = mt * BLOCK_M;
            const int buf = local & 1;
            const uint32_t use = (uint32_t)(local >> 1);
            const int row0 = m0 + 32 * q;
            if (!mbar_wait(&tfull[buf], use & 1u, abort_flag, P.error, 4)) { ok = false; break; }
            tc_fence_after();
            if (MODE == TC_DGRAD && !mbar_wait(&auxfull[buf], use & 1u, abort_flag, P.error, 5)) { ok = false; break; }
            const uint32_t t_row = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * kMaxBN);
            // the accumulator is read in pieces of 16 columns, each fetched while the piece before is worked on
            uint32_t acc[2][16];
            if (nact > 0) tmem_ld16_issue(t_row + (uint32_t)(32 * group), acc[0]);
#pragma unroll
            for (int ci = 0; ci < 2; ++ci) {
                if (ci >= nact) break;
                const int c = group + 4 * ci;
                const int col = S.n0 + 32 * c;
                const uint8_t* aux_row = sAux + (uint32_t)buf * kWsAuxTile + (uint32_t)c * kWsAuxBox + (uint32_t)(32 * q + lane) * 64u;
                // the previous chunk's store must have read the tile before it is rewritten
                if (lane == 0) tma_store_wait_read();
                __syncwarp();
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t (&cur)[16] = acc[half];
                    float bv[16];
                    if (MODE == TC_FWD) {
                        // p.bias is zero-padded to the padded width: no bounds checks
                        const float4* b4 = reinterpret_cast<const float4*>(p.bias + col + 16 * half);
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const float4 t4 = __ldg(b4 + g);
                            bv[4 * g] = t4.x; bv[4 * g + 1] = t4.y; bv[4 * g + 2] = t4.z; bv[4 * g + 3] = t4.w;
                        }
                    }
                    tmem_ld16_wait(cur);
                    // next piece: the other half of this chunk, or the first half of the warp's second chunk
                    if (half == 0) tmem_ld16_issue(t_row + (uint32_t)(32 * c + 16), acc[1]);
                    else if (ci + 1 < nact) tmem_ld16_issue(t_row + (uint32_t)(32 * (c + 4)), acc[0]);
                    else {
                        // (issued loads are complete at this point) the accumulator has been read: hand the buffer back
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&tempty[buf]);
                    }
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        uint32_t o[4];
                        uint4* piece = reinterpret_cast<uint4*>(tile_row + (((2 * half + g) ^ sw) << 4));
                        if (MODE == TC_FWD) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float v0 = elu_fast(__uint_as_float(cur[8 * g + 2 * e]) + bv[8 * g + 2 * e], P.alpha);
                                const float v1 = elu_fast(__uint_as_float(cur[8 * g + 2 * e + 1]) + bv[8 * g + 2 * e + 1], P.alpha);
                                __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
                                o[e] = *reinterpret_cast<uint32_t*>(&h2);
                            }
                        } else {
                            const uint4 hv = *reinterpret_cast<const uint4*>(aux_row + (((2 * half + g) ^ sw) << 4));
                            const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 h2 = *reinterpret_cast<const __nv_bfloat162*>(&hw[e]);
                                const float h0 = __low2float(h2), h1 = __high2float(h2);
                                const float v0 = __uint_as_float(cur[8 * g + 2 * e]) * (h0 > 0.f ? 1.0f : h0 + P.alpha);
                                const float v1 = __uint_as_float(cur[8 * g + 2 * e + 1]) * (h1 > 0.f ? 1.0f : h1 + P.alpha);
                                __nv_bfloat162 r2 = __floats2bfloat162_rn(v0, v1);
                                o[e] = *reinterpret_cast<uint32_t*>(&r2);
                            }
                        }
                        *piece = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
                fence_async_smem();                           // tile writes -> visible to the copy engine
                __syncwarp();
                // rows at or beyond the tensor's extent are clipped by the store itself
                if (lane == 0 && row0 < p.m_extent) tma_store_2d(tmOut, tile, col, row0);
                if (MODE == TC_DGRAD) {
                    if (p.colsum) {
                        // partial bias gradient: lanes 0..15 add columns 2l, 2l+1 over rows 0..15 of the tile, lanes
                        // 16..31 over rows 16..31 (rows past the extent hold zeros)
                        float s0 = 0.f, s1 = 0.f;
                        const int cp = lane & 15, rbase = lane & 16;
                        const uint8_t* mine = tile + ((cp & 3) << 2);
#pragma unroll
                        for (int r = 0; r < 16; ++r) {
                            const int rr = rbase + r;
                            const uint32_t w = *reinterpret_cast<const uint32_t*>(mine + rr * 64 + (((cp >> 2) ^ ((rr >> 1) & 3)) << 4));
                            const __nv_bfloat162 v2 = *reinterpret_cast<const __nv_bfloat162*>(&w);
                            s0 += __low2float(v2); s1 += __high2float(v2);
                        }
                        s0 += __shfl_xor_sync(0xffffffffu, s0, 16);
                        s1 += __shfl_xor_sync(0xffffffffu, s1, 16);
                        if (lane < 16)
                            *reinterpret_cast<float2*>(p.colsum + (size_t)(mt * 4 + q) * p.ld_colsum + col + 2 * cp) = make_float2(s0, s1);
                    }
                }
            }
            if (MODE == TC_DGRAD) {
                // this warp has read its part of the row tile's post-activations
                __syncwarp();
                if (lane == 0) mbar_arrive(&auxempty[buf]);
            }
            if (nact == 0) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tempty[buf]);
            }
        }
        if (lane == 0) tma_store_wait_all();   // stores done before the CTA retires
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------ fused forward chain
// All hidden layers of a net on one 128-row tile inside one CTA: the BF16 activations of a layer
// stay in shared memory, in the K-major swizzled layout the next layer's MMA reads as its A
// operand (and the TMA store reads to write them to global memory for the backward pass); only
// the weights (and the observations of the first layer) stream through the ring.  A tile runs a
// short program the host compiled from the layer widths: MMA jobs, each a run of k-blocks into
// one accumulator of up to 256 tensor-memory columns, and epilogues, each turning one
// accumulator into activations.  Jobs and epilogues name what they wait for, so an epilogue
// overlaps the jobs that do not need its result.  A first layer wider than 256 is produced in
// two halves, and the second layer accumulates over each half as soon as it exists.
constexpr int kChainLayers = 4;                  // hidden layers per net
constexpr int kChainJobs = 8;
constexpr int kChainEpis = 6;
// The operand ring is cut into 16 KiB slots: a k-block takes one slot for its A tile (first layer only)
// and one or two for its B tile, contiguous, and both ends of the ring skip the tail when a k-block
// would wrap.  Jobs with small tiles therefore keep more k-blocks in flight.
constexpr int kSlots = 9;
constexpr uint32_t kSlotBytes = 16384;
constexpr uint32_t kActBytes = BLOCK_M * kMaxBN * 2;     // 64 KiB = four [128 rows][64] blocks
constexpr int kChainBiasFloats = 2 * (512 + (kChainLayers - 1) * 256);
constexpr int kChainHeadFloats = 256 + kEpiWarps * 32;   // head constants, then one log-probability partial per epilogue thread
constexpr size_t kChainSmem = 1024 + (size_t)kSlots * kSlotBytes + kActBytes + kChainBiasFloats * 4 + kChainHeadFloats * 4 + 512;
__host__ __device__ constexpr int slots_of(int a_ring, int bn) { return a_ring + (bn * BLOCK_K * 2 + (int)kSlotBytes - 1) / (int)kSlotBytes; }
constexpr int kPrevItem = 16;                    // added to an epilogue index: that epilogue of the CTA's previous item

struct ChainJob {
    int layer;           // whose weights
    int n0, bn;          // output columns [n0, n0 + bn) = rows of the weight operand
    int kb0, nkb;        // k-blocks [kb0, kb0 + nkb) of that layer's contraction
    int a_ring;          // 1: A k-blocks (observations) come through the ring; 0: block i of the activation buffer
    int tmem_col;        // accumulator columns [tmem_col, tmem_col + bn)
    int accumulate;      // 1: adds to what the accumulator holds
    int wait_epi;        // epilogue that must have finished before the first MMA (-1: none; + kPrevItem: of the previous item):
                         // it wrote the activations this job reads, or drained the accumulator this job overwrites
};
struct ChainEpi {
    int head;            // 1: the head epilogue (rollout outputs) instead of bias + ELU
    int layer, n0, ncols, tmem_col;   // columns [n0, n0 + ncols) of `layer` from these accumulator columns
    int wait_job;        // the job that completes the accumulator
    int write_job;       // a later job that still reads the activation buffer (-1: none): done before the buffer is rewritten
};
struct ChainNet {
    int nlayers, njobs, nepis;
    int flip;            // 1: odd items of a CTA use the other half of tensor memory for every accumulator
    ChainJob job[kChainJobs];
    ChainEpi epi[kChainEpis];
    const float* bias[kChainLayers];  // zero-padded to the padded width
    int bias_n[kChainLayers];         // that width
    int bias_off[kChainLayers];       // where the kernel keeps the layer's bias in shared memory (floats)
    int is_actor, A, head_n;          // head epilogue: policy head with A outputs, or the value head; its accumulator holds
                                      // h Wt_hi in columns [0, head_n) and h Wt_lo in [head_n, 2 head_n)
    const float* head_bias;           // [64] zero-padded
};
// What the head epilogue of the rollout writes (storage row of the current step).
struct ChainHeadOut {
    float* actions; float* mu; float* sigma; float* logp; float* values; float* actions_out;   // actions_out may be null
    int act_stride;
    const float* log_std;
    uint32_t seed_lo, seed_hi, global_step;
};
struct ChainParams {
    CUtensorMap tmX[2];                       // first-layer input, boxes of 64 x 128 rows
    CUtensorMap tmW[2][kChainLayers + 1];     // [out][in] weights, boxes of 64 x (columns per job); last: the head
    ChainHeadOut ho;
    CUtensorMap tmOut[2][kChainLayers];       // activations, boxes of 64 columns x 32 rows
    ChainNet net[2];                          // same numbers of jobs and epilogues, same waits
    int nnets, rows, total_items;             // items = (row tile, net), nets interleaved
    int store;                                // 1: the activations are also written to global memory (tmOut)
    float alpha;
    int* error;
};

__global__ void __launch_bounds__(kThreads, 1) chain_fwd_kernel(const __grid_constant__ ChainParams P) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sRing = smem;
    uint8_t* sAct = sRing + kSlots * kSlotBytes;
    float* sBias = reinterpret_cast<float*>(sAct + kActBytes);
    float* sHead = sBias + kChainBiasFloats;   // policy head bias [64], log_std [64], sigma [64], value head bias
    uint64_t* full = reinterpret_cast<uint64_t*>(sHead + kChainHeadFloats);
    uint64_t* empty = full + kSlots;
    uint64_t* job_done = empty + kSlots;       // one completion per item each
    uint64_t* epi_done = job_done + kChainJobs;
    uint64_t* drain = epi_done + kChainEpis;
    uint64_t* head_bar = drain + 1;            // one per lane quarter: the three other warps of a row group have written their partials
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(head_bar + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // set-up spread over lanes (a single thread pays about five cycles per dependent instruction): warp 0 initialises
    // the barriers, a lane each; warp 1 allocates tensor memory; warp 2 prefetches the tensor maps, a lane each
    if (warp == 0) {
        if (lane < kSlots) { mbar_init(&full[lane], 1); mbar_init(&empty[lane], 1); }
        if (lane < kChainJobs) mbar_init(&job_done[lane], 1);
        if (lane < kChainEpis) mbar_init(&epi_done[lane], kEpiWarps);
        if (lane == 0) { mbar_init(drain, 1); *abort_flag = 0; }
        if (lane < 4) mbar_init(&head_bar[lane], 3);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    if (warp == 2) {
        constexpr int per_net = 1 + 2 * kChainLayers;
        const int n = lane / per_net, r = lane - n * per_net;
        if (n < P.nnets) {
            if (r == 0) tma_prefetch_desc(&P.tmX[n]);
            else if (r - 1 < P.net[n].nlayers) tma_prefetch_desc(&P.tmW[n][r - 1]);
            else if (r - 1 - kChainLayers >= 0 && r - 1 - kChainLayers < P.net[n].nlayers) tma_prefetch_desc(&P.tmOut[n][r - 1 - kChainLayers]);
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // The epilogues read the biases between two MMA jobs: keep them close.  Biases, head biases and log_std are
    // parameters: the launch before this one in the stream (the observation staging) does not write them, and it
    // has itself waited for everything earlier, so they are staged before the wait, beside that launch.  Only the
    // epilogue warps need them: they stage them and meet at a barrier of their own, so that the producer's first
    // loads do not wait for this.
    constexpr int kEpiThreads = 32 * kEpiWarps;
    const int et = (int)threadIdx.x - 64;          // index among the epilogue threads
    if (warp >= 2) {
        for (int n = 0; n < P.nnets; ++n)
            for (int l = 0; l < P.net[n].nlayers; ++l)
                for (int i = et; i < P.net[n].bias_n[l]; i += kEpiThreads) sBias[P.net[n].bias_off[l] + i] = P.net[n].bias[l][i];
        for (int n = 0; n < P.nnets; ++n) {
            const ChainNet& N = P.net[n];
            if (N.A <= 0) continue;                  // no head epilogue
            if (N.is_actor) {
                for (int i = et; i < 64; i += kEpiThreads) {
                    const float ls = i < N.A ? P.ho.log_std[i] : 0.f;
                    sHead[i] = N.head_bias[i];
                    sHead[64 + i] = ls;
                    sHead[128 + i] = expf(ls);
                }
            } else if (et == 0) {
                sHead[192] = N.head_bias[0];
            }
        }
    }
    chain_wait();
    if (warp >= 2) {
        // sigma does not depend on the state: one vector per rollout step
        for (int n = 0; n < P.nnets; ++n) {
            const ChainNet& N = P.net[n];
            if (N.A > 0 && N.is_actor && blockIdx.x == 0)
                for (int i = et; i < P.ho.act_stride; i += kEpiThreads) P.ho.sigma[i] = i < N.A ? expf(P.ho.log_std[i]) : 0.f;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
    }

    if (warp == 0) {
        // ================================ TMA producer =================================
        if (lane == 0) {
            int pos = 0;
            uint32_t full_bits = 0, empty_bits = 0;     // parity of the next use of each slot's barriers
            uint32_t issued_mask = 0, issued_parity = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x) {
                const int ni = item % P.nnets, m0 = (item / P.nnets) * BLOCK_M;
                const ChainNet& N = P.net[ni];
                for (int j = 0; ok && j < N.njobs; ++j) {
                    const ChainJob& J = N.job[j];
                    const int need = slots_of(J.a_ring, J.bn);
                    const uint32_t bytes = (uint32_t)J.bn * BLOCK_K * 2 + (J.a_ring ? kSlotBytes : 0u);
                    for (int kb = J.kb0; ok && kb < J.kb0 + J.nkb; ++kb) {
                        if (pos + need > kSlots) pos = 0;
                        for (int s = pos; s < pos + need; ++s)
                            if (!mbar_wait(&empty[s], ((empty_bits >> s) & 1u) ^ 1u, abort_flag, P.error, 11)) { ok = false; break; }
                        if (!ok) break;
                        mbar_expect_tx(&full[pos], bytes);
                        uint8_t* dst = sRing + pos * kSlotBytes;
                        if (J.a_ring) { tma_load_2d(dst, &P.tmX[ni], kb * BLOCK_K, m0, &full[pos]); dst += kSlotBytes; }
                        tma_load_2d(dst, &P.tmW[ni][J.layer], kb * BLOCK_K, J.n0, &full[pos]);
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
            const uint64_t ring_desc0 = smem_desc(smem_u32(sRing), 16, 1024);
            const uint64_t act_desc0 = smem_desc(smem_u32(sAct), 16, 1024);
            for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++t) {
                const ChainNet& N = P.net[item % P.nnets];
                const uint32_t flip = (N.flip && (t & 1u)) ? 256u : 0u;
                for (int j = 0; ok && j < N.njobs; ++j) {
                    const ChainJob& J = N.job[j];
                    if (J.wait_epi >= kPrevItem) {
                        if (t > 0 && !mbar_wait(&epi_done[J.wait_epi - kPrevItem], (t - 1) & 1u, abort_flag, P.error, 12)) { ok = false; break; }
                    } else if (J.wait_epi >= 0) {
                        if (!mbar_wait(&epi_done[J.wait_epi], t & 1u, abort_flag, P.error, 12)) { ok = false; break; }
                    }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + ((uint32_t)J.tmem_col ^ flip);
                    const uint32_t idesc = instr_desc(J.bn, 0, 0);
                    const int need = slots_of(J.a_ring, J.bn);
                    for (int i = 0; i < J.nkb; ++i) {
                        if (pos + need > kSlots) pos = 0;
                        if (!mbar_wait(&full[pos], (full_bits >> pos) & 1u, abort_flag, P.error, 13)) { ok = false; break; }
                        full_bits ^= 1u << pos;
                        tc_fence_after();
                        // descriptors differ only in their address field (16-byte units): additions, not rebuilds
                        const uint64_t ring_desc = ring_desc0 + (uint64_t)((uint32_t)pos * (kSlotBytes >> 4));
                        const uint64_t da = J.a_ring ? ring_desc : act_desc0 + (uint64_t)((uint32_t)i * (kStageA >> 4));
                        const uint64_t db = ring_desc + (J.a_ring ? (uint64_t)(kSlotBytes >> 4) : 0ull);
                        constexpr uint32_t kstep = (UMMA_K * 2) >> 4;
                        umma_bf16(d_tmem, da, db, idesc, (J.accumulate || i > 0) ? 1u : 0u);
                        umma_bf16(d_tmem, da + kstep, db + kstep, idesc, 1u);
                        umma_bf16(d_tmem, da + 2 * kstep, db + 2 * kstep, idesc, 1u);
                        umma_bf16(d_tmem, da + 3 * kstep, db + 3 * kstep, idesc, 1u);
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
        // pieces), piece j is kept at j ^ (r & 7), the 128-byte swizzle both the MMA and the store expect
        uint8_t* tile = sAct + g * kStageA + q * (32 * 128);
        uint8_t* tile_row = tile + lane * 128;
        const int sw = lane & 7;
        bool ok = true;
        uint32_t t = 0;
        uint32_t head_uses = 0;                    // policy-head epilogues this warp has waited for
        for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++t) {
            const int ni = item % P.nnets, m0 = (item / P.nnets) * BLOCK_M;
            const ChainNet& N = P.net[ni];
            const uint32_t flip = (N.flip && (t & 1u)) ? 256u : 0u;
            for (int e = 0; e < N.nepis; ++e) {
                const ChainEpi& E = N.epi[e];
                if (!mbar_wait(&job_done[E.wait_job], t & 1u, abort_flag, P.error, 14)) { ok = false; break; }
                tc_fence_after();
                if (E.head) {
                    // rollout outputs of the tile's rows, one thread per row (the first column group's warps)
                    // (the accumulator loads are warp-wide; only the stores depend on the row being there)
                    const int n = m0 + 32 * q + lane;
                    const bool live = n < P.rows;
                    const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + ((uint32_t)E.tmem_col ^ flip);
                    const ChainHeadOut& H = P.ho;
                    if (N.is_actor) {
                        // one thread per row and group of four actions (one Philox block): the four warps that own the
                        // same rows (g = 0..3) take the groups in turn, so a policy of up to 16 actions is one round
                        float* arow = H.actions + (size_t)n * H.act_stride;
                        float* mrow = H.mu + (size_t)n * H.act_stride;
                        float* orow = H.actions_out ? H.actions_out + (size_t)n * H.act_stride : nullptr;
                        float logp = 0.f;
                        for (int c = 4 * g; c < H.act_stride; c += 16) {
                            float av[4] = {0.f, 0.f, 0.f, 0.f}, mv[4] = {0.f, 0.f, 0.f, 0.f};
                            if (c < N.A) {
                                uint32_t a4[4], l4[4];
                                tmem_ld4(taddr + (uint32_t)c, a4);
                                tmem_ld4(taddr + (uint32_t)(N.head_n + c), l4);
                                float eps[4];
                                gaussian_quad(H.seed_lo, H.seed_hi, (uint32_t)n, H.global_step, (uint32_t)(c >> 2), eps);
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const int i = c + k;
                                    if (i < N.A) {
                                        const float m = (__uint_as_float(a4[k]) + __uint_as_float(l4[k])) + sHead[i];
                                        const float ls = sHead[64 + i], sg = sHead[128 + i];
                                        const float a = fmaf(sg, eps[k], m);
                                        const float d = a - m;
                                        logp += -(d * d) / (2.0f * sg * sg) - ls - 0.91893853320467274178f;
                                        av[k] = a; mv[k] = m;
                                    }
                                }
                            }
                            if (live) {
                                *reinterpret_cast<float4*>(arow + c) = make_float4(av[0], av[1], av[2], av[3]);
                                *reinterpret_cast<float4*>(mrow + c) = make_float4(mv[0], mv[1], mv[2], mv[3]);
                                if (orow) { orow[c] = av[0]; orow[c + 1] = av[1]; orow[c + 2] = av[2]; orow[c + 3] = av[3]; }   // caller's buffer: 4-byte aligned only
                            }
                        }
                        // the row's log-probability: the partials of the four warps, added in the order of the actions.
                        // The three other warps publish theirs and arrive on the row group's barrier; the first warp
                        // waits for them with the usual bound.  The next item's partials cannot be written before this
                        // epilogue has been reported done by all of its warps (the item's first job waits for that).
                        float* part = sHead + 256;
                        if (g != 0) {
                            part[(4 * q + g) * 32 + lane] = logp;
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&head_bar[q]);
                        } else {
                            if (!mbar_wait(&head_bar[q], head_uses & 1u, abort_flag, P.error, 16)) { ok = false; break; }
                            ++head_uses;
                            if (live) {
                                float lp = logp;
#pragma unroll
                                for (int gg = 1; gg < 4; ++gg) lp += part[(4 * q + gg) * 32 + lane];
                                H.logp[n] = lp;
                            }
                        }
                    } else if (g == 0) {
                        uint32_t a4[4], l4[4];
                        tmem_ld4(taddr, a4);
                        tmem_ld4(taddr + (uint32_t)N.head_n, l4);
                        if (live) H.values[n] = (__uint_as_float(a4[0]) + __uint_as_float(l4[0])) + sHead[192];
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&epi_done[e]);
                    continue;
                }
                const bool active = 64 * g < E.ncols;          // uniform across the warp
                // Nothing still reads the activation buffer: the results go to it as they are formed, 16 accumulator
                // columns at a time, the next 16 in flight meanwhile.
                const bool direct = active && E.write_job < 0;
                if (direct) {
                    if (P.store) {
                        if (lane == 0) tma_store_wait_read();   // this warp's last store has read the rows
                        __syncwarp();
                    }
                    const float* bias = sBias + N.bias_off[E.layer] + E.n0 + 64 * g;
                    const uint32_t t_row = tmem_base + ((uint32_t)(32 * q) << 16) + (((uint32_t)E.tmem_col ^ flip) + (uint32_t)(64 * g));
                    uint32_t acc[2][16];
                    tmem_ld16_issue(t_row, acc[0]);
#pragma unroll
                    for (int pc = 0; pc < 4; ++pc) {
                        uint32_t (&cur)[16] = acc[pc & 1];
                        float bv[16];
                        const float4* b4 = reinterpret_cast<const float4*>(bias + 16 * pc);
#pragma unroll
                        for (int gg = 0; gg < 4; ++gg) {
                            const float4 t4 = b4[gg];
                            bv[4 * gg] = t4.x; bv[4 * gg + 1] = t4.y; bv[4 * gg + 2] = t4.z; bv[4 * gg + 3] = t4.w;
                        }
                        tmem_ld16_wait(cur);
                        if (pc < 3) tmem_ld16_issue(t_row + (uint32_t)(16 * (pc + 1)), acc[(pc + 1) & 1]);
#pragma unroll
                        for (int gq = 0; gq < 2; ++gq) {
                            uint32_t o[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const float v0 = elu_fast(__uint_as_float(cur[8 * gq + 2 * k]) + bv[8 * gq + 2 * k], P.alpha);
                                const float v1 = elu_fast(__uint_as_float(cur[8 * gq + 2 * k + 1]) + bv[8 * gq + 2 * k + 1], P.alpha);
                                __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
                                o[k] = *reinterpret_cast<uint32_t*>(&h2);
                            }
                            *reinterpret_cast<uint4*>(tile_row + (((2 * pc + gq) ^ sw) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                    fence_async_smem();                         // rows -> visible to the MMA and the copy engine
                }
                uint4 outv[8];
                if (active && !direct) {
                    const float* bias = sBias + N.bias_off[E.layer] + E.n0 + 64 * g;
#pragma unroll
                    for (int ci = 0; ci < 2; ++ci) {
                        uint32_t acc[32];
                        tmem_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (((uint32_t)E.tmem_col ^ flip) + (uint32_t)(64 * g + 32 * ci)), acc);
                        const float4* b4 = reinterpret_cast<const float4*>(bias + 32 * ci);
#pragma unroll
                        for (int gg = 0; gg < 4; ++gg) {
                            const float4 ba = b4[2 * gg], bb = b4[2 * gg + 1];
                            const float bv[8] = {ba.x, ba.y, ba.z, ba.w, bb.x, bb.y, bb.z, bb.w};
                            uint32_t o[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const float v0 = elu_fast(__uint_as_float(acc[8 * gg + 2 * k]) + bv[2 * k], P.alpha);
                                const float v1 = elu_fast(__uint_as_float(acc[8 * gg + 2 * k + 1]) + bv[2 * k + 1], P.alpha);
                                __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
                                o[k] = *reinterpret_cast<uint32_t*>(&h2);
                            }
                            outv[4 * ci + gg] = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
                // the accumulator is in registers; the buffer may still feed a job that runs meanwhile
                if (E.write_job >= 0 && !mbar_wait(&job_done[E.write_job], t & 1u, abort_flag, P.error, 15)) { ok = false; break; }
                if (active && !direct) {
                    if (P.store) {
                        if (lane == 0) tma_store_wait_read();   // this warp's last store has read the rows
                        __syncwarp();
                    }
#pragma unroll
                    for (int p8 = 0; p8 < 8; ++p8) *reinterpret_cast<uint4*>(tile_row + ((p8 ^ sw) << 4)) = outv[p8];
                    fence_async_smem();                         // rows -> visible to the MMA and the copy engine
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    // rows at or beyond the tensor's extent are clipped by the store itself
                    if (P.store && active && m0 + 32 * q < P.rows) tma_store_2d(&P.tmOut[ni][E.layer], tile, E.n0 + 64 * g, m0 + 32 * q);
                    mbar_arrive(&epi_done[e]);
                }
            }
        }
        if (P.store && lane == 0) tma_store_wait_all();   // stores done before the CTA retires
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------- small kernels
struct CvtEntry {
    const float* bsrc; float* bdst;             // bias -> zero-padded FP32 copy
    const float* src; int in, out, ld_src;      // FP32 master W[in][ld_src]
    __nv_bfloat16* wt; int ld_wt;               // [out][ld_wt]  (contraction = in)   forward operand
    __nv_bfloat16* wn; int ld_wn;               // [in][ld_wn]   (contraction = out)  data-gradient operand, may be null
    __nv_bfloat16* wt_lo;                       // [out][ld_wt]  what BF16 rounding left of the weight (heads only, else null)
};

__global__ void convert_weights_kernel(const CvtEntry* __restrict__ table) {
    const CvtEntry e = table[blockIdx.y];
    const int total = e.in * e.out;
    for (int o = blockIdx.x * blockDim.x + threadIdx.x; o < e.out; o += gridDim.x * blockDim.x) e.bdst[o] = e.bsrc[o];
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int i = idx / e.out, o = idx - i * e.out;
        const __nv_bfloat16 v = __float2bfloat16_rn(e.src[(size_t)i * e.ld_src + o]);
        e.wt[(size_t)o * e.ld_wt + i] = v;
        if (e.wn) e.wn[(size_t)i * e.ld_wn + o] = v;
        if (e.wt_lo) e.wt_lo[(size_t)o * e.ld_wt + i] = __float2bfloat16_rn(e.src[(size_t)i * e.ld_src + o] - __bfloat162float(v));
    }
}

// ------------------------------------------------------------------------------- host side
inline int round_up(int x, int m) { return (x + m - 1) / m * m; }
inline int pick_bn(int width) { return std::min(kMaxBN, width); }   // widths are multiples of 64

}  // namespace

struct UmmaEngine {
    UmmaSetup s;
    int nh[2];                                   // hidden layers per net
    int kp[2];                                   // padded observation width
    int pw[2][kMaxLayers];                       // padded hidden widths
    std::vector<void*> allocs;
    __nv_bfloat16 *obs16_act[2] = {}, *h_act[2][kMaxLayers] = {};
    __nv_bfloat16 *x16[2] = {}, *h[2][kMaxLayers] = {}, *dz[2][kMaxLayers] = {};
    __nv_bfloat16* x16_alt[2] = {};               // second minibatch input buffer (the gather of the next step fills it)
    __nv_bfloat16 *dmu16 = nullptr, *dv16 = nullptr;
    __nv_bfloat16 *wt[2][kMaxLayers] = {}, *wn[2][kMaxLayers] = {};
    float* bias_pad[2][kMaxLayers] = {};         // [pw] zero-padded copies of the hidden biases
    float* bias_slots[2][kMaxLayers] = {};       // [4 m_tiles][pw] bias-gradient partials written by the data-gradient epilogue
    int n_slots = 0, n_sources = 0;
    float* head_slots[2] = {};                   // [head/loss blocks][pw of the last hidden layer]: its bias-gradient partials
    CvtEntry* cvt_dev = nullptr; int n_cvt = 0; int cvt_max = 0;
    int* error_dev = nullptr;
    int num_sms = 148;
    std::vector<TcParams> act_fwd, act_fwd_critic, upd_fwd, upd_dgrad, upd_wgrad;
    // the launches that read the minibatch observations, once more for the second input buffer
    std::vector<TcParams> upd_fwd_alt, upd_wgrad_alt;
    // forward and data-gradient launches of the actor alone (the distillation step trains no critic)
    std::vector<TcParams> fwd_actor[2], dgrad_actor;
    // fused forward (one launch for all hidden layers) where the widths allow it, else empty
    std::vector<ChainParams> chain_act, chain_act_critic;
    ColsumBatch colsum{}, colsum_rest{};         // all layers the epilogue does not cover / those minus the last ones
    // head operand copies (output-major with high and low parts, input-major)
    __nv_bfloat16 *wht[2] = {}, *whn[2] = {};
    float* head_bias_pad[2] = {};
    bool head_copies = false;                    // the optimiser step keeps wht / whn / head_bias_pad current
    int head_n[2] = {};                          // head outputs rounded up to 16; wht rows [head_n, 2 head_n) hold the
                                                 // low-order parts of the weights (what BF16 rounding left)
};

namespace {

template <typename T>
bool ealloc(UmmaEngine* e, T** p, size_t count) {
    void* q = nullptr;
    const size_t bytes = std::max<size_t>(count, 1) * sizeof(T);
    if (guarded_malloc(&q, bytes) != cudaSuccess) return false;
    e->allocs.push_back(q);
    if (cudaMemsetAsync(q, 0, bytes, e->s.stream) != cudaSuccess) return false;
    *p = reinterpret_cast<T*>(q);
    return true;
}

void finish_params(TcParams& P, float alpha, int* error) {
    int items = 0;
    for (int i = 0; i < P.count; ++i) {
        P.p[i].item_begin = items;
        items += P.p[i].m_tiles * P.p[i].n_tiles * P.p[i].splits;
    }
    P.total_items = items;
    P.alpha = alpha;
    P.error = error;
}

void plan_ws(TcParams& P, int num_sms, int mode);

// The problems of one net out of a launch's parameters, as a launch of their own (no items if there are none).
TcParams only_net(const TcParams& P, int ni) {
    TcParams Q;
    memset(&Q, 0, sizeof Q);
    for (int i = 0; i < P.count; ++i) {
        if (P.p[i].net_id != ni) continue;
        const int j = Q.count++;
        Q.tmA[j] = P.tmA[i]; Q.tmB[j] = P.tmB[i]; Q.tmOut[j] = P.tmOut[i]; Q.tmAux[j] = P.tmAux[i];
        Q.p[j] = P.p[i];
    }
    finish_params(Q, P.alpha, P.error);
    plan_ws(Q, P.ws.num_sms, P.ws.mode);
    Q.ws.b_early = P.ws.b_early;
    return Q;
}

// D[rows x width_out] = A[rows x k] * B[width_out x k]^T, both operands contraction-major.
bool add_rowmajor_problem(TcParams& P, const __nv_bfloat16* A, int rows, int k, const __nv_bfloat16* B, int width_out, int max_bn = kMaxBN) {
    const int i = P.count;
    TcProblem& p = P.p[i];
    memset(&p, 0, sizeof p);
    p.bn = std::min(max_bn, pick_bn(width_out));
    p.m_extent = rows; p.n_extent = width_out;
    p.m_tiles = (rows + BLOCK_M - 1) / BLOCK_M;
    p.n_tiles = (width_out + p.bn - 1) / p.bn;
    p.kblocks = k / BLOCK_K; p.splits = 1; p.kb_per_split = p.kblocks;
    if (!make_tmap(&P.tmA[i], A, rows, k, k, BLOCK_K, BLOCK_M)) return false;
    if (!make_tmap(&P.tmB[i], B, width_out, k, k, BLOCK_K, p.bn)) return false;
    P.count++;
    return true;
}

// Binds the CTAs of a forward / data-gradient launch to slabs.  Every slab starts with one CTA; the rest go,
// one at a time, to the slab whose busiest CTA has the most work left (row tiles x cost of a tile), so that
// the slabs finish together.  The cost of a tile is what bounds it: its products or its epilogue.
void plan_ws(TcParams& P, int num_sms, int mode) {
    WsPlan& W = P.ws;
    memset(&W, 0, sizeof W);
    W.num_sms = num_sms; W.mode = mode;
    const uint32_t kWsOperandBytes = ws_operand_bytes(mode);
    struct Cost { int m_tiles; double tile; };
    Cost cost[kMaxSlabs];
    for (int i = 0; i < P.count; ++i) {
        const TcProblem& p = P.p[i];
        for (int nt = 0; nt < p.n_tiles && W.nslabs < kMaxSlabs; ++nt) {
            WsSlab& S = W.slab[W.nslabs];
            S.prob = i; S.n0 = nt * p.bn;
            const uint32_t b_bytes = (uint32_t)p.kblocks * (uint32_t)p.bn * 128u;
            S.resident = b_bytes + 3u * kStageA <= kWsOperandBytes ? 1 : 0;
            const uint32_t per_stage = S.resident ? kStageA : kStageA + (uint32_t)p.bn * 128u;
            S.stages = (int)std::min<uint32_t>(kWsMaxStages, (kWsOperandBytes - (S.resident ? b_bytes : 0u)) / per_stage);
            const double mma = 512.0 * p.kblocks * p.bn / 256.0, epi = 2800.0 * p.bn / 256.0;
            cost[W.nslabs] = Cost{p.m_tiles, std::max(mma, epi) + 300.0};
            W.nslabs++;
        }
    }
    if (W.nslabs == 0) { W.grid = 0; return; }
    int alloc[kMaxSlabs];
    int used = 0;
    for (int i = 0; i < W.nslabs; ++i) { alloc[i] = 1; used++; }
    const int max_ctas = std::min(num_sms, kMaxCtas);
    auto load = [&](int i) { return ((cost[i].m_tiles + alloc[i] - 1) / alloc[i]) * cost[i].tile; };
    while (used < max_ctas) {
        int best = -1;
        for (int i = 0; i < W.nslabs; ++i)
            if (alloc[i] < cost[i].m_tiles && (best < 0 || load(i) > load(best))) best = i;
        if (best < 0) break;
        alloc[best]++; used++;
    }
    int cta = 0;
    for (int i = 0; i < W.nslabs; ++i) {
        W.slab[i].cta_begin = cta; W.slab[i].cta_count = alloc[i];
        for (int k = 0; k < alloc[i]; ++k) W.cta_slab[cta++] = (unsigned char)i;
    }
    W.grid = cta;
}

template <int MODE>
cudaError_t launch_ws(const TcParams& P, cudaStream_t s) {
    if (P.total_items == 0 || P.ws.grid == 0) return cudaSuccess;
    LaunchScope scope_(MODE == TC_FWD ? "tc_gemm_fwd" : "tc_gemm_dgrad", s);
    return launch_chained(ws_gemm_kernel<MODE>, P.ws.grid, kThreads, kWsSmem, s, P);
}

cudaError_t launch_wgrad(const TcParams& P, int num_sms, cudaStream_t s) {
    if (P.total_items == 0) return cudaSuccess;
    const int grid = std::min(P.total_items, num_sms);
    LaunchScope scope_("tc_gemm_wgrad", s);
    return launch_chained(wgrad_gemm_kernel, grid, kThreads, kWgradSmem, s, P);
}



// The program of one net for the fused forward; false when the widths do not fit the kernel
// (first hidden layer <= 512 and a multiple of 128 beyond 256, the others <= 256).
// head_n > 0: a head job of that many output columns (a multiple of 16, at most 64) follows the last layer.
bool compile_chain(ChainNet& N, int nh, const int* pw, int kp, int* bn_of_layer, int head_n) {
    memset(&N, 0, sizeof N);
    if (head_n > 0 && nh == 1 && pw[0] > 256) return false;
    if (nh < 1 || nh > kChainLayers || pw[0] > 512 || (pw[0] > 256 && pw[0] % 128 != 0)) return false;
    for (int l = 1; l < nh; ++l)
        if (pw[l] > 256) return false;
    int nj = 0, ne = 0;
    auto job = [&](int layer, int n0, int bn, int kb0, int nkb, int a_ring, int tmem_col, int accumulate, int wait_epi) {
        N.job[nj] = ChainJob{layer, n0, bn, kb0, nkb, a_ring, tmem_col, accumulate, wait_epi};
        return nj++;
    };
    int last_col = 0;                  // accumulator half of the most recent epilogue
    auto epi = [&](int layer, int n0, int ncols, int tmem_col, int wait_job, int write_job) {
        N.epi[ne] = ChainEpi{0, layer, n0, ncols, tmem_col, wait_job, write_job};
        last_col = tmem_col;
        return ne++;
    };
    const int kb_in = kp / BLOCK_K;
    for (int l = 0; l < nh; ++l) bn_of_layer[l] = pw[l];
    if (pw[0] <= 256 || nh < 2) {
        if (pw[0] > 256) {
            // a single wide layer: two independent halves, each waiting for its own accumulator to be drained
            const int half = pw[0] / 2;
            bn_of_layer[0] = half;
            const int j0 = job(0, 0, half, 0, kb_in, 1, 0, 0, kPrevItem + 0);
            const int j1 = job(0, half, half, 0, kb_in, 1, 256, 0, kPrevItem + 1);
            epi(0, 0, half, 0, j0, -1);
            epi(0, half, half, 256, j1, -1);
        } else if (nh == 1) {
            const int j0 = job(0, 0, pw[0], 0, kb_in, 1, 0, 0, kPrevItem + 0);
            epi(0, 0, pw[0], 0, j0, -1);
        } else {
            // plain chain: the accumulators alternate between the halves of tensor memory, and a job waits
            // for the epilogue of the layer before.  The half the first job of an item overwrites was
            // drained by an epilogue that a later job of the item before already waited for; with an odd
            // number of layers that holds because the halves swap from item to item.
            int prev_e = -1;
            for (int l = 0; l < nh; ++l) {
                const int col = (l & 1) ? 256 : 0;
                const int j = l == 0 ? job(0, 0, pw[0], 0, kb_in, 1, col, 0, -1)
                                     : job(l, 0, pw[l], 0, pw[l - 1] / BLOCK_K, 0, col, 0, prev_e);
                prev_e = epi(l, 0, pw[l], col, j, -1);
            }
            N.flip = (nh & 1) ? 1 : 0;
        }
    } else {
        // wide first layer: both halves up front, the second layer accumulates over them
        const int half = pw[0] / 2, hk = half / BLOCK_K;
        bn_of_layer[0] = half;
        const int last_e = nh;                                    // index of the item's last epilogue (nh + 1 epilogues)
        const bool last_in_256 = ((nh - 2) & 1) != 0;             // layers 2.. alternate 256, 0, 256, ...
        const int j0 = job(0, 0, half, 0, kb_in, 1, 0, 0, last_in_256 ? -1 : kPrevItem + last_e);
        const int j1 = job(0, half, half, 0, kb_in, 1, 256, 0, last_in_256 ? kPrevItem + last_e : -1);
        const int e0 = epi(0, 0, half, 0, j0, -1);
        const int j2 = job(1, 0, pw[1], 0, hk, 0, 0, 0, e0);
        const int e1 = epi(0, half, half, 256, j1, j2);
        const int j3 = job(1, 0, pw[1], hk, hk, 0, 0, 1, e1);
        int prev_e = epi(1, 0, pw[1], 0, j3, -1);
        for (int l = 2; l < nh; ++l) {
            const int col = (l & 1) ? 0 : 256;
            const int j = job(l, 0, pw[l], 0, pw[l - 1] / BLOCK_K, 0, col, 0, prev_e);
            prev_e = epi(l, 0, pw[l], col, j, -1);
        }
    }
    if (head_n > 0) {
        if (nj == kChainJobs || ne == kChainEpis) return false;
        // the head reads the last activations from the buffer and accumulates in the half the last layer left free
        const int last_e = ne - 1;
        const int jh = job(nh, 0, 2 * head_n, 0, pw[nh - 1] / BLOCK_K, 0, last_col ^ 256, 0, last_e);
        N.epi[ne] = ChainEpi{1, nh - 1, 0, 2 * head_n, last_col ^ 256, jh, -1};
        N.head_n = head_n;
        const int eh = ne++;
        // an item starts once the head epilogue of the item before is done: every accumulator is drained by then
        N.flip = 0;
        for (int j = 0; j < nj; ++j)
            if (N.job[j].wait_epi < 0 || N.job[j].wait_epi >= kPrevItem) N.job[j].wait_epi = j == 0 ? kPrevItem + eh : -1;
    }
    N.nlayers = nh; N.njobs = nj; N.nepis = ne;
    return nj <= kChainJobs && ne <= kChainEpis;
}

cudaError_t launch_chain(const ChainParams& P, int num_sms, cudaStream_t s) {
    if (P.total_items == 0) return cudaSuccess;
    const int grid = std::min(P.total_items, num_sms);
    LaunchScope scope_("tc_mlp_fwd", s);
    return launch_chained(chain_fwd_kernel, grid, kThreads, kChainSmem, s, P);
}

}  // namespace

// Splits of the contraction (the minibatch rows) for every weight-gradient problem, chosen so that
// the work items (tile x split) fill the SMs once with items of about equal cost: starting from one
// split each, the problem with the most expensive item gets another split while the items still fit.
// The cost of an item is the bytes it streams, (128 + columns) per contraction row.
WgradPlan umma_wgrad_plan(const UmmaSetup& s) {
    WgradPlan plan{};
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int kblocks = (s.R + BLOCK_K - 1) / BLOCK_K;
    struct Prob { int ni, l, tiles, unit, splits; };
    std::vector<Prob> probs;
    int items = 0;
    for (int ni = 0; ni < 2; ++ni) {
        const int nh = s.nl[ni] - 1;
        for (int l = 0; l <= nh; ++l) {
            const int wa = round_up(l == 0 ? s.in_dim[ni] : s.out[ni][l - 1], 64);
            const int wb = l == nh ? 64 : round_up(s.out[ni][l], 64);
            const int bn = pick_bn(wb);
            Prob q{ni, l, ((wa + BLOCK_M - 1) / BLOCK_M) * ((wb + bn - 1) / bn), BLOCK_M + bn, 1};
            probs.push_back(q);
            items += q.tiles;
        }
    }
    const int max_splits = std::max(1, std::min(32, kblocks));
    auto item_cost = [&](const Prob& q) { return (long long)q.unit * ((kblocks + q.splits - 1) / q.splits); };
    while (true) {
        int best = -1;
        for (int i = 0; i < (int)probs.size(); ++i) {
            const Prob& q = probs[i];
            if (q.splits >= max_splits || items + q.tiles > sms) continue;
            if (best < 0 || item_cost(q) > item_cost(probs[best])) best = i;
        }
        if (best < 0) break;
        // stop when the most expensive item overall can no longer be split: more splits elsewhere gain nothing
        bool is_max = true;
        for (const Prob& q : probs) if (item_cost(q) > item_cost(probs[best])) is_max = false;
        if (!is_max) break;
        probs[best].splits++;
        items += probs[best].tiles;
    }
    plan.max_splits = 1;
    for (const Prob& q : probs) { plan.splits[q.ni][q.l] = q.splits; plan.max_splits = std::max(plan.max_splits, q.splits); }
    return plan;
}

UmmaEngine* umma_create(const UmmaSetup& s, std::string* err) {
    auto failmsg = [&](const char* m) { if (err) *err = m; return (UmmaEngine*)nullptr; };
    if (s.model.precision != RSLRL_BF16) return failmsg("only the BF16 tensor-core mode is available");
    if (!get_encode_fn()) return failmsg("cuTensorMapEncodeTiled is not available from the driver");
    int dev = 0; cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return failmsg("no CUDA device");
    if (prop.major != 10) return failmsg("the tensor-core mode needs an sm_100 device");
    if (cudaFuncSetAttribute(wgrad_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWgradSmem) != cudaSuccess)
        return failmsg("could not reserve shared memory for the tensor-core kernels");
    if (cudaFuncSetAttribute(ws_gemm_kernel<TC_FWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWsSmem) != cudaSuccess ||
        cudaFuncSetAttribute(ws_gemm_kernel<TC_DGRAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWsSmem) != cudaSuccess)
        return failmsg("could not reserve shared memory for the tensor-core kernels");
    if (cudaFuncSetAttribute(chain_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kChainSmem) != cudaSuccess)
        return failmsg("could not reserve shared memory for the fused forward kernel");
    UmmaEngine* e = new UmmaEngine();
    e->s = s;
    e->num_sms = prop.multiProcessorCount;
    auto bail = [&](const char* m) { if (err) *err = m; umma_destroy(e); return (UmmaEngine*)nullptr; };
    const int N = s.N, R = s.R;
    if (!ealloc(e, &e->error_dev, 1)) return bail("allocation failed");
    for (int ni = 0; ni < 2; ++ni) {
        e->nh[ni] = s.nl[ni] - 1;
        e->kp[ni] = round_up(s.in_dim[ni], 64);
        for (int l = 0; l < e->nh[ni]; ++l) e->pw[ni][l] = round_up(s.out[ni][l], 64);
        // a launch holds both nets' column blocks of one layer (128 columns each in the data gradient)
        for (int l = 0; l < e->nh[ni]; ++l)
            if (2 * ((e->pw[ni][l] + 127) / 128) > kMaxSlabs) return bail("hidden layers wider than 4096 are not supported in the BF16 mode");
    }
    const bool shared = s.model.shared_obs != 0;
    for (int ni = 0; ni < 2; ++ni) {
        if (ni == 1 && shared) { e->obs16_act[1] = e->obs16_act[0]; e->x16[1] = e->x16[0]; e->x16_alt[1] = e->x16_alt[0]; }
        else {
            if (!ealloc(e, &e->obs16_act[ni], (size_t)N * e->kp[ni])) return bail("allocation failed");
            if (!ealloc(e, &e->x16[ni], (size_t)R * e->kp[ni]) || !ealloc(e, &e->x16_alt[ni], (size_t)R * e->kp[ni]))
                return bail("allocation failed");
        }
        for (int l = 0; l < e->nh[ni]; ++l) {
            const int kin = l == 0 ? e->kp[ni] : e->pw[ni][l - 1];
            if (!ealloc(e, &e->h_act[ni][l], (size_t)N * e->pw[ni][l]) || !ealloc(e, &e->h[ni][l], (size_t)R * e->pw[ni][l]) ||
                !ealloc(e, &e->dz[ni][l], (size_t)R * e->pw[ni][l]) || !ealloc(e, &e->wt[ni][l], (size_t)e->pw[ni][l] * kin) ||
                !ealloc(e, &e->bias_pad[ni][l], (size_t)e->pw[ni][l]))
                return bail("allocation failed");
            if (l > 0 && !ealloc(e, &e->wn[ni][l], (size_t)e->pw[ni][l - 1] * e->pw[ni][l])) return bail("allocation failed");
        }
    }
    if (!ealloc(e, &e->dmu16, (size_t)R * 64) || !ealloc(e, &e->dv16, (size_t)R * 64)) return bail("allocation failed");
    // head weights as tensor-core operands (output-major and input-major, padded to 64 outputs)
    for (int ni = 0; ni < 2; ++ni) {
        const int pl = e->pw[ni][e->nh[ni] - 1];
        e->head_n[ni] = ((ni == 0 ? s.out[0][e->nh[0]] : 1) + 15) / 16 * 16;
        if (!ealloc(e, &e->wht[ni], (size_t)128 * pl) || !ealloc(e, &e->whn[ni], (size_t)pl * 64) ||
            !ealloc(e, &e->head_bias_pad[ni], (size_t)64))
            return bail("allocation failed");
    }

    // weight conversion table
    std::vector<CvtEntry> table;
    for (int ni = 0; ni < 2; ++ni)
        for (int l = 0; l < e->nh[ni]; ++l) {
            CvtEntry c{};
            c.bsrc = s.param + s.b_off[ni][l]; c.bdst = e->bias_pad[ni][l];
            c.src = s.param + s.w_off[ni][l]; c.in = s.in[ni][l]; c.out = s.out[ni][l]; c.ld_src = s.out_p[ni][l];
            c.wt = e->wt[ni][l]; c.ld_wt = l == 0 ? e->kp[ni] : e->pw[ni][l - 1];
            c.wn = l > 0 ? e->wn[ni][l] : nullptr; c.ld_wn = e->pw[ni][l];
            table.push_back(c);
            e->cvt_max = std::max(e->cvt_max, c.in * c.out);
        }
    for (int ni = 0; ni < 2; ++ni) {
        const int l = e->nh[ni];                       // the head
        if (s.out[ni][l] > 64) continue;
        CvtEntry c{};
        c.bsrc = s.param + s.b_off[ni][l]; c.bdst = e->head_bias_pad[ni];
        c.src = s.param + s.w_off[ni][l]; c.in = s.in[ni][l]; c.out = s.out[ni][l]; c.ld_src = s.out_p[ni][l];
        c.wt = e->wht[ni]; c.ld_wt = e->pw[ni][l - 1];
        c.wn = e->whn[ni]; c.ld_wn = 64;
        c.wt_lo = e->wht[ni] + (size_t)e->head_n[ni] * c.ld_wt;
        table.push_back(c);
        e->cvt_max = std::max(e->cvt_max, c.in * c.out);
    }
    e->n_cvt = (int)table.size();
    e->head_copies = e->n_cvt <= kMaxCvt && s.out[0][e->nh[0]] <= 64;
    if (!ealloc(e, &e->cvt_dev, table.size())) return bail("allocation failed");
    if (cudaMemcpyAsync(e->cvt_dev, table.data(), table.size() * sizeof(CvtEntry), cudaMemcpyHostToDevice, s.stream) != cudaSuccess ||
        cudaStreamSynchronize(s.stream) != cudaSuccess)
        return bail("copy of the conversion table failed");

    const float alpha = s.model.elu_alpha;
    const int maxh = std::max(e->nh[0], e->nh[1]);
    // ---- forward launches (act rows and update rows), one per hidden layer index -----------
    auto build_fwd = [&](std::vector<TcParams>& out, int rows, bool actor, bool critic, bool act_buffers) -> bool {
        for (int l = 0; l < maxh; ++l) {
            TcParams P; memset(&P, 0, sizeof P);
            for (int ni = 0; ni < 2; ++ni) {
                if ((ni == 0 && !actor) || (ni == 1 && !critic) || l >= e->nh[ni]) continue;
                const __nv_bfloat16* in = l == 0 ? (act_buffers ? e->obs16_act[ni] : e->x16[ni])
                                                 : (act_buffers ? e->h_act[ni][l - 1] : e->h[ni][l - 1]);
                const int k = l == 0 ? e->kp[ni] : e->pw[ni][l - 1];
                if (!add_rowmajor_problem(P, in, rows, k, e->wt[ni][l], e->pw[ni][l])) return false;
                TcProblem& p = P.p[P.count - 1];
                p.bias = e->bias_pad[ni][l]; p.bias_n = e->pw[ni][l];
                p.net_id = ni; p.layer_id = l;
                p.out16 = act_buffers ? e->h_act[ni][l] : e->h[ni][l]; p.ld_out = e->pw[ni][l];
                if (!make_tmap(&P.tmOut[P.count - 1], p.out16, rows, e->pw[ni][l], e->pw[ni][l], 32, 32, CU_TENSOR_MAP_SWIZZLE_64B)) return false;
            }
            finish_params(P, alpha, e->error_dev);
            plan_ws(P, e->num_sms, TC_FWD);
            // the launch before the first layer's may be the optimiser step that rewrites the weights; the other
            // layers follow a forward launch
            P.ws.b_early = l > 0 ? 1 : 0;
            out.push_back(P);
        }
        return true;
    };
    if (!build_fwd(e->act_fwd, N, true, true, true) || !build_fwd(e->act_fwd_critic, N, false, true, true) ||
        !build_fwd(e->upd_fwd, R, true, true, false))
        return bail("tensor map encoding failed");
    // ---- fused forward: every hidden layer of both nets in one launch ------------------------
    auto build_chain = [&](std::vector<ChainParams>& out, int rows, bool actor, bool critic, bool act_buffers) -> bool {
        ChainParams P; memset(&P, 0, sizeof P);
        int bias_floats = 0;
        for (int ni = 0; ni < 2; ++ni) {
            if ((ni == 0 && !actor) || (ni == 1 && !critic)) continue;
            const int n = P.nnets;
            int bn[kChainLayers] = {};
            const int n_out = ni == 0 ? s.out[0][e->nh[0]] : 1;
            const int head_n = e->head_copies ? e->head_n[ni] : 0;
            if (e->nh[ni] > kChainLayers || !compile_chain(P.net[n], e->nh[ni], e->pw[ni], e->kp[ni], bn, head_n)) return true;   // not applicable
            if (head_n > 0) {
                const int pl = e->pw[ni][e->nh[ni] - 1];
                if (!make_tmap(&P.tmW[n][e->nh[ni]], e->wht[ni], 128, pl, pl, BLOCK_K, 2 * head_n)) return false;
                P.net[n].is_actor = ni == 0; P.net[n].A = n_out; P.net[n].head_bias = e->head_bias_pad[ni];
            }
            if (!make_tmap(&P.tmX[n], act_buffers ? e->obs16_act[ni] : e->x16[ni], rows, e->kp[ni], e->kp[ni], BLOCK_K, BLOCK_M)) return false;
            for (int l = 0; l < e->nh[ni]; ++l) {
                const int kin = l == 0 ? e->kp[ni] : e->pw[ni][l - 1];
                __nv_bfloat16* o = act_buffers ? e->h_act[ni][l] : e->h[ni][l];
                if (!make_tmap(&P.tmW[n][l], e->wt[ni][l], e->pw[ni][l], kin, kin, BLOCK_K, bn[l]) ||
                    !make_tmap(&P.tmOut[n][l], o, rows, e->pw[ni][l], e->pw[ni][l], 64, 32))
                    return false;
                P.net[n].bias[l] = e->bias_pad[ni][l];
                P.net[n].bias_n[l] = e->pw[ni][l];
                P.net[n].bias_off[l] = bias_floats;
                bias_floats += e->pw[ni][l];
            }
            P.nnets++;
        }
        if (P.nnets == 2) {
            // items of both nets alternate in a CTA and wait for each other's epilogues by index
            const ChainNet &a = P.net[0], &b = P.net[1];
            bool same = a.njobs == b.njobs && a.nepis == b.nepis && a.flip == b.flip;
            for (int j = 0; same && j < a.njobs; ++j) same = a.job[j].wait_epi == b.job[j].wait_epi && a.job[j].tmem_col == b.job[j].tmem_col;
            for (int k = 0; same && k < a.nepis; ++k)
                same = a.epi[k].wait_job == b.epi[k].wait_job && a.epi[k].write_job == b.epi[k].write_job && a.epi[k].tmem_col == b.epi[k].tmem_col;
            if (!same) return true;   // not applicable
        }
        P.rows = rows;
        P.total_items = P.nnets * ((rows + BLOCK_M - 1) / BLOCK_M);
        // with the heads inside the kernel nothing reads the hidden activations of a rollout step afterwards
        P.store = 0;
        for (int n = 0; n < P.nnets; ++n) if (P.net[n].head_n == 0) P.store = 1;
        P.alpha = alpha; P.error = e->error_dev;
        out.push_back(P);
        return true;
    };
    // (the rollout's few row tiles gain from the single launch; on the many tiles of a minibatch the
    // per-layer launches, whose epilogues overlap the next tile's MMAs, measured slightly faster)
    if (!build_chain(e->chain_act, N, true, true, true) || !build_chain(e->chain_act_critic, N, false, true, true))
        return bail("tensor map encoding failed");
    // ---- data-gradient launches: step b produces dZ of hidden layer nh-2-b -------------------
    for (int b = 0; b + 1 < maxh; ++b) {
        TcParams P; memset(&P, 0, sizeof P);
        for (int ni = 0; ni < 2; ++ni) {
            const int l = e->nh[ni] - 1 - b;
            if (l < 1) continue;
            // slabs of 128 columns: every epilogue warp then has one 32-column chunk per row tile, whose stored
            // post-activations it fetches while the products still run
            if (!add_rowmajor_problem(P, e->dz[ni][l], R, e->pw[ni][l], e->wn[ni][l], e->pw[ni][l - 1], 128))
                return bail("tensor map encoding failed");
            TcProblem& p = P.p[P.count - 1];
            p.out16 = e->dz[ni][l - 1]; p.ld_out = e->pw[ni][l - 1];
            p.aux16 = e->h[ni][l - 1]; p.ld_aux = e->pw[ni][l - 1];
            p.net_id = ni; p.layer_id = l - 1;
            if (e->n_sources < kMaxBiasSources) {     // beyond that the column-sum kernel takes the layer
                e->n_sources++;
                e->n_slots = 4 * p.m_tiles;
                if (!ealloc(e, &e->bias_slots[ni][l - 1], (size_t)e->n_slots * e->pw[ni][l - 1])) return bail("allocation failed");
                p.colsum = e->bias_slots[ni][l - 1]; p.ld_colsum = e->pw[ni][l - 1];
            }
            if (!make_tmap(&P.tmOut[P.count - 1], p.out16, R, e->pw[ni][l - 1], e->pw[ni][l - 1], 32, 32, CU_TENSOR_MAP_SWIZZLE_64B) ||
                !make_tmap(&P.tmAux[P.count - 1], p.aux16, R, e->pw[ni][l - 1], e->pw[ni][l - 1], 32, BLOCK_M, CU_TENSOR_MAP_SWIZZLE_64B))
                return bail("tensor map encoding failed");
        }
        finish_params(P, alpha, e->error_dev);
        plan_ws(P, e->num_sms, TC_DGRAD);
        P.ws.b_early = 1;                  // data-gradient launches follow the head/loss kernel or each other
        e->upd_dgrad.push_back(P);
    }
    // ---- weight-gradient problems (all layers of both nets, heads included) ------------------
    {
        const int kblocks = (R + BLOCK_K - 1) / BLOCK_K;
        const WgradPlan plan = umma_wgrad_plan(s);
        TcParams P; memset(&P, 0, sizeof P);
        auto flush = [&]() { if (P.count) { finish_params(P, alpha, e->error_dev); e->upd_wgrad.push_back(P); memset(&P, 0, sizeof P); } };
        for (int ni = 0; ni < 2; ++ni)
            for (int l = 0; l <= e->nh[ni]; ++l) {
                const bool head = l == e->nh[ni];
                const __nv_bfloat16* A = l == 0 ? e->x16[ni] : e->h[ni][l - 1];
                const int wa = l == 0 ? e->kp[ni] : e->pw[ni][l - 1];
                const __nv_bfloat16* B = head ? (ni == 0 ? e->dmu16 : e->dv16) : e->dz[ni][l];
                const int wb = head ? 64 : e->pw[ni][l];
                if (P.count == kMaxProblems) flush();
                const int i = P.count;
                TcProblem& p = P.p[i];
                p.bn = pick_bn(wb);
                p.m_extent = s.in[ni][l]; p.n_extent = s.out_p[ni][l];
                p.m_tiles = (wa + BLOCK_M - 1) / BLOCK_M; p.n_tiles = (wb + p.bn - 1) / p.bn;
                const int want = std::min(plan.splits[ni][l], s.splits);      // s.splits rows of partials exist
                p.kb_per_split = (kblocks + want - 1) / want;
                p.kblocks = kblocks; p.splits = (kblocks + p.kb_per_split - 1) / p.kb_per_split;
                p.out32 = s.partials + s.w_off[ni][l]; p.ld_out32 = s.out_p[ni][l]; p.split_stride = s.P_dev;
                p.net_id = ni; p.layer_id = l;
                if (!make_tmap(&P.tmA[i], A, R, wa, wa, 64, BLOCK_K) || !make_tmap(&P.tmB[i], B, R, wb, wb, 64, BLOCK_K))
                    return bail("tensor map encoding failed");
                P.count++;
            }
        flush();
    }
    // ---- the same launches reading the second minibatch input buffer ----------------------------
    e->upd_fwd_alt = e->upd_fwd; e->upd_wgrad_alt = e->upd_wgrad;
    for (size_t li = 0; li < e->upd_fwd_alt.size(); ++li) {
        TcParams& P = e->upd_fwd_alt[li];
        for (int i = 0; i < P.count; ++i) {
            if (P.p[i].layer_id != 0) continue;
            const int ni = P.p[i].net_id;
            if (!make_tmap(&P.tmA[i], e->x16_alt[ni], R, e->kp[ni], e->kp[ni], BLOCK_K, BLOCK_M)) return bail("tensor map encoding failed");
        }
    }
    for (TcParams& P : e->upd_wgrad_alt)
        for (int i = 0; i < P.count; ++i) {
            if (P.p[i].layer_id != 0) continue;
            const int ni = P.p[i].net_id;
            if (!make_tmap(&P.tmA[i], e->x16_alt[ni], R, e->kp[ni], e->kp[ni], 64, BLOCK_K)) return bail("tensor map encoding failed");
        }
    for (const TcParams& P : e->upd_fwd) e->fwd_actor[0].push_back(only_net(P, 0));
    for (const TcParams& P : e->upd_fwd_alt) e->fwd_actor[1].push_back(only_net(P, 0));
    for (const TcParams& P : e->upd_dgrad) e->dgrad_actor.push_back(only_net(P, 0));
    // ---- bias-gradient partials of the last hidden layers, written by the head/loss kernel ----
    if (e->n_sources + 2 <= kMaxBiasSources)
        for (int ni = 0; ni < 2; ++ni)
            if (!ealloc(e, &e->head_slots[ni], (size_t)head_loss_blocks(s.Bmb) * e->pw[ni][e->nh[ni] - 1])) return bail("allocation failed");
    // ---- bias gradients of the hidden layers: column sums of dZ -------------------------------
    e->colsum.count = 0; e->colsum.splits = s.splits; e->colsum.split_stride = s.P_dev; e->colsum.is_bf16 = 1;
    // (only of the last one of each net: the others come from the data-gradient epilogue)
    for (int ni = 0; ni < 2; ++ni)
        for (int l = 0; l < e->nh[ni]; ++l) {
            if (e->bias_slots[ni][l]) continue;
            if (e->colsum.count == kMaxColsum) return bail("too many layers for the bias-gradient launch");
            ColsumProblem& q = e->colsum.p[e->colsum.count++];
            q.X = e->dz[ni][l]; q.out = s.partials + s.b_off[ni][l]; q.rows = R; q.n = s.out[ni][l]; q.ld = e->pw[ni][l];
            if (l < e->nh[ni] - 1) e->colsum_rest.p[e->colsum_rest.count++] = q;
        }
    e->colsum_rest.splits = e->colsum.splits; e->colsum_rest.split_stride = e->colsum.split_stride; e->colsum_rest.is_bf16 = 1;
    if (cudaStreamSynchronize(s.stream) != cudaSuccess) return bail("stream synchronisation failed");
    return e;
}

void umma_destroy(UmmaEngine* e) {
    if (!e) return;
    for (void* p : e->allocs) guarded_free(p);
    delete e;
}

void umma_fill_cvt(UmmaEngine* e, AdamArgs* a) {
    const UmmaSetup& s = e->s;
    a->n_cvt = 0;
    for (int ni = 0; ni < 2; ++ni)
        for (int l = 0; l < e->nh[ni] && a->n_cvt < kMaxCvt; ++l) {
            CvtRange& c = a->cvt[a->n_cvt++];
            c.w_off = (int)s.w_off[ni][l]; c.b_off = (int)s.b_off[ni][l];
            c.in = s.in[ni][l]; c.out = s.out[ni][l]; c.out_p = s.out_p[ni][l];
            c.wt = e->wt[ni][l]; c.ld_wt = l == 0 ? e->kp[ni] : e->pw[ni][l - 1];
            c.wn = l > 0 ? e->wn[ni][l] : nullptr; c.ld_wn = e->pw[ni][l];
            c.wt_lo = nullptr;
            c.bias_pad = e->bias_pad[ni][l];
        }
    for (int ni = 0; ni < 2 && e->head_copies; ++ni) {
        if (a->n_cvt == kMaxCvt) break;
        const int l = e->nh[ni];
        CvtRange& c = a->cvt[a->n_cvt++];
        c.w_off = (int)s.w_off[ni][l]; c.b_off = (int)s.b_off[ni][l];
        c.in = s.in[ni][l]; c.out = s.out[ni][l]; c.out_p = s.out_p[ni][l];
        c.wt = e->wht[ni]; c.ld_wt = e->pw[ni][l - 1];
        c.wn = e->whn[ni]; c.ld_wn = 64;
        c.wt_lo = e->wht[ni] + (size_t)e->head_n[ni] * c.ld_wt;
        c.bias_pad = e->head_bias_pad[ni];
    }
}

void umma_fill_bias_sources(UmmaEngine* e, ReduceArgs* r, const HeadLossArgs& hl) {
    const UmmaSetup& s = e->s;
    r->n_bias = 0;
    if (hl.colsum_written)
        for (int ni = 0; ni < 2; ++ni) {
            const int l = e->nh[ni] - 1;
            BiasSource& b = r->bias[r->n_bias++];
            b.p_off = (int)s.b_off[ni][l]; b.n = s.out[ni][l];
            b.slots = e->head_slots[ni]; b.nslots = hl.nblocks_used; b.ld = e->pw[ni][l];
        }
    for (int ni = 0; ni < 2; ++ni)
        for (int l = 0; l < e->nh[ni]; ++l) {
            if (!e->bias_slots[ni][l]) continue;
            BiasSource& b = r->bias[r->n_bias++];
            b.p_off = (int)s.b_off[ni][l]; b.n = s.out[ni][l];
            b.slots = e->bias_slots[ni][l]; b.nslots = e->n_slots; b.ld = e->pw[ni][l];
        }
}

cudaError_t umma_refresh_weights(UmmaEngine* e) {
    dim3 grid(std::max(1, std::min(64, (e->cvt_max + 255) / 256)), e->n_cvt);
    LaunchScope scope_("convert_weights", e->s.stream);
    convert_weights_kernel<<<grid, 256, 0, e->s.stream>>>(e->cvt_dev);
    return cudaGetLastError();
}

cudaError_t umma_act_forward(UmmaEngine* e, const float* d_obs_a, const float* d_obs_c, float* store_a, float* store_c,
                             int sa, int sc, bool do_actor, const ActOut& out, const float* log_std, uint64_t seed,
                             uint32_t global_step, bool* heads_done, const void** ha, int* ldha, const void** hc, int* ldhc) {
    const UmmaSetup& s = e->s;
    cudaError_t err;
    const bool shared = s.model.shared_obs != 0;
    *heads_done = false;
    if (do_actor) {
        err = launch_pad_rows(d_obs_a, s.in_dim[0], store_a, sa, e->obs16_act[0], e->kp[0], s.N, s.stream);
        if (err != cudaSuccess) return err;
        if (!shared) {
            err = launch_pad_rows(d_obs_c, s.in_dim[1], store_c, sc, e->obs16_act[1], e->kp[1], s.N, s.stream);
            if (err != cudaSuccess) return err;
        }
    } else {
        err = launch_pad_rows(d_obs_c, s.in_dim[1], nullptr, 0, e->obs16_act[1], e->kp[1], s.N, s.stream);
        if (err != cudaSuccess) return err;
    }
    std::vector<ChainParams>& fused = do_actor ? e->chain_act : e->chain_act_critic;
    if (!fused.empty()) {
        ChainParams& P = fused[0];
        if (P.net[0].A > 0) {
            // the heads run in the same launch and write the rollout outputs of this step
            P.ho.actions = out.actions; P.ho.mu = out.mu; P.ho.sigma = out.sigma; P.ho.logp = out.logp;
            P.ho.values = out.values; P.ho.actions_out = out.actions_out; P.ho.act_stride = out.act_stride;
            P.ho.log_std = log_std;
            P.ho.seed_lo = (uint32_t)seed; P.ho.seed_hi = (uint32_t)(seed >> 32); P.ho.global_step = global_step;
            *heads_done = true;
        }
        err = launch_chain(P, e->num_sms, s.stream);
        if (err != cudaSuccess) return err;
    } else {
        const std::vector<TcParams>& seq = do_actor ? e->act_fwd : e->act_fwd_critic;
        for (const TcParams& P : seq) {
            err = launch_ws<TC_FWD>(P, s.stream);
            if (err != cudaSuccess) return err;
        }
    }
    *ha = e->h_act[0][e->nh[0] - 1]; *ldha = e->pw[0][e->nh[0] - 1];
    *hc = e->h_act[1][e->nh[1] - 1]; *ldhc = e->pw[1][e->nh[1] - 1];
    return cudaSuccess;
}

void umma_gather_targets(UmmaEngine* e, GatherArgs* g, int buf) {
    g->x_a = nullptr; g->x_c = nullptr;
    g->x_a16 = buf ? e->x16_alt[0] : e->x16[0]; g->ldxa16 = e->kp[0];
    g->x_c16 = buf ? e->x16_alt[1] : e->x16[1]; g->ldxc16 = e->kp[1];
}

cudaError_t umma_update_forward(UmmaEngine* e, int buf, bool actor_only) {
    FamilyScope family_("tc_gemm_fwd", e->s.stream);
    for (const TcParams& P : actor_only ? e->fwd_actor[buf] : buf ? e->upd_fwd_alt : e->upd_fwd) {
        cudaError_t err = launch_ws<TC_FWD>(P, e->s.stream);
        if (err != cudaSuccess) return err;
    }
    return cudaSuccess;
}

void umma_head_loss_targets(UmmaEngine* e, HeadLossArgs* a) {
    a->Ha = e->h[0][e->nh[0] - 1]; a->ldha = e->pw[0][e->nh[0] - 1];
    a->Hc = e->h[1][e->nh[1] - 1]; a->ldhc = e->pw[1][e->nh[1] - 1];
    a->bf16_act = 1;
    a->dZa = e->dz[0][e->nh[0] - 1]; a->lddza = a->ldha;
    a->dZc = e->dz[1][e->nh[1] - 1]; a->lddzc = a->ldhc;
    a->dmu16 = e->dmu16; a->lddmu16 = 64; a->dv16 = e->dv16; a->lddv16 = 64;
    a->colsum_a = e->head_slots[0]; a->colsum_c = e->head_slots[1];
}

cudaError_t umma_zero_critic_gradients(UmmaEngine* e) {
    // what the critic's data-gradient launches would write: dL/dz of its hidden layers below the last one
    // (the head/loss kernel writes the last) and the bias-gradient partials of their epilogues
    const int R = e->s.R;
    for (int l = 0; l + 1 < e->nh[1]; ++l) {
        cudaError_t err = cudaMemsetAsync(e->dz[1][l], 0, (size_t)R * e->pw[1][l] * sizeof(__nv_bfloat16), e->s.stream);
        if (err != cudaSuccess) return err;
        if (e->bias_slots[1][l]) {
            err = cudaMemsetAsync(e->bias_slots[1][l], 0, (size_t)e->n_slots * e->pw[1][l] * sizeof(float), e->s.stream);
            if (err != cudaSuccess) return err;
        }
    }
    return cudaSuccess;
}

cudaError_t umma_update_backward(UmmaEngine* e, bool last_bias_done, int buf, bool actor_only) {
    cudaError_t err;
    {
        FamilyScope family_("tc_gemm_dgrad", e->s.stream);
        for (const TcParams& P : actor_only ? e->dgrad_actor : e->upd_dgrad) {
            err = launch_ws<TC_DGRAD>(P, e->s.stream);
            if (err != cudaSuccess) return err;
        }
    }
    for (const TcParams& P : buf ? e->upd_wgrad_alt : e->upd_wgrad) {
        err = launch_wgrad(P, e->num_sms, e->s.stream);
        if (err != cudaSuccess) return err;
    }
    return launch_colsum(last_bias_done ? e->colsum_rest : e->colsum, e->s.stream);
}

cudaError_t umma_read_error(UmmaEngine* e, int* host_code) {
    cudaError_t err = cudaMemcpyAsync(host_code, e->error_dev, sizeof(int), cudaMemcpyDeviceToHost, e->s.stream);
    if (err != cudaSuccess) return err;
    err = cudaStreamSynchronize(e->s.stream);
    if (err != cudaSuccess || *host_code == 0) return err;
    // reported once: the word is cleared so that later calls are judged on their own
    return cudaMemsetAsync(e->error_dev, 0, sizeof(int), e->s.stream);
}

}  // namespace rslrl
