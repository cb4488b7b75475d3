// RSLRL_TF32: hidden-layer products on tcgen05 kind::tf32 tiles.  Operands are the FP32 buffers of the
// FP32 mode, staged in shared memory by TMA as K-major tiles of 32 floats per 128-byte swizzle row (K and
// N tails are filled with zeros by the copy engine); accumulators are FP32 in tensor memory, two buffers,
// so that the epilogue of a tile overlaps the products of the next.  Epilogues: bias + ELU (forward) or the
// ELU derivative from the stored post-activation (data gradient); FP32 results leave through a 32 x 32 tile
// per epilogue warp and one TMA store.
//
// Warp roles as in the BF16 kernels: warp 0 = TMA producer, warp 1 = MMA issuer and owner of the tensor
// memory, warps 2..17 = epilogue (lane quarter warp & 3, 32-column chunk (warp - 2) / 4 of a tile of up to
// 128 columns).  Every wait is bounded in time; on expiry the CTA raises an error flag, drains its own
// asynchronous work, frees its tensor memory and returns.
#include "guard.h"
#include "tf32.h"
#include "tc_ptx.cuh"

#include <algorithm>
#include <cstring>
#include <vector>

namespace rslrl {

using namespace tc;

namespace {

constexpr int kTfBlockK = 32;                     // floats per 128-byte swizzle row
constexpr int kTfMaxBN = 128;
constexpr int kTfStages = 4;
constexpr uint32_t kTfStageB = kTfMaxBN * 128;    // 16 KiB
constexpr uint32_t kTfTile = 32 * 32 * 4;         // 4 KiB result tile per epilogue warp
constexpr size_t kTfSmem = 1024 + (size_t)kTfStages * (kStageA + kTfStageB) + kEpiWarps * kTfTile + 512;

enum TfMode { TF_FWD = 0, TF_DGRAD = 1, TF_BIAS = 2, TF_PLAIN = 3 };   // epilogue: bias + ELU, ELU' from aux, bias, none

struct TfProblem {
    int m_extent, n_extent;        // rows / columns of D that exist (stores are clipped to them)
    int m_tiles, n_tiles, bn, kblocks;
    int item_begin;
    int row_offset;                // first row of A in its tensor (act reads step t of the rollout storage in place)
    const float* bias;             // forward: readable up to a multiple of 32 columns past n_extent
};

struct TfParams {
    CUtensorMap tmA[2], tmB[2], tmOut[2], tmAux[2];
    TfProblem p[2];
    int count, total_items;
    float alpha;
    int* error;
};

// D[tmem] (+)= A[smem] * B[smem], FP32 words used with TF32 precision
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// Instruction descriptor: TF32 x TF32 -> FP32, both operands K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t instr_desc_tf32(int bn) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(BLOCK_M >> 4) << 24);
}

struct TfItem { int prob, m0, n0; };
__device__ __forceinline__ TfItem tf_decode(const TfParams& P, int item) {
    const int pi = (P.count > 1 && item >= P.p[1].item_begin) ? 1 : 0;
    const TfProblem& p = P.p[pi];
    const int local = item - p.item_begin;
    TfItem it;
    it.prob = pi;
    it.m0 = (local / p.n_tiles) * BLOCK_M;
    it.n0 = (local % p.n_tiles) * p.bn;
    return it;
}

template <int MODE>
__global__ void __launch_bounds__(kThreads, 1) tf32_gemm_kernel(const __grid_constant__ TfParams P) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = smem + kTfStages * kStageA;
    uint8_t* sOut = sB + kTfStages * kTfStageB;
    uint64_t* full = reinterpret_cast<uint64_t*>(sOut + kEpiWarps * kTfTile);
    uint64_t* empty = full + kTfStages;
    uint64_t* tfull = empty + kTfStages;
    uint64_t* tempty = tfull + 2;
    uint64_t* drain = tempty + 2;
    uint64_t* auxbar = drain + 1;                           // one per epilogue warp
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(auxbar + kEpiWarps);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kTfStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&tfull[b], 1); mbar_init(&tempty[b], kEpiWarps); }
        mbar_init(drain, 1);
        for (int w = 0; w < kEpiWarps; ++w) mbar_init(&auxbar[w], 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    if (warp == 0 && lane == 0)
        for (int i = 0; i < P.count; ++i) {
            tma_prefetch_desc(&P.tmA[i]); tma_prefetch_desc(&P.tmB[i]); tma_prefetch_desc(&P.tmOut[i]);
            if (MODE == TF_DGRAD) tma_prefetch_desc(&P.tmAux[i]);
        }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    chain_wait();

    if (warp == 0) {
        // ================================ TMA producer =================================
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            uint32_t issued_mask = 0, issued_parity = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x) {
                const TfItem it = tf_decode(P, item);
                const TfProblem& p = P.p[it.prob];
                const uint32_t bytes = kStageA + (uint32_t)p.bn * 128u;
                for (int kb = 0; kb < p.kblocks; ++kb) {
                    if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag, P.error, 1)) { ok = false; break; }
                    mbar_expect_tx(&full[stage], bytes);
                    tma_load_2d(sA + stage * kStageA, &P.tmA[it.prob], kb * kTfBlockK, p.row_offset + it.m0, &full[stage]);
                    tma_load_2d(sB + stage * kTfStageB, &P.tmB[it.prob], kb * kTfBlockK, it.n0, &full[stage]);
                    issued_mask |= 1u << stage;
                    issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == kTfStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA's shared memory goes away
                for (int s = 0; s < kTfStages; ++s) {
                    if (!(issued_mask & (1u << s))) continue;
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(&full[s], (issued_parity >> s) & 1u) && global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer ===================================
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            int local = 0;
            // descriptors differ only in their address field (16-byte units): one add per stage and k-step
            const uint64_t a_desc0 = smem_desc(smem_u32(sA), 16, 1024);
            const uint64_t b_desc0 = smem_desc(smem_u32(sB), 16, 1024);
            for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++local) {
                const TfItem it = tf_decode(P, item);
                const TfProblem& p = P.p[it.prob];
                const int buf = local & 1;
                const uint32_t use = (uint32_t)(local >> 1);
                if (!mbar_wait(&tempty[buf], (use & 1u) ^ 1u, abort_flag, P.error, 2)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * kMaxBN;
                const uint32_t idesc = instr_desc_tf32(p.bn);
                for (int kb = 0; kb < p.kblocks; ++kb) {
                    if (!mbar_wait(&full[stage], phase, abort_flag, P.error, 3)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t da = a_desc0 + (uint64_t)((uint32_t)stage * (kStageA >> 4));
                    const uint64_t db = b_desc0 + (uint64_t)((uint32_t)stage * (kTfStageB >> 4));
                    // four k-steps of 8 floats (32 bytes) each
                    umma_tf32(d_tmem, da, db, idesc, kb > 0 ? 1u : 0u);
                    umma_tf32(d_tmem, da + 2, db + 2, idesc, 1u);
                    umma_tf32(d_tmem, da + 4, db + 4, idesc, 1u);
                    umma_tf32(d_tmem, da + 6, db + 6, idesc, 1u);
                    umma_commit(&empty[stage]);       // frees the stage once these MMAs have read it
                    if (++stage == kTfStages) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(&tfull[buf]);     // accumulator complete
            }
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
        const int group = (warp - 2) >> 2;         // columns [32 group, 32 group + 32) of the tile
        // lane r owns row r of the warp's 32 x 32 FP32 tile (128 bytes = eight 16-byte pieces), piece j is kept
        // at j ^ (r & 7): the 128-byte swizzle of the tensor maps, conflict-free for the warp.  For the data
        // gradient the same tile first receives the stored post-activations by TMA load.
        uint8_t* tile = sOut + (warp - 2) * kTfTile;
        uint8_t* tile_row = tile + lane * 128;
        const int sw = lane & 7;
        uint64_t* my_aux = &auxbar[warp - 2];
        uint32_t aux_phase = 0;
        bool aux_pending = false;
        bool ok = true;
        int local = 0;
        for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++local) {
            const TfItem it = tf_decode(P, item);
            const TfProblem& p = P.p[it.prob];
            const int buf = local & 1;
            const uint32_t use = (uint32_t)(local >> 1);
            const int col = it.n0 + 32 * group;
            const int row0 = it.m0 + 32 * q;
            const bool active = 32 * group < p.bn && col < p.n_extent;     // uniform across the warp
            if (active) {
                // the previous item's store must have read the tile before it is reused
                if (lane == 0) {
                    tma_store_wait_read();
                    if (MODE == TF_DGRAD) {
                        mbar_expect_tx(my_aux, kTfTile);
                        tma_load_2d(tile, &P.tmAux[it.prob], col, row0, my_aux);
                    }
                }
                if (MODE == TF_DGRAD) aux_pending = true;
                __syncwarp();
            }
            if (!mbar_wait(&tfull[buf], use & 1u, abort_flag, P.error, 4)) { ok = false; break; }
            tc_fence_after();
            if (MODE == TF_DGRAD && active) {
                if (!mbar_wait(my_aux, aux_phase, abort_flag, P.error, 5)) { ok = false; break; }
                aux_phase ^= 1u;
                aux_pending = false;
            }
            if (active) {
                uint32_t acc[32];
                tmem_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * kMaxBN + 32 * group), acc);
                // the accumulator has been read: hand the tensor-memory buffer back first
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tempty[buf]);
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    float4* piece = reinterpret_cast<float4*>(tile_row + ((g ^ sw) << 4));
                    float4 o;
                    if (MODE == TF_FWD) {
                        const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + col) + g);
                        o.x = elu_fast(__uint_as_float(acc[4 * g]) + b.x, P.alpha);
                        o.y = elu_fast(__uint_as_float(acc[4 * g + 1]) + b.y, P.alpha);
                        o.z = elu_fast(__uint_as_float(acc[4 * g + 2]) + b.z, P.alpha);
                        o.w = elu_fast(__uint_as_float(acc[4 * g + 3]) + b.w, P.alpha);
                    } else if (MODE == TF_BIAS) {
                        const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + col) + g);
                        o.x = __uint_as_float(acc[4 * g]) + b.x;
                        o.y = __uint_as_float(acc[4 * g + 1]) + b.y;
                        o.z = __uint_as_float(acc[4 * g + 2]) + b.z;
                        o.w = __uint_as_float(acc[4 * g + 3]) + b.w;
                    } else if (MODE == TF_PLAIN) {
                        o.x = __uint_as_float(acc[4 * g]); o.y = __uint_as_float(acc[4 * g + 1]);
                        o.z = __uint_as_float(acc[4 * g + 2]); o.w = __uint_as_float(acc[4 * g + 3]);
                    } else {
                        const float4 h = *piece;
                        o.x = __uint_as_float(acc[4 * g]) * elu_grad_from_h(h.x, P.alpha);
                        o.y = __uint_as_float(acc[4 * g + 1]) * elu_grad_from_h(h.y, P.alpha);
                        o.z = __uint_as_float(acc[4 * g + 2]) * elu_grad_from_h(h.z, P.alpha);
                        o.w = __uint_as_float(acc[4 * g + 3]) * elu_grad_from_h(h.w, P.alpha);
                    }
                    *piece = o;
                }
                fence_async_smem();                           // tile writes -> visible to the copy engine
                __syncwarp();
                // rows and columns at or beyond the tensor's extent are clipped by the store itself
                if (lane == 0 && row0 < p.m_extent) tma_store_2d(&P.tmOut[it.prob], tile, col, row0);
            } else {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tempty[buf]);
            }
        }
        if (lane == 0) {
            if (MODE == TF_DGRAD && aux_pending) {      // gave up with a load in flight: let it land first
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(my_aux, aux_phase) && global_ns() - t0 < kWaitLimitNs) {}
            }
            tma_store_wait_all();   // stores done before the CTA retires
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------ weight gradient
// dW[features_in x features_out] = X^T dZ over the minibatch rows, both operands as stored ([row][feature], the
// contraction index outermost: MN-major tiles of 32 features x 32 rows, one 128-byte row per minibatch row, swizzled
// in units of 32 bytes, the form the tensor cores take for MN-major operands of 32-bit elements).
// A work item is a 128 x (<= 256) tile of one layer over one split of the row range; its FP32 result is a partial
// that the gradient reduction sums.  A split without rows (the row range does not always fill the last one) writes
// zeros.
constexpr int kTfWgProblems = 2 * kMaxLayers;     // every layer of both nets
constexpr int kTfWgStages = 4;
constexpr uint32_t kTfWgBox = 32 * 32 * 4;        // 4 KiB: 32 features x 32 rows
constexpr uint32_t kTfWgStageA = 4 * kTfWgBox;    // 128 features
constexpr int kTfWgMaxBN = 256;                   // output features per tile
constexpr uint32_t kTfWgStageB = (kTfWgMaxBN / 32) * kTfWgBox;    // up to 256 features
constexpr size_t kTfWgSmem = 1024 + (size_t)kTfWgStages * (kTfWgStageA + kTfWgStageB) + 512;

struct TfWgProblem {
    int m_extent, n_store;         // input features; output columns that are written (the padded width of the layer)
    int m_tiles, n_tiles, bn;
    int kblocks, kb_per_split, splits;
    int item_begin;
    float* out; int ld_out;        // partial of split 0: [m_extent][ld_out]
    long long split_stride;
};
struct TfWgParams {
    CUtensorMap tmA[kTfWgProblems], tmB[kTfWgProblems];   // [rows][features], boxes of 32 features x 32 rows
    TfWgProblem p[kTfWgProblems];
    int count, total_items;
    int* error;
};
struct TfWgItem { int prob, m0, n0, kb0, kb1, split; };
__device__ __forceinline__ TfWgItem tf_wg_decode(const TfWgParams& P, int item) {
    int pi = 0;
#pragma unroll 1
    for (int i = 1; i < P.count; ++i)
        if (item >= P.p[i].item_begin) pi = i;
    const TfWgProblem& p = P.p[pi];
    const int local = item - p.item_begin;
    const int per_split = p.m_tiles * p.n_tiles;
    TfWgItem it;
    it.prob = pi;
    it.split = local / per_split;
    const int rem = local - it.split * per_split;
    it.m0 = (rem / p.n_tiles) * BLOCK_M;
    it.n0 = (rem % p.n_tiles) * p.bn;
    it.kb0 = min(p.kblocks, it.split * p.kb_per_split);
    it.kb1 = min(p.kblocks, it.kb0 + p.kb_per_split);
    return it;
}

// Shared-memory descriptor of an MN-major operand of 32-bit elements: 128-byte swizzle in units of 32 bytes (the
// tensor maps' CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B), whose pattern repeats every four rows of 128 bytes.
__device__ __forceinline__ uint64_t smem_desc_mn32(uint32_t addr, uint32_t lead_bytes, uint32_t stride_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lead_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((stride_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;                 // descriptor version of this architecture
    d |= 1ull << 61;                 // 128-byte swizzle with 32-byte units
    return d;
}

// Instruction descriptor: TF32 x TF32 -> FP32, both operands MN-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t instr_desc_tf32_mn(int bn) {
    return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(bn >> 3) << 17) |
           ((uint32_t)(BLOCK_M >> 4) << 24);
}

__global__ void __launch_bounds__(kThreads, 1) tf32_wgrad_kernel(const __grid_constant__ TfWgParams P) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = smem + kTfWgStages * kTfWgStageA;
    uint64_t* full = reinterpret_cast<uint64_t*>(sB + kTfWgStages * kTfWgStageB);
    uint64_t* empty = full + kTfWgStages;
    uint64_t* tfull = empty + kTfWgStages;
    uint64_t* tempty = tfull + 2;
    uint64_t* drain = tempty + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kTfWgStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
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
        // a k-block is up to twelve boxes of 32 features x 32 rows (four of A, up to eight of B): lane l issues box l
        int stage = 0; uint32_t phase = 0;
        uint32_t issued_mask = 0, issued_parity = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x) {
            const TfWgItem it = tf_wg_decode(P, item);
            const TfWgProblem& p = P.p[it.prob];
            const uint32_t bytes = kTfWgStageA + (uint32_t)(p.bn / 32) * kTfWgBox;
            const bool mine = lane < 4 + p.bn / 32;
            const CUtensorMap* tm = lane < 4 ? &P.tmA[it.prob] : &P.tmB[it.prob];
            const int x = lane < 4 ? it.m0 + 32 * lane : it.n0 + 32 * (lane - 4);
            uint8_t* base = lane < 4 ? sA + (uint32_t)lane * kTfWgBox : sB + (uint32_t)(lane - 4) * kTfWgBox;
            const uint32_t per_stage = lane < 4 ? kTfWgStageA : kTfWgStageB;
            for (int kb = it.kb0; kb < it.kb1; ++kb) {
                int good = 1;
                if (lane == 0) {
                    good = mbar_wait(&empty[stage], phase ^ 1u, abort_flag, P.error, 21) ? 1 : 0;
                    if (good) mbar_expect_tx(&full[stage], bytes);
                }
                good = __shfl_sync(0xffffffffu, good, 0);
                if (!good) { ok = false; break; }
                if (mine) tma_load_2d(base + (uint32_t)stage * per_stage, tm, x, kb * kTfBlockK, &full[stage]);
                issued_mask |= 1u << stage;
                issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                if (++stage == kTfWgStages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok && lane == 0) {
            // let the copies already issued land before the CTA's shared memory goes away
            for (int s = 0; s < kTfWgStages; ++s) {
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
            // MN-major operands: 4096 bytes between blocks of 32 features, 512 between groups of four rows (one
            // period of the swizzle); a k-step is eight rows (1024 bytes); descriptors differ only in their address
            // field (16-byte units)
            const uint64_t a_desc0 = smem_desc_mn32(smem_u32(sA), kTfWgBox, 512);
            const uint64_t b_desc0 = smem_desc_mn32(smem_u32(sB), kTfWgBox, 512);
            constexpr uint32_t kstep = 1024 >> 4;
            for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++local) {
                const TfWgItem it = tf_wg_decode(P, item);
                const TfWgProblem& p = P.p[it.prob];
                const int buf = local & 1;
                const uint32_t use = (uint32_t)(local >> 1);
                if (!mbar_wait(&tempty[buf], (use & 1u) ^ 1u, abort_flag, P.error, 22)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * kMaxBN;
                const uint32_t idesc = instr_desc_tf32_mn(p.bn);
                for (int kb = it.kb0; kb < it.kb1; ++kb) {
                    if (!mbar_wait(&full[stage], phase, abort_flag, P.error, 23)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t da = a_desc0 + (uint64_t)((uint32_t)stage * (kTfWgStageA >> 4));
                    const uint64_t db = b_desc0 + (uint64_t)((uint32_t)stage * (kTfWgStageB >> 4));
                    umma_tf32(d_tmem, da, db, idesc, kb > it.kb0 ? 1u : 0u);
                    umma_tf32(d_tmem, da + kstep, db + kstep, idesc, 1u);
                    umma_tf32(d_tmem, da + 2 * kstep, db + 2 * kstep, idesc, 1u);
                    umma_tf32(d_tmem, da + 3 * kstep, db + 3 * kstep, idesc, 1u);
                    umma_commit(&empty[stage]);       // frees the stage once these MMAs have read it
                    if (++stage == kTfWgStages) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(&tfull[buf]);     // accumulator complete (at once for a split without rows)
            }
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
        const int group = (warp - 2) >> 2;         // chunks of 32 columns: group and group + 4
        bool ok = true;
        int local = 0;
        for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x, ++local) {
            const TfWgItem it = tf_wg_decode(P, item);
            const TfWgProblem& p = P.p[it.prob];
            const int buf = local & 1;
            const uint32_t use = (uint32_t)(local >> 1);
            const int row = it.m0 + 32 * q + lane;
            if (!mbar_wait(&tfull[buf], use & 1u, abort_flag, P.error, 24)) { ok = false; break; }
            tc_fence_after();
            // a warp takes the 32-column chunks `group` and `group + 4` of the tile
#pragma unroll
            for (int ci = 0; ci < 2; ++ci) {
                const int chunk = group + 4 * ci;
                const int col = it.n0 + 32 * chunk;
                if (32 * chunk >= p.bn || col >= p.n_store) break;          // uniform across the warp
                uint32_t acc[32];
                tmem_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * kMaxBN + 32 * chunk), acc);
                if (it.kb0 >= it.kb1) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[i] = 0u;             // nothing was accumulated
                }
                if (row < p.m_extent) {
                    float* dst = p.out + (size_t)it.split * p.split_stride + (size_t)row * p.ld_out + col;
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        if (col + 4 * g < p.n_store)
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

// Transposed copies of the hidden-layer weights: W[in][ld_src] -> Wt[out][ld_dst].
struct TransposeEntry { const float* src; float* dst; int in, out, ld_src, ld_dst; };

__global__ void tf32_transpose_kernel(const TransposeEntry* __restrict__ table) {
    __shared__ float t[32][33];
    const TransposeEntry e = table[blockIdx.z];
    const int i0 = blockIdx.y * 32, o0 = blockIdx.x * 32;
    if (i0 >= e.in || o0 >= e.out) return;
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int i = i0 + r, o = o0 + threadIdx.x;
        t[r][threadIdx.x] = (i < e.in && o < e.out) ? e.src[(size_t)i * e.ld_src + o] : 0.f;
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int o = o0 + r, i = i0 + threadIdx.x;
        if (o < e.out && i < e.in) e.dst[(size_t)o * e.ld_dst + i] = t[threadIdx.x][r];
    }
}

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

// 2-D FP32 tensor [rows][cols] with row stride ld (floats); box = box_cols x box_rows, 128-byte swizzle.
bool make_tmap_f32(CUtensorMap* tm, const void* base, long long rows, int cols, int ld, int box_cols, int box_rows,
                   CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct Tf32Engine {
    Tf32Setup s;
    int nh[2];
    std::vector<void*> allocs;
    float* wt[2][kMaxLayers] = {};                // [out][ld_wt] transposed weight copies
    int ld_wt[2][kMaxLayers] = {};
    TransposeEntry* table_dev = nullptr; int n_table = 0, max_in = 0, max_out = 0;
    int* error_dev = nullptr;
    int num_sms = 148;
    std::vector<TfParams> act_fwd, last_fwd, upd_fwd, upd_dgrad;   // one launch per hidden layer index / backward step
    TfWgParams upd_wgrad;                                          // one launch for every layer of both nets
};

namespace {

template <typename T>
bool talloc(Tf32Engine* e, T** p, size_t count) {
    void* q = nullptr;
    const size_t bytes = std::max<size_t>(count, 1) * sizeof(T);
    if (guarded_malloc(&q, bytes) != cudaSuccess) return false;
    e->allocs.push_back(q);
    if (cudaMemsetAsync(q, 0, bytes, e->s.stream) != cudaSuccess) return false;
    *p = reinterpret_cast<T*>(q);
    return true;
}

void finish(TfParams& P, float alpha, int* error) {
    int items = 0;
    for (int i = 0; i < P.count; ++i) { P.p[i].item_begin = items; items += P.p[i].m_tiles * P.p[i].n_tiles; }
    P.total_items = items; P.alpha = alpha; P.error = error;
}

// D[rows x n] = A[rows x k] * B[n x k]^T with A [a_rows_total][lda], B [n][ldb], D [rows][ldd]; aux (may be null) like D.
// n_store (>= n, default n): columns of D that are written; those at and beyond n come out as zero.
bool add_problem(TfParams& P, const float* A, long long a_rows_total, int rows, int k, int lda, const float* B, int n, int ldb,
                 float* D, int ldd, const float* aux, const float* bias, int n_store = 0) {
    const int i = P.count;
    TfProblem& p = P.p[i];
    memset(&p, 0, sizeof p);
    if (n_store < n) n_store = n;
    p.bn = std::min(kTfMaxBN, round_up(n_store, 16));
    p.m_extent = rows; p.n_extent = n_store;
    p.m_tiles = (rows + BLOCK_M - 1) / BLOCK_M;
    p.n_tiles = (n_store + p.bn - 1) / p.bn;
    p.kblocks = (k + kTfBlockK - 1) / kTfBlockK;
    p.bias = bias;
    if (!make_tmap_f32(&P.tmA[i], A, a_rows_total, k, lda, kTfBlockK, BLOCK_M)) return false;
    if (!make_tmap_f32(&P.tmB[i], B, n, k, ldb, kTfBlockK, p.bn)) return false;
    if (!make_tmap_f32(&P.tmOut[i], D, rows, n_store, ldd, 32, 32)) return false;
    if (aux && !make_tmap_f32(&P.tmAux[i], aux, rows, n, ldd, 32, 32)) return false;
    P.count++;
    return true;
}

template <int MODE>
cudaError_t launch_tf(const TfParams& P, int num_sms, cudaStream_t s) {
    if (P.total_items == 0) return cudaSuccess;
    const int grid = std::min(P.total_items, num_sms);
    LaunchScope scope_(MODE == TF_FWD ? "tc_gemm_fwd" : MODE == TF_DGRAD ? "tc_gemm_dgrad" : "tc_gemm_linear", s);
    return launch_chained(tf32_gemm_kernel<MODE>, grid, kThreads, kTfSmem, s, P);
}

}  // namespace

Tf32Engine* tf32_create(const Tf32Setup& s, std::string* err) {
    auto failmsg = [&](const char* m) { if (err) *err = m; return (Tf32Engine*)nullptr; };
    if (!get_encode_fn()) return failmsg("cuTensorMapEncodeTiled is not available from the driver");
    int dev = 0; cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return failmsg("no CUDA device");
    if (prop.major != 10) return failmsg("the tensor-core mode needs an sm_100 device");
    if (cudaFuncSetAttribute(tf32_gemm_kernel<TF_FWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTfSmem) != cudaSuccess ||
        cudaFuncSetAttribute(tf32_gemm_kernel<TF_DGRAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTfSmem) != cudaSuccess ||
        cudaFuncSetAttribute(tf32_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTfWgSmem) != cudaSuccess)
        return failmsg("could not reserve shared memory for the tensor-core kernels");
    Tf32Engine* e = new Tf32Engine();
    e->s = s;
    e->num_sms = prop.multiProcessorCount;
    auto bail = [&](const char* m) { if (err) *err = m; tf32_destroy(e); return (Tf32Engine*)nullptr; };
    if (!talloc(e, &e->error_dev, 1)) return bail("allocation failed");
    std::vector<TransposeEntry> table;
    for (int ni = 0; ni < 2; ++ni) {
        e->nh[ni] = s.nl[ni] - 1;
        for (int l = 0; l < e->nh[ni]; ++l) {
            e->ld_wt[ni][l] = round_up(s.in[ni][l], 4);
            if (!talloc(e, &e->wt[ni][l], (size_t)s.out[ni][l] * e->ld_wt[ni][l])) return bail("allocation failed");
            table.push_back(TransposeEntry{s.param + s.w_off[ni][l], e->wt[ni][l], s.in[ni][l], s.out[ni][l], s.out_p[ni][l], e->ld_wt[ni][l]});
            e->max_in = std::max(e->max_in, s.in[ni][l]); e->max_out = std::max(e->max_out, s.out[ni][l]);
        }
    }
    e->n_table = (int)table.size();
    if (!talloc(e, &e->table_dev, table.size())) return bail("allocation failed");
    if (cudaMemcpyAsync(e->table_dev, table.data(), table.size() * sizeof(TransposeEntry), cudaMemcpyHostToDevice, s.stream) != cudaSuccess ||
        cudaStreamSynchronize(s.stream) != cudaSuccess)
        return bail("copy of the transpose table failed");

    const int maxh = std::max(e->nh[0], e->nh[1]);
    // forward launches, one per hidden layer index; kind 0: act on rollout step t, 1: critic on the last observation, 2: update
    auto build_fwd = [&](std::vector<TfParams>& out, int kind) -> bool {
        const int rows = kind == 2 ? s.R : s.N;
        for (int l = 0; l < maxh; ++l) {
            TfParams P; memset(&P, 0, sizeof P);
            for (int ni = 0; ni < 2; ++ni) {
                if ((kind == 1 && ni == 0) || l >= e->nh[ni]) continue;
                float* const* h = kind == 2 ? s.up_h[ni] : s.act_h[ni];
                const float* A; long long a_rows; int lda;
                if (l > 0) { A = h[l - 1]; a_rows = rows; lda = s.hid_ld[ni][l - 1]; }
                else if (kind == 0) { A = s.obs_storage[ni]; a_rows = (long long)s.T * s.N; lda = s.obs_stride[ni]; }
                else if (kind == 1) { A = s.last_obs_c; a_rows = rows; lda = s.obs_stride[1]; }
                else { A = s.x[ni]; a_rows = rows; lda = s.in_ld[ni]; }
                if (!add_problem(P, A, a_rows, rows, s.in[ni][l], lda, e->wt[ni][l], s.out[ni][l], e->ld_wt[ni][l], h[l], s.hid_ld[ni][l],
                                 nullptr, s.param + s.b_off[ni][l]))
                    return false;
            }
            finish(P, s.elu_alpha, e->error_dev);
            out.push_back(P);
        }
        return true;
    };
    if (!build_fwd(e->act_fwd, 0) || !build_fwd(e->last_fwd, 1) || !build_fwd(e->upd_fwd, 2)) return bail("tensor map encoding failed");
    // data-gradient launches: step `back` produces dL/dz of hidden layer nh - 2 - back from that of nh - 1 - back:
    // dZ[l-1] = (dZ[l] W[l]^T) * ELU'(h[l-1]); the operand W[l] is [in][out_p] as stored (contraction = out, contiguous)
    for (int back = 0; back + 1 < maxh; ++back) {
        TfParams P; memset(&P, 0, sizeof P);
        for (int ni = 0; ni < 2; ++ni) {
            const int l = e->nh[ni] - 1 - back;
            if (l < 1) continue;
            if (!add_problem(P, s.up_dz[ni][l], s.R, s.R, s.out[ni][l], s.hid_ld[ni][l], s.param + s.w_off[ni][l], s.in[ni][l], s.out_p[ni][l],
                             s.up_dz[ni][l - 1], s.hid_ld[ni][l - 1], s.up_h[ni][l - 1], nullptr))
                return bail("tensor map encoding failed");
        }
        finish(P, s.elu_alpha, e->error_dev);
        e->upd_dgrad.push_back(P);
    }
    // weight gradients: dW[l] = hin[l]^T dZ[l] over the rows of each split (the heads' dZ is dL/d(head output))
    {
        TfWgParams& W = e->upd_wgrad;
        memset(&W, 0, sizeof W);
        if (s.kchunk % kTfBlockK != 0 || s.splits < 1) return bail("rows per weight-gradient split must be a multiple of 32");
        int items = 0;
        for (int ni = 0; ni < 2; ++ni)
            for (int l = 0; l < s.nl[ni]; ++l) {
                if (W.count == kTfWgProblems) return bail("too many layers for the weight-gradient launch");
                const int i = W.count;
                TfWgProblem& p = W.p[i];
                const bool head = l == e->nh[ni];
                const float* hin = l == 0 ? s.x[ni] : s.up_h[ni][l - 1];
                const int ldin = l == 0 ? s.in_ld[ni] : s.hid_ld[ni][l - 1];
                const float* dz = head ? s.dhead[ni] : s.up_dz[ni][l];
                const int lddz = head ? s.ld_dhead[ni] : s.hid_ld[ni][l];
                p.m_extent = s.in[ni][l]; p.n_store = s.out_p[ni][l];
                p.bn = std::min(kTfWgMaxBN, round_up(s.out[ni][l], 32));
                p.m_tiles = (p.m_extent + BLOCK_M - 1) / BLOCK_M;
                p.n_tiles = (p.n_store + p.bn - 1) / p.bn;
                p.kblocks = (s.R + kTfBlockK - 1) / kTfBlockK;
                p.kb_per_split = s.kchunk / kTfBlockK;
                p.splits = s.splits;
                p.item_begin = items; items += p.m_tiles * p.n_tiles * p.splits;
                p.out = s.partials + s.w_off[ni][l]; p.ld_out = s.out_p[ni][l]; p.split_stride = s.split_stride;
                if (!make_tmap_f32(&W.tmA[i], hin, s.R, s.in[ni][l], ldin, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) ||
                    !make_tmap_f32(&W.tmB[i], dz, s.R, s.out[ni][l], lddz, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
                    return bail("tensor map encoding failed");
                W.count++;
            }
        W.total_items = items; W.error = e->error_dev;
    }
    if (cudaStreamSynchronize(s.stream) != cudaSuccess) return bail("stream synchronisation failed");
    return e;
}

void tf32_destroy(Tf32Engine* e) {
    if (!e) return;
    for (void* p : e->allocs) guarded_free(p);
    delete e;
}

cudaError_t tf32_refresh_weights(Tf32Engine* e) {
    if (e->n_table == 0) return cudaSuccess;
    dim3 grid((e->max_out + 31) / 32, (e->max_in + 31) / 32, e->n_table);
    LaunchScope scope_("convert_weights", e->s.stream);
    tf32_transpose_kernel<<<grid, dim3(32, 8), 0, e->s.stream>>>(e->table_dev);
    return cudaGetLastError();
}

cudaError_t tf32_act_forward(Tf32Engine* e, int t, bool do_actor) {
    for (const TfParams& P0 : do_actor ? e->act_fwd : e->last_fwd) {
        TfParams P = P0;
        if (do_actor)
            for (int i = 0; i < P.count; ++i)
                if (&P0 == &e->act_fwd[0]) P.p[i].row_offset = t * e->s.N;      // the first layer reads the storage rows of step t
        cudaError_t err = launch_tf<TF_FWD>(P, e->num_sms, e->s.stream);
        if (err != cudaSuccess) return err;
    }
    return cudaSuccess;
}

cudaError_t tf32_update_forward(Tf32Engine* e) {
    FamilyScope family_("tc_gemm_fwd", e->s.stream);
    for (const TfParams& P : e->upd_fwd) {
        cudaError_t err = launch_tf<TF_FWD>(P, e->num_sms, e->s.stream);
        if (err != cudaSuccess) return err;
    }
    return cudaSuccess;
}

cudaError_t tf32_update_dgrad(Tf32Engine* e, int back) {
    if (back < 0 || back >= (int)e->upd_dgrad.size()) return cudaSuccess;
    return launch_tf<TF_DGRAD>(e->upd_dgrad[back], e->num_sms, e->s.stream);
}

cudaError_t tf32_update_wgrad(Tf32Engine* e) {
    const TfWgParams& W = e->upd_wgrad;
    if (W.total_items == 0) return cudaSuccess;
    LaunchScope scope_("tc_gemm_wgrad", e->s.stream);
    return launch_chained(tf32_wgrad_kernel, std::min(W.total_items, e->num_sms), kThreads, kTfWgSmem, e->s.stream, W);
}

cudaError_t tf32_read_error(Tf32Engine* e, int* host_code) {
    cudaError_t err = cudaMemcpyAsync(host_code, e->error_dev, sizeof(int), cudaMemcpyDeviceToHost, e->s.stream);
    if (err != cudaSuccess) return err;
    err = cudaStreamSynchronize(e->s.stream);
    if (err != cudaSuccess || *host_code == 0) return err;
    return cudaMemsetAsync(e->error_dev, 0, sizeof(int), e->s.stream);
}

// ------------------------------------------------------------------ prepared launches for other callers
struct Tf32Op {
    int kind = 0;                 // a TfMode: P; 100: W
    TfParams P;
    TfWgParams W;
    int num_sms = 148;
};

namespace {

__global__ void tf32_transpose_one_kernel(TransposeEntry e) {
    __shared__ float t[32][33];
    const int i0 = blockIdx.y * 32, o0 = blockIdx.x * 32;
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int i = i0 + r, o = o0 + threadIdx.x;
        t[r][threadIdx.x] = (i < e.in && o < e.out) ? e.src[(size_t)i * e.ld_src + o] : 0.f;
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int o = o0 + r, i = i0 + threadIdx.x;
        if (o < e.out && i < e.in) e.dst[(size_t)o * e.ld_dst + i] = t[threadIdx.x][r];
    }
}

int device_sms() {
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

}  // namespace

bool tf32_ops_init(std::string* err) {
    auto failmsg = [&](const char* m) { if (err) *err = m; return false; };
    if (!get_encode_fn()) return failmsg("cuTensorMapEncodeTiled is not available from the driver");
    int dev = 0; cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return failmsg("no CUDA device");
    if (prop.major != 10) return failmsg("the tensor-core mode needs an sm_100 device");
    if (cudaFuncSetAttribute(tf32_gemm_kernel<TF_FWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTfSmem) != cudaSuccess ||
        cudaFuncSetAttribute(tf32_gemm_kernel<TF_DGRAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTfSmem) != cudaSuccess ||
        cudaFuncSetAttribute(tf32_gemm_kernel<TF_BIAS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTfSmem) != cudaSuccess ||
        cudaFuncSetAttribute(tf32_gemm_kernel<TF_PLAIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTfSmem) != cudaSuccess ||
        cudaFuncSetAttribute(tf32_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTfWgSmem) != cudaSuccess)
        return failmsg("could not reserve shared memory for the tensor-core kernels");
    return true;
}

Tf32Op* tf32_op_gemm(const float* A, int rows, int k, int lda, const float* B, int n, int ldb, float* D, int ldd,
                     const float* bias, int* error_dev, int n_store) {
    Tf32Op* op = new Tf32Op();
    op->kind = bias ? TF_BIAS : TF_PLAIN;
    op->num_sms = device_sms();
    memset(&op->P, 0, sizeof op->P);
    if (!add_problem(op->P, A, rows, rows, k, lda, B, n, ldb, D, ldd, nullptr, bias, n_store)) { delete op; return nullptr; }
    finish(op->P, 0.f, error_dev);
    return op;
}

Tf32Op* tf32_op_gemm_act(int kind, const float* A, int rows, int k, int lda, const float* B, int n, int ldb, float* D, int ldd,
                         const float* bias_or_aux, float alpha, int* error_dev, int n_store) {
    if (!bias_or_aux || (kind != 0 && kind != 1)) return nullptr;
    Tf32Op* op = new Tf32Op();
    op->kind = kind == 0 ? TF_FWD : TF_DGRAD;
    op->num_sms = device_sms();
    memset(&op->P, 0, sizeof op->P);
    if (!add_problem(op->P, A, rows, rows, k, lda, B, n, ldb, D, ldd, kind == 1 ? bias_or_aux : nullptr,
                     kind == 0 ? bias_or_aux : nullptr, n_store)) { delete op; return nullptr; }
    finish(op->P, alpha, error_dev);
    return op;
}

Tf32Op* tf32_op_wgrad(const Tf32WgradDesc* d, int count, int rows, int splits, int kchunk, long long split_stride, int* error_dev) {
    if (count < 1 || count > kTfWgProblems || splits < 1 || kchunk < kTfBlockK || kchunk % kTfBlockK != 0) return nullptr;
    Tf32Op* op = new Tf32Op();
    op->kind = 100;
    op->num_sms = device_sms();
    TfWgParams& W = op->W;
    memset(&W, 0, sizeof W);
    int items = 0;
    for (int i = 0; i < count; ++i) {
        TfWgProblem& p = W.p[i];
        p.m_extent = d[i].m; p.n_store = d[i].n_store;
        p.bn = std::min(kTfWgMaxBN, round_up(d[i].n, 32));
        p.m_tiles = (p.m_extent + BLOCK_M - 1) / BLOCK_M;
        p.n_tiles = (p.n_store + p.bn - 1) / p.bn;
        p.kblocks = (rows + kTfBlockK - 1) / kTfBlockK;
        p.kb_per_split = kchunk / kTfBlockK;
        p.splits = splits;
        p.item_begin = items; items += p.m_tiles * p.n_tiles * p.splits;
        p.out = d[i].out; p.ld_out = d[i].ld_out; p.split_stride = split_stride;
        if (!make_tmap_f32(&W.tmA[i], d[i].A, rows, d[i].m, d[i].lda, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) ||
            !make_tmap_f32(&W.tmB[i], d[i].B, rows, d[i].n, d[i].ldb, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B)) {
            delete op;
            return nullptr;
        }
        W.count++;
    }
    W.total_items = items; W.error = error_dev;
    return op;
}

cudaError_t tf32_op_launch(const Tf32Op* op, cudaStream_t stream) {
    if (!op) return cudaErrorInvalidValue;
    if (op->kind == 100) {
        if (op->W.total_items == 0) return cudaSuccess;
        LaunchScope scope_("tc_gemm_wgrad", stream);
        return launch_chained(tf32_wgrad_kernel, std::min(op->W.total_items, op->num_sms), kThreads, kTfWgSmem, stream, op->W);
    }
    if (op->kind == TF_FWD) return launch_tf<TF_FWD>(op->P, op->num_sms, stream);
    if (op->kind == TF_DGRAD) return launch_tf<TF_DGRAD>(op->P, op->num_sms, stream);
    if (op->kind == TF_BIAS) return launch_tf<TF_BIAS>(op->P, op->num_sms, stream);
    return launch_tf<TF_PLAIN>(op->P, op->num_sms, stream);
}

void tf32_op_free(Tf32Op* op) { delete op; }

cudaError_t tf32_transpose(const float* src, int in, int out, int ld_src, float* dst, int ld_dst, cudaStream_t stream) {
    if (in <= 0 || out <= 0) return cudaSuccess;
    const TransposeEntry e{src, dst, in, out, ld_src, ld_dst};
    tf32_transpose_one_kernel<<<dim3((out + 31) / 32, (in + 31) / 32), dim3(32, 8), 0, stream>>>(e);
    return cudaGetLastError();
}

}  // namespace rslrl
