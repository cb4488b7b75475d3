// Shared device helpers of the rslrl_b200 kernels: counter-based random streams, ELU, small
// reductions.  Nothing here is shared with the CPU oracle.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace rslrl {

constexpr int kMaxActions = 64;
constexpr int kMaxLayers = 9;           // up to 8 hidden layers + head
constexpr uint32_t kStreamNoise = 1u;
constexpr uint32_t kStreamPerm = 2u;
constexpr int kFeistelRounds = 6;

// ---------------------------------------------------------------------------------------
// Philox-4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).
// ---------------------------------------------------------------------------------------
struct U4 { uint32_t x, y, z, w; };

__host__ __device__ __forceinline__ U4 philox4x32_10(U4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c.x;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c.z;
        U4 n;
        n.x = (uint32_t)(p1 >> 32) ^ c.y ^ k0;
        n.y = (uint32_t)p1;
        n.z = (uint32_t)(p0 >> 32) ^ c.w ^ k1;
        n.w = (uint32_t)p0;
        c = n;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c;
}

// uint32 -> (0,1): ((x >> 9) + 1/2) * 2^-23; 24 significant bits, exact in float.
__device__ __forceinline__ float uniform_open01(uint32_t x) {
    return ((float)(x >> 9) + 0.5f) * 1.1920928955078125e-07f;
}

// Four standard normals for (env n, global step, action quad j): two Box-Muller pairs.
__device__ __forceinline__ void gaussian_quad(uint32_t seed_lo, uint32_t seed_hi, uint32_t n,
                                              uint32_t step, uint32_t quad, float out[4]) {
    U4 c{n, step, quad, kStreamNoise};
    const U4 r = philox4x32_10(c, seed_lo, seed_hi);
    const float u0 = uniform_open01(r.x), u1 = uniform_open01(r.y);
    const float u2 = uniform_open01(r.z), u3 = uniform_open01(r.w);
    const float r01 = sqrtf(-2.0f * logf(u0));
    const float r23 = sqrtf(-2.0f * logf(u2));
    float s, co;
    sincospif(2.0f * u1, &s, &co);
    out[0] = r01 * co; out[1] = r01 * s;
    sincospif(2.0f * u3, &s, &co);
    out[2] = r23 * co; out[3] = r23 * s;
}

// Keyed bijection of [0, size): balanced Feistel network over 2*half_bits bits with cycle
// walking.  Round function: word 0 of Philox(counter = (right half, epoch, iteration,
// kStreamPerm | round << 8), key = seed), masked to half_bits bits.
struct PermKey {
    uint32_t seed_lo, seed_hi, iteration, epoch;
    uint32_t size;
    uint32_t half_bits;
};

__host__ __device__ inline uint32_t feistel_half_bits(uint32_t size) {
    uint32_t bits = 0;
    while (bits < 32 && ((uint64_t)1 << bits) < (uint64_t)size) ++bits;
    if (bits < 2) bits = 2;
    bits += bits & 1u;
    return bits / 2;
}

__device__ __forceinline__ uint32_t feistel_network(const PermKey& pk, uint32_t x) {
    const uint32_t h = pk.half_bits;
    const uint32_t mask = (1u << h) - 1u;
    uint32_t left = x >> h, right = x & mask;
#pragma unroll 1
    for (int rnd = 0; rnd < kFeistelRounds; ++rnd) {
        U4 c{right, pk.epoch, pk.iteration, kStreamPerm | ((uint32_t)rnd << 8)};
        const uint32_t f = philox4x32_10(c, pk.seed_lo, pk.seed_hi).x & mask;
        const uint32_t nl = right;
        right = left ^ f;
        left = nl;
    }
    return (left << h) | right;
}

__device__ __forceinline__ uint32_t feistel_permute(const PermKey& pk, uint32_t i) {
    uint32_t x = feistel_network(pk, i);
    // Cycle walking ends: the network is a bijection of [0, 2^(2h)), so the orbit of i
    // returns to i (which is < size) after finitely many steps.
    while (x >= pk.size) x = feistel_network(pk, x);
    return x;
}

// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float elu_f(float z, float alpha) {
    return z > 0.0f ? z : alpha * expm1f(z);
}
// ELU'(z) written in terms of the stored post-activation h.
__device__ __forceinline__ float elu_grad_from_h(float h, float alpha) {
    return h > 0.0f ? 1.0f : h + alpha;
}

// Programmatic dependent launch: a kernel launched with launch_chained() may be scheduled while its
// predecessor in the stream still runs.  chain_begin() waits until every earlier grid has completed
// and its memory is visible, then lets the successor be scheduled (which in turn waits for this grid
// to complete): at most one waiting grid is resident at a time.  It comes before the first access to
// global memory, by every thread, and is a no-op for a plainly launched kernel.
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void chain_begin() { chain_wait(); chain_release(); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_float(float x);
template <> __device__ __forceinline__ float from_float<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) {
    return __float2bfloat16_rn(x);
}

}  // namespace rslrl
