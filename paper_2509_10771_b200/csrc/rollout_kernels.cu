// Rollout-side kernels: observation staging, policy/value heads with the Philox-keyed
// Gaussian sample and log-density, transition recording, and the GAE reverse scan with
// advantage normalisation.
#include "common.cuh"
#include "kernels.h"
#include <algorithm>

namespace rslrl {

namespace {

// ---------------------------------------------------------------------------------------
// dst[r][0..dst_ld) = src[r][0..dim) followed by zeros; optional bf16 twin.
// ---------------------------------------------------------------------------------------
// One warp per row, lanes on consecutive columns: coalesced loads and stores, no index division.
__global__ void pad_rows_kernel(const float* __restrict__ src, int dim, float* __restrict__ dst,
                                int dst_ld, __nv_bfloat16* __restrict__ dst16, int dst16_ld,
                                int rows) {
    chain_begin();
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const int ld = max(dst ? dst_ld : 0, dst16 ? dst16_ld : 0);
    for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < rows; r += warps) {
        const float* __restrict__ s = src + (size_t)r * dim;
        float* __restrict__ d = dst ? dst + (size_t)r * dst_ld : nullptr;
        __nv_bfloat16* __restrict__ d16 = dst16 ? dst16 + (size_t)r * dst16_ld : nullptr;
        for (int c0 = 0; c0 < ld; c0 += 128) {
            float v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int c = c0 + 32 * q + lane;
                v[q] = c < dim ? s[c] : 0.f;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int c = c0 + 32 * q + lane;
                if (d && c < dst_ld) d[c] = v[q];
                if (d16 && c < dst16_ld) d16[c] = __float2bfloat16_rn(v[q]);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// Heads.  One warp per row; lanes split the hidden width, so the row is read coalesced.
// Lane i ends up owning outputs i and i + 32.
// ---------------------------------------------------------------------------------------
constexpr float kHalfLog2Pi = 0.91893853320467274178f;

template <typename T>
__device__ __forceinline__ void head_dot(const T* __restrict__ h, int n, const float* __restrict__ W,
                                         int ldw, const float* __restrict__ bias, int nout,
                                         float& out_lo, float& out_hi) {
    const int lane = threadIdx.x & 31;
    out_lo = 0.f; out_hi = 0.f;
    for (int o0 = 0; o0 < nout; o0 += 8) {
        float acc[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[q] = 0.f;
        for (int k = lane; k < n; k += 32) {
            const float hv = to_float(h[k]);
            const float* w = W + (size_t)k * ldw + o0;
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

template <typename T>
__global__ void __launch_bounds__(256) act_head_kernel(const T* __restrict__ Ha, int ldha,
                                                       const T* __restrict__ Hc, int ldhc,
                                                       const HeadParams hp, const ActOut out, int N,
                                                       uint32_t seed_lo, uint32_t seed_hi,
                                                       uint32_t global_step) {
    chain_begin();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp == 0) {
        for (int i = lane; i < out.act_stride; i += 32)
            out.sigma[i] = i < hp.A ? expf(hp.log_std[i]) : 0.f;
    }
    if (warp >= N) return;
    const int n = warp;
    float mu_lo, mu_hi, v_lo, v_hi;
    head_dot(Ha + (size_t)n * ldha, hp.n_a, hp.Wa, hp.ldwa, hp.ba, hp.A, mu_lo, mu_hi);
    head_dot(Hc + (size_t)n * ldhc, hp.n_c, hp.Wc, hp.ldwc, hp.bc, 1, v_lo, v_hi);
    // lane i finishes actions i and i + 32; the four lanes of a quad draw the same Philox block
    float logp_part = 0.f;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int i = lane + 32 * half;
        if (i >= out.act_stride) continue;
        float a = 0.f, m = 0.f;
        if (i < hp.A) {
            float eps[4];
            gaussian_quad(seed_lo, seed_hi, (uint32_t)n, global_step, (uint32_t)(i >> 2), eps);
            const float e = (i & 3) == 0 ? eps[0] : (i & 3) == 1 ? eps[1] : (i & 3) == 2 ? eps[2] : eps[3];
            const float ls = hp.log_std[i];
            const float sg = expf(ls);
            m = half ? mu_hi : mu_lo;
            a = fmaf(sg, e, m);
            const float d = a - m;
            logp_part += -(d * d) / (2.0f * sg * sg) - ls - kHalfLog2Pi;
        }
        out.actions[(size_t)n * out.act_stride + i] = a;
        out.mu[(size_t)n * out.act_stride + i] = m;
        if (out.actions_out) out.actions_out[(size_t)n * out.act_stride + i] = a;
    }
    const float logp = warp_sum(logp_part);
    if (lane == 0) {
        out.logp[n] = logp;
        out.values[n] = v_lo;
    }
}

template <typename T>
__global__ void __launch_bounds__(256) value_head_kernel(const T* __restrict__ Hc, int ldhc,
                                                         const HeadParams hp, float* __restrict__ values,
                                                         int N) {
    chain_begin();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (warp >= N) return;
    float v, unused;
    head_dot(Hc + (size_t)warp * ldhc, hp.n_c, hp.Wc, hp.ldwc, hp.bc, 1, v, unused);
    if ((threadIdx.x & 31) == 0) values[warp] = v;
}

__global__ void record_step_kernel(const float* __restrict__ rew, const uint8_t* __restrict__ dones,
                                   const uint8_t* __restrict__ timeouts, float* __restrict__ s_rew,
                                   uint8_t* __restrict__ s_dones, uint8_t* __restrict__ s_timeouts,
                                   int N) {
    chain_begin();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) {
        s_rew[i] = rew[i];
        s_dones[i] = dones[i] ? 1 : 0;
        s_timeouts[i] = timeouts[i] ? 1 : 0;
    }
}

// ---------------------------------------------------------------------------------------
// GAE.  One thread per environment, t-major arrays: a warp reads 32 consecutive environments
// of one time step (coalesced).  The loads of a thread do not depend on the recurrence, so
// they are issued ahead of the FMA chain in chunks.  Each thread keeps a running
// (count, mean, M2) of its advantages (Welford); warps and then the block merge them with
// Chan's pairwise formula and write one (count, mean, M2) triple per block.
// ---------------------------------------------------------------------------------------
constexpr int kGaeThreads = 128;

struct Moments { float n, mean, m2; };

__device__ __forceinline__ Moments merge(const Moments a, const Moments b) {
    Moments r;
    r.n = a.n + b.n;
    if (r.n == 0.f) { r.mean = 0.f; r.m2 = 0.f; return r; }
    const float d = b.mean - a.mean;
    const float fb = b.n / r.n;
    r.mean = a.mean + d * fb;
    r.m2 = a.m2 + b.m2 + d * d * a.n * fb;
    return r;
}

__device__ __forceinline__ Moments warp_merge(Moments mom) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Moments other;
        other.n = __shfl_down_sync(0xffffffffu, mom.n, o);
        other.mean = __shfl_down_sync(0xffffffffu, mom.mean, o);
        other.m2 = __shfl_down_sync(0xffffffffu, mom.m2, o);
        mom = merge(mom, other);
    }
    return mom;
}

__global__ void __launch_bounds__(kGaeThreads) gae_scan_kernel(
    const float* __restrict__ rewards, const float* __restrict__ values,
    const uint8_t* __restrict__ dones, const uint8_t* __restrict__ timeouts,
    const float* __restrict__ last_values, float* __restrict__ returns,
    float* __restrict__ advantages, int T, int N, float gamma, float lam,
    float* __restrict__ block_moments) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    Moments mom{0.f, 0.f, 0.f};
    if (n < N) {
        float next_v = last_values[n];
        float next_a = 0.f;
        constexpr int CH = 8;
        for (int t_hi = T; t_hi > 0; t_hi -= CH) {
            const int cnt = min(CH, t_hi);
            float r[CH], v[CH];
            uint8_t d[CH], to[CH];
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                if (j < cnt) {
                    const size_t idx = (size_t)(t_hi - 1 - j) * N + n;
                    r[j] = rewards[idx]; v[j] = values[idx];
                    d[j] = dones[idx]; to[j] = timeouts[idx];
                }
            }
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                if (j < cnt) {
                    const size_t idx = (size_t)(t_hi - 1 - j) * N + n;
                    const float nd = d[j] ? 0.f : 1.f;
                    const float rb = to[j] ? fmaf(gamma, v[j], r[j]) : r[j];
                    const float delta = fmaf(gamma * nd, next_v, rb) - v[j];
                    next_a = fmaf(gamma * lam * nd, next_a, delta);
                    next_v = v[j];
                    advantages[idx] = next_a;
                    returns[idx] = next_a + v[j];
                    mom.n += 1.f;
                    const float dm = next_a - mom.mean;
                    mom.mean += dm / mom.n;
                    mom.m2 = fmaf(dm, next_a - mom.mean, mom.m2);
                }
            }
        }
    }
    mom = warp_merge(mom);
    __shared__ Moments wm[kGaeThreads / 32];
    if ((threadIdx.x & 31) == 0) wm[threadIdx.x >> 5] = mom;
    __syncthreads();
    if (threadIdx.x == 0) {
        Moments tot = wm[0];
        for (int w = 1; w < kGaeThreads / 32; ++w) tot = merge(tot, wm[w]);
        block_moments[3 * blockIdx.x + 0] = tot.n;
        block_moments[3 * blockIdx.x + 1] = tot.mean;
        block_moments[3 * blockIdx.x + 2] = tot.m2;
    }
}

// Every block re-derives the global mean / std from the block triples in the same fixed
// order (so all blocks agree bit for bit), then normalises its slice.
__global__ void __launch_bounds__(256) gae_normalize_kernel(float* __restrict__ advantages,
                                                            long long total,
                                                            const float* __restrict__ block_moments,
                                                            int nblocks, int unbiased, float eps) {
    __shared__ float s_mean, s_inv;
    __shared__ Moments s_wm[8];
    {
        // thread i merges triples i, i+256, ... in order; then a fixed shuffle tree per warp and the
        // eight warps in order
        Moments mom{0.f, 0.f, 0.f};
        for (int b = threadIdx.x; b < nblocks; b += 256) {
            Moments o{block_moments[3 * b], block_moments[3 * b + 1], block_moments[3 * b + 2]};
            mom = merge(mom, o);
        }
        mom = warp_merge(mom);
        if ((threadIdx.x & 31) == 0) s_wm[threadIdx.x >> 5] = mom;
        __syncthreads();
        if (threadIdx.x == 0) {
            Moments tot = s_wm[0];
            for (int w = 1; w < 8; ++w) tot = merge(tot, s_wm[w]);
            const float denom = unbiased ? (tot.n - 1.f) : tot.n;
            const float var = denom > 0.f ? tot.m2 / denom : 0.f;
            s_mean = tot.mean;
            s_inv = 1.0f / (sqrtf(var) + eps);
        }
    }
    __syncthreads();
    const float mean = s_mean, inv = s_inv;
    const long long n4 = total / 4;
    float4* a4 = reinterpret_cast<float4*>(advantages);
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n4;
         i += (long long)gridDim.x * blockDim.x) {
        float4 v = a4[i];
        v.x = (v.x - mean) * inv; v.y = (v.y - mean) * inv;
        v.z = (v.z - mean) * inv; v.w = (v.w - mean) * inv;
        a4[i] = v;
    }
    for (long long i = n4 * 4 + blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x)
        advantages[i] = (advantages[i] - mean) * inv;
}

}  // namespace

cudaError_t launch_pad_rows(const float* src, int dim, float* dst, int dst_ld, __nv_bfloat16* dst16,
                            int dst16_ld, int rows, cudaStream_t s) {
    if (rows <= 0) return cudaSuccess;
    const int blocks = std::min((rows + 7) / 8, 148 * 8);      // a warp per row
    LaunchScope scope_("pad_rows", s);
    return launch_chained(pad_rows_kernel, blocks, 256, 0, s, src, dim, dst, dst_ld, dst16, dst16_ld, rows);
}

cudaError_t launch_act_head(const void* Ha, int ldha, const void* Hc, int ldhc, bool bf16_act,
                            const HeadParams& hp, const ActOut& out, int N, uint64_t seed,
                            uint32_t global_step, cudaStream_t s) {
    const int blocks = (N * 32 + 255) / 256;
    const uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
    LaunchScope scope_("act_head", s);
    if (bf16_act)
        return launch_chained(act_head_kernel<__nv_bfloat16>, blocks, 256, 0, s, (const __nv_bfloat16*)Ha, ldha,
                              (const __nv_bfloat16*)Hc, ldhc, hp, out, N, lo, hi, global_step);
    return launch_chained(act_head_kernel<float>, blocks, 256, 0, s, (const float*)Ha, ldha, (const float*)Hc, ldhc,
                          hp, out, N, lo, hi, global_step);
}

cudaError_t launch_value_head(const void* Hc, int ldhc, bool bf16_act, const HeadParams& hp,
                              float* values, int N, cudaStream_t s) {
    const int blocks = (N * 32 + 255) / 256;
    LaunchScope scope_("value_head", s);
    if (bf16_act)
        return launch_chained(value_head_kernel<__nv_bfloat16>, blocks, 256, 0, s, (const __nv_bfloat16*)Hc, ldhc, hp, values, N);
    return launch_chained(value_head_kernel<float>, blocks, 256, 0, s, (const float*)Hc, ldhc, hp, values, N);
}

cudaError_t launch_record_step(const float* rew, const uint8_t* dones, const uint8_t* timeouts,
                               float* s_rew, uint8_t* s_dones, uint8_t* s_timeouts, int N,
                               cudaStream_t s) {
    LaunchScope scope_("record_step", s);
    return launch_chained(record_step_kernel, (N + 255) / 256, 256, 0, s, rew, dones, timeouts, s_rew, s_dones, s_timeouts, N);
}

int gae_scan_blocks(int N) { return (N + kGaeThreads - 1) / kGaeThreads; }

cudaError_t launch_gae(const float* rewards, const float* values, const uint8_t* dones,
                       const uint8_t* timeouts, const float* last_values, float* returns,
                       float* advantages, int T, int N, float gamma, float lam, int normalize,
                       int unbiased, float adv_eps, float* scratch, cudaStream_t s) {
    if (T <= 0 || N <= 0) return cudaSuccess;
    const int blocks = gae_scan_blocks(N);
    cudaError_t e;
    {
        LaunchScope scope_("gae_scan", s);
        gae_scan_kernel<<<blocks, kGaeThreads, 0, s>>>(rewards, values, dones, timeouts, last_values,
                                                       returns, advantages, T, N, gamma, lam, scratch);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess || !normalize) return e;
    const long long total = (long long)T * N;
    const int nb = (int)std::min((total / 4 + 255) / 256 + 1, (long long)(148 * 8));
    LaunchScope scope_("gae_normalize", s);
    gae_normalize_kernel<<<nb, 256, 0, s>>>(advantages, total, scratch, blocks, unbiased, adv_eps);
    return cudaGetLastError();
}

}  // namespace rslrl
