// FP32 matrix products on the FP32 pipes (the RSLRL_FP32 mode, and every product that is too
// small or too ragged for the tensor-core kernels): register-tiled SIMT GEMM with fused
// bias+ELU, ELU-derivative and split-partial epilogues, plus a column-sum kernel for the
// bias gradients.
#include "common.cuh"
#include "kernels.h"
#include <algorithm>

namespace rslrl {

namespace {

constexpr int BK = 8;
constexpr int NT = 256;   // threads per block, arranged 16 x 16

template <int BM, int BN, bool TA, bool TB, int EPI>
__global__ void __launch_bounds__(NT) sgemm_kernel(const GemmBatch batch) {
    constexpr int TM = BM / 16, TN = BN / 16;
    // z = problem * max_splits + split
    int max_splits = batch.p[0].splits;
    for (int i = 1; i < batch.count; ++i) max_splits = max(max_splits, batch.p[i].splits);
    const int prob = blockIdx.z / max_splits;
    const int split = blockIdx.z % max_splits;
    const GemmProblem& g = batch.p[prob];
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    if (split >= g.splits || m0 >= g.M || n0 >= g.Cn) return;
    const int k_begin = split * g.kchunk;
    const int k_end = min(g.K, k_begin + g.kchunk);

    __shared__ __align__(16) float As[2][BK][BM];
    __shared__ __align__(16) float Bs[2][BK][BN];

    const int tid = threadIdx.x;
    const int ty = tid / 16, tx = tid % 16;

    constexpr int A_VEC = BM * BK / 4, B_VEC = BN * BK / 4;
    constexpr int A_PER = (A_VEC + NT - 1) / NT, B_PER = (B_VEC + NT - 1) / NT;
    float4 ra[A_PER], rb[B_PER];

    auto load_tiles = [&](int k0) {
#pragma unroll
        for (int it = 0; it < A_PER; ++it) {
            const int i = tid + it * NT;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < A_VEC) {
                if (!TA) {          // A[m][k], k contiguous
                    const int m = m0 + i / 2, k = k0 + (i % 2) * 4;
                    if (m < g.M && k < k_end) {
                        v = *reinterpret_cast<const float4*>(g.A + (size_t)m * g.lda + k);
                        if (k + 1 >= k_end) v.y = 0.f;
                        if (k + 2 >= k_end) v.z = 0.f;
                        if (k + 3 >= k_end) v.w = 0.f;
                    }
                } else {            // A[k][m], m contiguous
                    const int k = k0 + i / (BM / 4), m = m0 + (i % (BM / 4)) * 4;
                    if (k < k_end && m < g.M) {
                        v = *reinterpret_cast<const float4*>(g.A + (size_t)k * g.lda + m);
                        if (m + 1 >= g.M) v.y = 0.f;
                        if (m + 2 >= g.M) v.z = 0.f;
                        if (m + 3 >= g.M) v.w = 0.f;
                    }
                }
            }
            ra[it] = v;
        }
#pragma unroll
        for (int it = 0; it < B_PER; ++it) {
            const int i = tid + it * NT;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < B_VEC) {
                if (!TB) {          // B[k][n], n contiguous
                    const int k = k0 + i / (BN / 4), n = n0 + (i % (BN / 4)) * 4;
                    if (k < k_end && n < g.N) {
                        v = *reinterpret_cast<const float4*>(g.B + (size_t)k * g.ldb + n);
                        if (n + 1 >= g.N) v.y = 0.f;
                        if (n + 2 >= g.N) v.z = 0.f;
                        if (n + 3 >= g.N) v.w = 0.f;
                    }
                } else {            // B[n][k], k contiguous
                    const int n = n0 + i / 2, k = k0 + (i % 2) * 4;
                    if (n < g.N && k < k_end) {
                        v = *reinterpret_cast<const float4*>(g.B + (size_t)n * g.ldb + k);
                        if (k + 1 >= k_end) v.y = 0.f;
                        if (k + 2 >= k_end) v.z = 0.f;
                        if (k + 3 >= k_end) v.w = 0.f;
                    }
                }
            }
            rb[it] = v;
        }
    };
    auto store_tiles = [&](int buf) {
#pragma unroll
        for (int it = 0; it < A_PER; ++it) {
            const int i = tid + it * NT;
            if (i < A_VEC) {
                if (!TA) {
                    const int m = i / 2, k = (i % 2) * 4;
                    As[buf][k + 0][m] = ra[it].x; As[buf][k + 1][m] = ra[it].y;
                    As[buf][k + 2][m] = ra[it].z; As[buf][k + 3][m] = ra[it].w;
                } else {
                    const int k = i / (BM / 4), m = (i % (BM / 4)) * 4;
                    *reinterpret_cast<float4*>(&As[buf][k][m]) = ra[it];
                }
            }
        }
#pragma unroll
        for (int it = 0; it < B_PER; ++it) {
            const int i = tid + it * NT;
            if (i < B_VEC) {
                if (!TB) {
                    const int k = i / (BN / 4), n = (i % (BN / 4)) * 4;
                    *reinterpret_cast<float4*>(&Bs[buf][k][n]) = rb[it];
                } else {
                    const int n = i / 2, k = (i % 2) * 4;
                    Bs[buf][k + 0][n] = rb[it].x; Bs[buf][k + 1][n] = rb[it].y;
                    Bs[buf][k + 2][n] = rb[it].z; Bs[buf][k + 3][n] = rb[it].w;
                }
            }
        }
    };

    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    // The K range of a split starts on a multiple of kchunk, itself a multiple of 8 floats, so
    // the float4 loads stay aligned.
    int buf = 0;
    if (k_begin < k_end) {
        load_tiles(k_begin);
        store_tiles(0);
    }
    __syncthreads();
    for (int k0 = k_begin; k0 < k_end; k0 += BK) {
        const bool more = k0 + BK < k_end;
        if (more) load_tiles(k0 + BK);
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM], b[TN];
#pragma unroll
            for (int i = 0; i < TM; i += 4) {
                const float4 v = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4 + i * 16]);
                a[i] = v.x; a[i + 1] = v.y; a[i + 2] = v.z; a[i + 3] = v.w;
            }
#pragma unroll
            for (int j = 0; j < TN; j += 4) {
                const float4 v = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4 + j * 16]);
                b[j] = v.x; b[j + 1] = v.y; b[j + 2] = v.z; b[j + 3] = v.w;
            }
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (more) {
            store_tiles(buf ^ 1);
            __syncthreads();
            buf ^= 1;
        }
    }

    // Thread (ty,tx) owns rows m0 + ty*4 + (i/4)*64 + i%4 and columns n0 + tx*4 + (j/4)*64 + j%4.
    float* C = g.C + (size_t)split * g.split_stride;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int m = m0 + ty * 4 + (i / 4) * 64 + (i % 4);
        if (m >= g.M) continue;
#pragma unroll
        for (int j = 0; j < TN; j += 4) {
            const int n = n0 + tx * 4 + (j / 4) * 64;
            if (n >= g.Cn) continue;
            float o[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float v = acc[i][j + q];
                const int nn = n + q;
                if (nn >= g.N) {
                    v = 0.f;
                } else if (EPI == EPI_BIAS_ELU) {
                    v = elu_f(v + g.bias[nn], batch.alpha);
                } else if (EPI == EPI_BIAS) {
                    v = v + g.bias[nn];
                } else if (EPI == EPI_DELU) {
                    v = v * elu_grad_from_h(g.aux[(size_t)m * g.ldaux + nn], batch.alpha);
                }
                o[q] = v;
            }
            // Cn is a multiple of 4 and ldc >= Cn: the float4 store stays inside the row.
            *reinterpret_cast<float4*>(C + (size_t)m * g.ldc + n) = make_float4(o[0], o[1], o[2], o[3]);
        }
    }
}

template <int BM, int BN>
cudaError_t launch_tiles(const GemmBatch& b, bool ta, bool tb, int epi, cudaStream_t s) {
    int mt = 0, nt = 0, sp = 1;
    for (int i = 0; i < b.count; ++i) {
        mt = std::max(mt, (b.p[i].M + BM - 1) / BM);
        nt = std::max(nt, (b.p[i].Cn + BN - 1) / BN);
        sp = std::max(sp, b.p[i].splits);
    }
    dim3 grid(nt, mt, sp * b.count);
#define RSLRL_SGEMM_CASE(TA_, TB_, EPI_, NAME_)                                                \
    if (ta == TA_ && tb == TB_ && epi == EPI_) {                                          \
        LaunchScope scope_(NAME_, s);                                                     \
        sgemm_kernel<BM, BN, TA_, TB_, EPI_><<<grid, NT, 0, s>>>(b);                      \
        return cudaGetLastError();                                                        \
    }
    RSLRL_SGEMM_CASE(false, false, EPI_BIAS_ELU, "sgemm_fwd")
    RSLRL_SGEMM_CASE(false, false, EPI_BIAS, "sgemm_fwd_linear")
    RSLRL_SGEMM_CASE(false, true, EPI_DELU, "sgemm_dgrad")
    RSLRL_SGEMM_CASE(false, true, EPI_PLAIN, "sgemm_dgrad_plain")
    RSLRL_SGEMM_CASE(true, false, EPI_PLAIN, "sgemm_wgrad")
#undef RSLRL_SGEMM_CASE
    return cudaErrorInvalidValue;
}

}  // namespace

// Tile shape: the one with the smallest estimated time.  The SM that gets the most tiles decides the time of a
// launch, so the estimate is ceil(tiles / SMs) x tile area / efficiency; the efficiencies (share of the FMA
// rate a tile shape can reach: smaller tiles read more shared memory per multiply-add) are measured ratios.
cudaError_t launch_sgemm(const GemmBatch& b, bool ta, bool tb, int epi, cudaStream_t s) {
    auto cost = [&](int bm, int bn, double eff) {
        long long tiles = 0;
        for (int i = 0; i < b.count; ++i)
            tiles += (long long)((b.p[i].M + bm - 1) / bm) * ((b.p[i].Cn + bn - 1) / bn) * b.p[i].splits;
        return (double)((tiles + 147) / 148) * bm * bn / eff;
    };
    const double c128 = cost(128, 128, 1.0), c12864 = cost(128, 64, 0.85), c64 = cost(64, 64, 0.55);
    if (c128 <= c12864 && c128 <= c64) return launch_tiles<128, 128>(b, ta, tb, epi, s);
    if (c12864 <= c64) return launch_tiles<128, 64>(b, ta, tb, epi, s);
    return launch_tiles<64, 64>(b, ta, tb, epi, s);
}

// ---------------------------------------------------------------------------------------
// Column sums over a split of the rows (bias gradients).  grid = (ceil(n/64), splits, count);
// a block of 1024 threads covers 64 columns (16 column quads) with 64 row lanes, so that the
// whole machine is busy even when there are only a few splits.  The 64 row-lane partials of a
// column are added in a fixed order: the result does not depend on scheduling.
// ---------------------------------------------------------------------------------------
namespace {
constexpr int kCsQuads = 16, kCsLanes = 64, kCsCols = 4 * kCsQuads;

__device__ __forceinline__ float4 load_quad(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load_quad(const __nv_bfloat16* p) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.y));
    return make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ void add4(float4& s, const float4 a) { s.x += a.x; s.y += a.y; s.z += a.z; s.w += a.w; }

template <typename T>
__global__ void __launch_bounds__(kCsQuads * kCsLanes) colsum_kernel(const ColsumBatch b) {
    const ColsumProblem& p = b.p[blockIdx.z];
    __shared__ float4 part[kCsLanes][kCsQuads];
    if (blockIdx.x * kCsCols >= p.n) return;
    const int quad = threadIdx.x % kCsQuads, rl = threadIdx.x / kCsQuads;
    const int n = blockIdx.x * kCsCols + 4 * quad;             // leading dimensions are multiples of 4
    const int chunk = (p.rows + b.splits - 1) / b.splits;
    const int r0 = blockIdx.y * chunk, r1 = min(p.rows, r0 + chunk);
    const T* X = reinterpret_cast<const T*>(p.X);
    float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0, s2 = s0, s3 = s0;
    if (n < p.ld) {
        int r = r0 + rl;
        for (; r + 3 * kCsLanes < r1; r += 4 * kCsLanes) {
            const float4 a0 = load_quad(X + (size_t)r * p.ld + n);
            const float4 a1 = load_quad(X + (size_t)(r + kCsLanes) * p.ld + n);
            const float4 a2 = load_quad(X + (size_t)(r + 2 * kCsLanes) * p.ld + n);
            const float4 a3 = load_quad(X + (size_t)(r + 3 * kCsLanes) * p.ld + n);
            add4(s0, a0); add4(s1, a1); add4(s2, a2); add4(s3, a3);
        }
        for (; r < r1; r += kCsLanes) add4(s0, load_quad(X + (size_t)r * p.ld + n));
    }
    part[rl][quad] = make_float4((s0.x + s1.x) + (s2.x + s3.x), (s0.y + s1.y) + (s2.y + s3.y),
                                 (s0.z + s1.z) + (s2.z + s3.z), (s0.w + s1.w) + (s2.w + s3.w));
    __syncthreads();
    if (threadIdx.x < kCsCols) {
        const int c = threadIdx.x;                 // column within the block
        const float* flat = reinterpret_cast<const float*>(&part[0][0]);
        float t = 0.f;
        for (int l = 0; l < kCsLanes; ++l) t += flat[l * kCsCols + c];
        const int col = blockIdx.x * kCsCols + c;
        if (col < p.n) p.out[(size_t)blockIdx.y * b.split_stride + col] = t;
    }
}
}  // namespace

cudaError_t launch_colsum(const ColsumBatch& b, cudaStream_t s) {
    if (b.count <= 0) return cudaSuccess;
    int nmax = 0;
    for (int i = 0; i < b.count; ++i) nmax = std::max(nmax, b.p[i].n);
    dim3 grid((nmax + kCsCols - 1) / kCsCols, b.splits, b.count);
    LaunchScope scope_("colsum", s);
    if (b.is_bf16) colsum_kernel<__nv_bfloat16><<<grid, kCsQuads * kCsLanes, 0, s>>>(b);
    else colsum_kernel<float><<<grid, kCsQuads * kCsLanes, 0, s>>>(b);
    return cudaGetLastError();
}

}  // namespace rslrl
