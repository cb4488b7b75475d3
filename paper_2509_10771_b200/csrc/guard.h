// Debug aids of the -DRSLRL_DEBUG build: every device allocation of the library sits between two guard
// regions of a fixed byte pattern, and kernels that index through data they read (shuffled row numbers,
// selected observation entries) check the index first.  Neither ever traps: a bad index is replaced by 0 and
// recorded in a device flag, a damaged guard is found by rslrl_debug_report, which the host calls between
// steps.  In the normal build guarded_malloc / guarded_free are cudaMalloc / cudaFree and the checks compile
// to nothing.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace rslrl {

cudaError_t guarded_malloc(void** p, size_t bytes);
cudaError_t guarded_free(void* p);
// Guard regions whose pattern is damaged, over all live allocations (synchronises the device).
cudaError_t guarded_check(int* damaged);
// A translation unit with index checks registers the function that reads and clears its flag.
void register_index_fault_reader(int (*reader)());
int take_index_faults();      // largest code recorded by any translation unit since the last call (0 = none)

}  // namespace rslrl

// A .cu file that defines RSLRL_INDEX_CHECKS before including this header gets checked_index(i, n, code):
// i if i < n; otherwise (debug build only) 0, with `code` recorded in that file's device flag.
#if defined(RSLRL_INDEX_CHECKS) && defined(__CUDACC__)
#ifdef RSLRL_DEBUG
namespace {
__device__ int g_index_fault;
int read_index_fault_() {
    int v = 0; const int zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_index_fault, sizeof(int)) != cudaSuccess) return 0;
    cudaMemcpyToSymbol(g_index_fault, &zero, sizeof(int));
    return v;
}
const int index_fault_reader_registered_ = (rslrl::register_index_fault_reader(&read_index_fault_), 0);
__device__ __forceinline__ uint32_t checked_index(uint32_t i, uint32_t n, int code) {
    if (i < n) return i;
    atomicMax(&g_index_fault, code);
    return 0u;
}
}  // namespace
#else
namespace {
__device__ __forceinline__ uint32_t checked_index(uint32_t i, uint32_t, int) { return i; }
}  // namespace
#endif
#endif
