// Guarded device allocations and the index-fault registry of the -DRSLRL_DEBUG build (see guard.h).
#include "guard.h"
#include "../../include/rslrl_b200.h"
#include <mutex>
#include <unordered_map>
#include <vector>
#include <stdint.h>

namespace rslrl {

namespace {

constexpr size_t kGuardBytes = 256;                 // keeps the 256-byte alignment cudaMalloc gives
constexpr uint32_t kGuardWord = 0xA5C35A3Cu;

struct Registry {
    std::mutex mu;
    std::unordered_map<void*, size_t> live;         // user pointer -> user bytes (rounded up to 256)
    std::vector<int (*)()> readers;
    int damaged_at_free = 0;                        // guard regions found damaged when their allocation was freed
};
Registry& registry() { static Registry r; return r; }

__global__ void guard_fill_kernel(uint32_t* g) { g[threadIdx.x] = kGuardWord; }

// block b checks guard region b (kGuardBytes / 4 words, one per thread)
__global__ void guard_check_kernel(const uint32_t* const* guards, int* damaged) {
    const uint32_t* g = guards[blockIdx.x];
    const int bad = __syncthreads_or(g[threadIdx.x] != kGuardWord);
    if (threadIdx.x == 0 && bad) atomicAdd(damaged, 1);
}

}  // namespace

#ifdef RSLRL_DEBUG

cudaError_t guarded_malloc(void** p, size_t bytes) {
    const size_t user = (bytes + kGuardBytes - 1) / kGuardBytes * kGuardBytes;
    char* base = nullptr;
    cudaError_t e = cudaMalloc((void**)&base, user + 2 * kGuardBytes);
    if (e != cudaSuccess) return e;
    guard_fill_kernel<<<1, kGuardBytes / 4>>>((uint32_t*)base);
    guard_fill_kernel<<<1, kGuardBytes / 4>>>((uint32_t*)(base + kGuardBytes + user));
    if ((e = cudaDeviceSynchronize()) != cudaSuccess) { cudaFree(base); return e; }
    *p = base + kGuardBytes;
    Registry& r = registry();
    std::lock_guard<std::mutex> lock(r.mu);
    r.live[*p] = user;
    return cudaSuccess;
}

cudaError_t guarded_free(void* p) {
    if (!p) return cudaSuccess;
    Registry& r = registry();
    size_t user = 0; bool known = false;
    {
        std::lock_guard<std::mutex> lock(r.mu);
        auto it = r.live.find(p);
        if (it != r.live.end()) { user = it->second; known = true; r.live.erase(it); }
    }
    if (known) {                                    // the guards of a freed allocation are looked at one last time
        uint32_t h[2][kGuardBytes / 4];
        int bad = 0;
        if (cudaMemcpy(h[0], (char*)p - kGuardBytes, kGuardBytes, cudaMemcpyDeviceToHost) == cudaSuccess &&
            cudaMemcpy(h[1], (char*)p + user, kGuardBytes, cudaMemcpyDeviceToHost) == cudaSuccess) {
            for (int g = 0; g < 2; ++g) {
                bool dmg = false;
                for (size_t i = 0; i < kGuardBytes / 4; ++i) dmg |= h[g][i] != kGuardWord;
                bad += dmg;
            }
        }
        if (bad) { std::lock_guard<std::mutex> lock(r.mu); r.damaged_at_free += bad; }
    }
    return cudaFree((char*)p - kGuardBytes);
}

cudaError_t guarded_check(int* damaged) {
    *damaged = 0;
    std::vector<const uint32_t*> guards;
    int at_free = 0;
    {
        Registry& r = registry();
        std::lock_guard<std::mutex> lock(r.mu);
        at_free = r.damaged_at_free;
        for (const auto& kv : r.live) {
            guards.push_back((const uint32_t*)((const char*)kv.first - kGuardBytes));
            guards.push_back((const uint32_t*)((const char*)kv.first + kv.second));
        }
    }
    *damaged = at_free;
    if (guards.empty()) return cudaSuccess;
    const uint32_t** d_list = nullptr; int* d_count = nullptr;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMalloc((void**)&d_list, guards.size() * sizeof(void*));
    if (e == cudaSuccess) e = cudaMalloc((void**)&d_count, sizeof(int));
    if (e == cudaSuccess) e = cudaMemcpy(d_list, guards.data(), guards.size() * sizeof(void*), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(d_count, 0, sizeof(int));
    if (e == cudaSuccess) {
        guard_check_kernel<<<(unsigned)guards.size(), kGuardBytes / 4>>>(d_list, d_count);
        int live_damaged = 0;
        e = cudaMemcpy(&live_damaged, d_count, sizeof(int), cudaMemcpyDeviceToHost);
        *damaged = at_free + live_damaged;
    }
    cudaFree(d_list); cudaFree(d_count);
    return e;
}

#else

cudaError_t guarded_malloc(void** p, size_t bytes) { return cudaMalloc(p, bytes); }
cudaError_t guarded_free(void* p) { return cudaFree(p); }
cudaError_t guarded_check(int* damaged) { *damaged = 0; return cudaDeviceSynchronize(); }

#endif

void register_index_fault_reader(int (*reader)()) {
    Registry& r = registry();
    std::lock_guard<std::mutex> lock(r.mu);
    r.readers.push_back(reader);
}

int take_index_faults() {
    std::vector<int (*)()> readers;
    {
        Registry& r = registry();
        std::lock_guard<std::mutex> lock(r.mu);
        readers = r.readers;
    }
    int worst = 0;
    for (auto fn : readers) { const int v = fn(); if (v > worst) worst = v; }
    return worst;
}

}  // namespace rslrl

extern "C" rslrl_status rslrl_debug_report(int32_t* h_debug_build, int32_t* h_damaged_guards, int32_t* h_index_fault) {
#ifdef RSLRL_DEBUG
    const int32_t is_debug = 1;
#else
    const int32_t is_debug = 0;
#endif
    if (h_debug_build) *h_debug_build = is_debug;
    int damaged = 0;
    if (rslrl::guarded_check(&damaged) != cudaSuccess) return RSLRL_ERR_CUDA;
    if (h_damaged_guards) *h_damaged_guards = damaged;
    if (h_index_fault) *h_index_fault = rslrl::take_index_faults();
    return RSLRL_OK;
}
