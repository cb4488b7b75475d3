// Launch accounting: every kernel launch of the library goes through a LaunchScope, which
// counts it and, while profiling is switched on, brackets it with a pair of CUDA events on the
// launching stream.  A FamilyScope brackets a run of launches of one family that follow each other
// with programmatic dependent launch (an event between them would take the overlap away): one pair
// for the run, every launch inside counted.  rslrl_profile_report turns the pairs into per-family totals.
#include "../../include/rslrl_b200.h"
#include "kernels.h"

#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <vector>

namespace rslrl {

namespace {
std::atomic<uint64_t> g_launches{0};
std::atomic<int> g_profiling{0};
std::mutex g_mutex;
struct Pair { const char* name; cudaEvent_t a, b; int launches; };
thread_local int t_family_slot = -1;   // the open FamilyScope of this thread, if it records
std::vector<Pair> g_pairs;          // recorded in this profiling session
std::vector<cudaEvent_t> g_pool;    // events ready for reuse

cudaEvent_t take_event() {
    if (!g_pool.empty()) { cudaEvent_t e = g_pool.back(); g_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}
}  // namespace

// RSLRL_SERIAL_LAUNCHES=1 in the environment switches programmatic dependent launch off.
bool chained_launches_enabled() {
    static const bool on = [] { const char* v = std::getenv("RSLRL_SERIAL_LAUNCHES"); return !(v && v[0] == '1'); }();
    return on;
}

LaunchScope::LaunchScope(const char* n, cudaStream_t s) : name(n), stream(s), slot(-1) {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!g_profiling.load(std::memory_order_relaxed)) return;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (t_family_slot >= 0 && t_family_slot < (int)g_pairs.size()) { g_pairs[t_family_slot].launches++; return; }
    Pair p{n, take_event(), take_event(), 1};
    if (!p.a || !p.b) return;
    cudaEventRecord(p.a, s);
    slot = (int)g_pairs.size();
    g_pairs.push_back(p);
}

LaunchScope::~LaunchScope() {
    if (slot < 0) return;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (slot < (int)g_pairs.size()) cudaEventRecord(g_pairs[slot].b, stream);
}

FamilyScope::FamilyScope(const char* n, cudaStream_t s) : stream(s), slot(-1) {
    if (!g_profiling.load(std::memory_order_relaxed) || t_family_slot >= 0) return;
    std::lock_guard<std::mutex> lock(g_mutex);
    Pair p{n, take_event(), take_event(), 0};
    if (!p.a || !p.b) return;
    cudaEventRecord(p.a, s);
    slot = (int)g_pairs.size();
    g_pairs.push_back(p);
    t_family_slot = slot;
}

FamilyScope::~FamilyScope() {
    if (slot < 0) return;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (slot < (int)g_pairs.size()) cudaEventRecord(g_pairs[slot].b, stream);
    t_family_slot = -1;
}

}  // namespace rslrl

using namespace rslrl;

extern "C" {

uint64_t rslrl_kernel_launch_count(void) { return g_launches.load(); }

rslrl_status rslrl_profile_enable(int32_t on) {
    g_profiling.store(on ? 1 : 0);
    return RSLRL_OK;
}

rslrl_status rslrl_profile_report(char* h_text, size_t capacity) {
    if (!h_text || capacity == 0) return RSLRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    struct Acc { long long count = 0; double ms = 0.0; };
    std::map<std::string, Acc> acc;
    cudaError_t err = cudaSuccess;
    for (Pair& p : g_pairs) {
        cudaError_t e = cudaEventSynchronize(p.b);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, p.a, p.b);
        if (e != cudaSuccess) err = e;
        else { Acc& a = acc[p.name]; a.count += p.launches; a.ms += ms; }
        g_pool.push_back(p.a); g_pool.push_back(p.b);
    }
    g_pairs.clear();
    t_family_slot = -1;
    std::string out;
    char line[160];
    for (const auto& kv : acc) {
        snprintf(line, sizeof line, "%s %lld %.6f\n", kv.first.c_str(), kv.second.count, kv.second.ms);
        out += line;
    }
    if (out.size() + 1 > capacity) return RSLRL_ERR_UNSUPPORTED;
    memcpy(h_text, out.c_str(), out.size() + 1);
    return err == cudaSuccess ? RSLRL_OK : RSLRL_ERR_CUDA;
}

}  // extern "C"
