// Optional per-kernel timing: CUDA events recorded on the caller's stream around the library's
// own launches, so a benchmark can report the duration of one kernel inside a longer step.
#include <cuda_runtime.h>

#include <vector>

#include "vp_internal.h"

namespace {
constexpr int kKinds = 4;
bool g_on = false;
std::vector<cudaEvent_t> g_begin[kKinds], g_end[kKinds];
std::vector<cudaEvent_t> g_pool;       // events handed back by vp_profile_read, reused by later marks
}  // namespace

void vp_prof_mark(int kind, int edge, cudaStream_t stream) {
    if (!g_on || kind < 0 || kind >= kKinds) return;
    cudaEvent_t ev;
    if (!g_pool.empty()) {
        ev = g_pool.back();
        g_pool.pop_back();
    } else if (cudaEventCreate(&ev) != cudaSuccess) {
        return;
    }
    cudaEventRecord(ev, stream);
    (edge ? g_end : g_begin)[kind].push_back(ev);
}

extern "C" int vp_profile_enable(int on) {
    g_on = on != 0;
    return VP_OK;
}

extern "C" int vp_profile_read(int kind, double* total_ms, int64_t* launches) {
    if (kind < 0 || kind >= kKinds || !total_ms || !launches) return VP_E_BAD_ARG;
    double total = 0;
    int64_t n = 0;
    int rc = VP_OK;
    const size_t pairs = g_begin[kind].size() < g_end[kind].size() ? g_begin[kind].size() : g_end[kind].size();
    for (size_t i = 0; i < pairs; i++) {
        float ms = 0;
        if (cudaEventSynchronize(g_end[kind][i]) != cudaSuccess ||
            cudaEventElapsedTime(&ms, g_begin[kind][i], g_end[kind][i]) != cudaSuccess)
            rc = VP_E_CUDA;
        else { total += ms; n++; }
    }
    for (cudaEvent_t e : g_begin[kind]) g_pool.push_back(e);
    for (cudaEvent_t e : g_end[kind]) g_pool.push_back(e);
    g_begin[kind].clear();
    g_end[kind].clear();
    *total_ms = total;
    *launches = n;
    return rc;
}
