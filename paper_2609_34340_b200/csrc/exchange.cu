// Plan execution over peer memory (Section 5, "Device-resident buffer layout"): the step between vp_pack and vp_unpack.
//
// A rank's staged send buffer holds one contiguous chunk per activation; the chunk of step k goes to the step's
// destination j = lane_dst[k][rank] and lands at j's running receive offset recv_off[k][j].  vp_exchange_put is the
// sender side: plain stores through pointers to the receivers' buffers -- ordinary device memory when the ranks share
// a GPU, peer-mapped memory of other GPUs over NVLink otherwise -- followed, per chunk part, by a system-wide fence and
// an addition to the receiver's device-resident arrival counter.  vp_exchange_wait is the receiver side: a bounded
// wait until the counter has reached the bytes the plan sends this rank, which is what replaces a global barrier.
// Double buffering is the caller's: two receive buffers and two counters per rank, alternated between invocations.
//
// No multicast, no cluster-scope bulk copies: every byte moves by an ordinary 16-byte (or narrower) load and store, so
// the same code is valid for local and for peer destinations.
#include <cuda_runtime.h>

#include "vp_internal.h"

namespace {

constexpr int kPutThreads = 256;

// CTA c copies the bytes [c, c + 1) x total / gridDim.x of the send buffer (rounded to 16 bytes), chunk by chunk.
__global__ void __launch_bounds__(kPutThreads)
exchange_put_kernel(const int32_t* __restrict__ n_steps, const int16_t* __restrict__ lane_dst, const int64_t* __restrict__ send_off,
                    const int64_t* __restrict__ recv_off, int N, int rank, int k_max, const unsigned char* __restrict__ staged,
                    unsigned char* const* __restrict__ recv_bufs, const int64_t* __restrict__ recv_capacity,
                    unsigned long long* const* __restrict__ arrived, int32_t* __restrict__ status) {
    const int K = min(max(*n_steps, 0), k_max);
    const long long total = send_off[(size_t)K * N + rank];
    if (total <= 0) return;
    long long lo = (total * blockIdx.x / gridDim.x) & ~15ll, hi = (total * (blockIdx.x + 1) / gridDim.x) & ~15ll;
    if (blockIdx.x == gridDim.x - 1) hi = total;
    if (lo >= hi) return;
    // the step that holds byte lo: the last k with send_off[k] <= lo (offsets are non-decreasing in k)
    int a = 0, b = K;
    while (b - a > 1) {
        const int m = (a + b) >> 1;
        if (send_off[(size_t)m * N + rank] <= lo) a = m; else b = m;
    }
    for (int k = a; k < K && send_off[(size_t)k * N + rank] < hi; k++) {
        const long long s0 = send_off[(size_t)k * N + rank], s1 = send_off[(size_t)(k + 1) * N + rank];
        const int j = lane_dst[(size_t)k * N + rank];
        if (j < 0 || s1 <= s0) continue;
        const long long from = max(s0, lo), to = min(s1, hi);
        if (from >= to) continue;
        const long long at = recv_off[(size_t)k * N + j] + (from - s0);
        if (at + (to - from) > recv_capacity[j]) {              // would overrun the receiver: not copied, reported
            if (threadIdx.x == 0) atomicOr(status, VP_ST_PACK_CAPACITY);
            continue;
        }
        const unsigned char* src = staged + from;
        unsigned char* dst = recv_bufs[j] + at;
        const long long n = to - from;
        if ((((uintptr_t)src | (uintptr_t)dst) & 15) == 0) {
            const long long vecs = n >> 4;
            long long e = threadIdx.x;
            for (; e + 3 * kPutThreads < vecs; e += 4 * kPutThreads) {      // four 16-byte loads in flight per thread
                const uint4 v0 = ((const uint4*)src)[e], v1 = ((const uint4*)src)[e + kPutThreads];
                const uint4 v2 = ((const uint4*)src)[e + 2 * kPutThreads], v3 = ((const uint4*)src)[e + 3 * kPutThreads];
                ((uint4*)dst)[e] = v0; ((uint4*)dst)[e + kPutThreads] = v1;
                ((uint4*)dst)[e + 2 * kPutThreads] = v2; ((uint4*)dst)[e + 3 * kPutThreads] = v3;
            }
            for (; e < vecs; e += kPutThreads) ((uint4*)dst)[e] = ((const uint4*)src)[e];
            for (long long e = (vecs << 4) + threadIdx.x; e < n; e += kPutThreads) dst[e] = src[e];
        } else {
            for (long long e = threadIdx.x; e < n; e += kPutThreads) dst[e] = src[e];
        }
        if (arrived) {
            // every thread's stores become visible system-wide before the count that announces them
            __threadfence_system();
            __syncthreads();
            if (threadIdx.x == 0 && arrived[j]) atomicAdd_system(arrived[j], (unsigned long long)n);
        }
    }
}

// One thread polls this rank's counter with acquire loads until it holds the expected bytes, at most max_polls times.
__global__ void exchange_wait_kernel(const int32_t* __restrict__ n_steps, const int64_t* __restrict__ recv_off, int N, int rank,
                                     int k_max, const unsigned long long* counter, unsigned long long base,
                                     unsigned int max_polls, int32_t* __restrict__ status) {
    const int K = min(max(*n_steps, 0), k_max);
    const unsigned long long want = base + (unsigned long long)recv_off[(size_t)K * N + rank];
    for (unsigned int p = 0; p <= max_polls; p++) {
        unsigned long long seen;
        asm volatile("ld.acquire.sys.global.u64 %0, [%1];" : "=l"(seen) : "l"(counter) : "memory");
        if (seen >= want) return;
        __nanosleep(200);
    }
    atomicOr(status, VP_ST_EXCHANGE_TIMEOUT);                   // gave up: the caller reads the bit; nothing hangs
}

}  // namespace

extern "C" int vp_exchange_put(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* send_off_b,
                               const int64_t* recv_off_b, int N, int rank, int k_max, const void* staged,
                               void* const* recv_bufs, const int64_t* recv_capacity_bytes, uint64_t* const* arrived,
                               int32_t* status, void* cuda_stream) {
    if (!n_steps_b || !lane_dst_b || !send_off_b || !recv_off_b || !staged || !recv_bufs || !recv_capacity_bytes || !status)
        return VP_E_BAD_ARG;
    if (N <= 0 || N > VP_MAX_N || rank < 0 || rank >= N || k_max <= 0) return VP_E_BAD_ARG;
    static int s_sms[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return VP_E_CUDA;
    int sms = dev >= 0 && dev < 64 ? s_sms[dev] : 0;
    if (!sms) {
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return VP_E_CUDA;
        if (dev >= 0 && dev < 64) s_sms[dev] = sms;
    }
    exchange_put_kernel<<<sms * 8, kPutThreads, 0, (cudaStream_t)cuda_stream>>>(
        n_steps_b, lane_dst_b, send_off_b, recv_off_b, N, rank, k_max, (const unsigned char*)staged,
        (unsigned char* const*)recv_bufs, recv_capacity_bytes, (unsigned long long* const*)arrived, status);
    g_vp_launches++;
    return cudaGetLastError() == cudaSuccess ? VP_OK : VP_E_CUDA;
}

extern "C" int vp_exchange_wait(const int32_t* n_steps_b, const int64_t* recv_off_b, int N, int rank, int k_max,
                                const uint64_t* arrived_counter, uint64_t counter_base, uint32_t max_polls, int32_t* status,
                                void* cuda_stream) {
    if (!n_steps_b || !recv_off_b || !arrived_counter || !status) return VP_E_BAD_ARG;
    if (N <= 0 || N > VP_MAX_N || rank < 0 || rank >= N || k_max <= 0) return VP_E_BAD_ARG;
    exchange_wait_kernel<<<1, 1, 0, (cudaStream_t)cuda_stream>>>(n_steps_b, recv_off_b, N, rank, k_max,
                                                                 (const unsigned long long*)arrived_counter,
                                                                 (unsigned long long)counter_base, max_polls, status);
    g_vp_launches++;
    return cudaGetLastError() == cudaSuccess ? VP_OK : VP_E_CUDA;
}
