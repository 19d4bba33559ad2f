// Peak-rate probes for the limits that bound the scheduler kernels: issue rate of plain 32-bit and 64-bit integer
// add / min (the arithmetic of Eq. 6 - 10), and shared-memory load bandwidth (credits and score tables).  A benchmark
// launches one, times it with events on its own stream and divides the returned operation count by the time; the
// result is the denominator of the scheduler's roofline fraction on the GPU at hand, at the clock it then ran at.
#include <cuda_runtime.h>

#include "vp_internal.h"

namespace {

constexpr int kChains = 8;        // independent dependency chains per thread
constexpr int kUnroll = 16;       // operations per chain and loop iteration

// x = min(x + a, b): one add and one min per step, kChains chains in flight per thread
template <typename T>
__global__ void __launch_bounds__(256) int_issue_kernel(int iters, T a, T b, unsigned long long* sink) {
    T x[kChains];
#pragma unroll
    for (int c = 0; c < kChains; c++) x[c] = (T)(threadIdx.x + c);
    for (int it = 0; it < iters; it++) {
#pragma unroll
        for (int u = 0; u < kUnroll; u++)
#pragma unroll
            for (int c = 0; c < kChains; c++) {
                const T s = x[c] + a;
                x[c] = s < b ? s : b;
            }
    }
    T acc = 0;
#pragma unroll
    for (int c = 0; c < kChains; c++) acc += x[c];
    if (acc == (T)0x7fffffff) *sink = (unsigned long long)acc;          // never true in practice: keeps the chains alive
}

// conflict-free 32-bit (or 64-bit) shared-memory loads: lane l reads word (base + l) of a rotating window
template <typename T>
__global__ void __launch_bounds__(256) smem_load_kernel(int iters, unsigned long long* sink) {
    __shared__ T buf[4096];
    for (int i = threadIdx.x; i < 4096; i += blockDim.x) buf[i] = (T)i;
    __syncthreads();
    T acc[kChains];
#pragma unroll
    for (int c = 0; c < kChains; c++) acc[c] = 0;
    unsigned at = threadIdx.x;
    for (int it = 0; it < iters; it++) {
#pragma unroll
        for (int u = 0; u < kUnroll; u++) {
#pragma unroll
            for (int c = 0; c < kChains; c++) acc[c] += buf[(at + 32u * (unsigned)c) & 4095u];
            at += 256u;
        }
    }
    T s = 0;
#pragma unroll
    for (int c = 0; c < kChains; c++) s += acc[c];
    if (s == (T)0x7ffffff1) *sink = (unsigned long long)s;
}

}  // namespace

extern "C" int vp_microbench(int kind, int iters, void* sink_device, int64_t* units_per_launch, void* cuda_stream) {
    if (kind < 0 || kind > 3 || iters <= 0 || !sink_device || !units_per_launch) return VP_E_BAD_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return VP_E_CUDA;
    const int threads = 256, grid = sms * 8;                             // 2048 threads per SM: every warp slot taken
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned long long* sink = (unsigned long long*)sink_device;
    const int64_t per_thread = (int64_t)iters * kUnroll * kChains;
    switch (kind) {
        case 0:                                                          // 32-bit add + min: 2 operations per step
            int_issue_kernel<uint32_t><<<grid, threads, 0, stream>>>(iters, 3u, 0x7ffffff0u, sink);
            *units_per_launch = 2 * per_thread * threads * grid;
            break;
        case 1:                                                          // 64-bit add + min
            int_issue_kernel<int64_t><<<grid, threads, 0, stream>>>(iters, (int64_t)3, (int64_t)1 << 60, sink);
            *units_per_launch = 2 * per_thread * threads * grid;
            break;
        case 2:                                                          // bytes of 32-bit shared-memory loads
            smem_load_kernel<uint32_t><<<grid, threads, 0, stream>>>(iters, sink);
            *units_per_launch = 4 * per_thread * threads * grid;
            break;
        default:                                                         // bytes of 64-bit shared-memory loads
            smem_load_kernel<unsigned long long><<<grid, threads, 0, stream>>>(iters, sink);
            *units_per_launch = 8 * per_thread * threads * grid;
            break;
    }
    g_vp_launches++;
    return cudaGetLastError() == cudaSuccess ? VP_OK : VP_E_CUDA;
}

// Write-only bandwidth probe: one cudaMemsetAsync over a caller-owned device buffer (the pack is 88 % writes, so the
// write-only rate is quoted beside the copy rate).
extern "C" int vp_memset_probe(void* device_buffer, size_t bytes, void* cuda_stream) {
    if (!device_buffer || !bytes) return VP_E_BAD_ARG;
    return cudaMemsetAsync(device_buffer, 0, bytes, (cudaStream_t)cuda_stream) == cudaSuccess ? VP_OK : VP_E_CUDA;
}
