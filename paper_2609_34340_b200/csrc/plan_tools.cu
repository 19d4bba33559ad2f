// Around the scheduler: the demand matrix from routing indices (its input side) and the modeled
// completion time of a plan, Eq. (2) (its quality measure).
#include <cuda_runtime.h>

#include "vp_internal.h"

namespace {

// One warp per group of four activations: slowest lane (bytes x rate_lcm / bw of its path), then lambda * rate_lcm + that,
// summed over the activations of the matrix.  Integer throughout, so the order of the sums does not matter.
__global__ void __launch_bounds__(256)
plan_time_kernel(const uint32_t* __restrict__ inst_wdiv, int n_inst, int64_t W, int N, int k_max, int B,
                 const int32_t* __restrict__ n_steps, const uint16_t* __restrict__ lane_inst,
                 const int64_t* __restrict__ lane_bytes, int64_t lambda_ns, int64_t* __restrict__ time_xw) {
    __shared__ unsigned long long s_sum;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    for (int b = blockIdx.x; b < B; b += gridDim.x) {
        if (threadIdx.x == 0) s_sum = 0;
        __syncthreads();
        int K = n_steps[b];
        K = K < 0 ? 0 : (K > k_max ? k_max : K);
        unsigned long long acc = 0;
        // four activations per warp step: their loads are independent, so they overlap
        for (int k0 = warp * 4; k0 < K; k0 += n_warps * 4) {
            int64_t tmax[4] = {0, 0, 0, 0};
#pragma unroll
            for (int u = 0; u < 4; u++) {
                if (k0 + u >= K) continue;
                const size_t row = ((size_t)b * k_max + k0 + u) * N;
                for (int i = lane; i < N; i += 32) {
                    const int64_t x = lane_bytes[row + i];
                    const unsigned id = lane_inst[row + i];
                    if (x > 0 && id < (unsigned)n_inst) {
                        const int64_t t = x * (int64_t)inst_wdiv[id];
                        tmax[u] = t > tmax[u] ? t : tmax[u];
                    }
                }
            }
#pragma unroll
            for (int o = 16; o; o >>= 1)
#pragma unroll
                for (int u = 0; u < 4; u++) {
                    const int64_t other = __shfl_xor_sync(0xffffffffu, tmax[u], o);
                    tmax[u] = other > tmax[u] ? other : tmax[u];
                }
#pragma unroll
            for (int u = 0; u < 4; u++)
                if (k0 + u < K) acc += (unsigned long long)(lambda_ns * W + tmax[u]);
        }
        if (lane == 0 && acc) atomicAdd(&s_sum, acc);
        __syncthreads();
        if (threadIdx.x == 0) time_xw[b] = (int64_t)s_sum;
        __syncthreads();
    }
}

// Histogram of (source rank, destination rank) pairs of routed copies.  Block = one slice of one source
// rank's copies; per-block counts in shared memory, then one atomic add per non-empty destination.
__global__ void __launch_bounds__(256)
demand_kernel(const int32_t* __restrict__ idx, int n_src, long long per_src, int experts_per_rank, int N, int src0,
              long long row_bytes, int slices, int64_t* __restrict__ demand_rows, int32_t* __restrict__ status) {
    __shared__ unsigned int cnt[VP_MAX_N];
    const int s = blockIdx.x / slices, slice = blockIdx.x % slices;
    if (s >= n_src) return;
    for (int j = threadIdx.x; j < N; j += blockDim.x) cnt[j] = 0;
    __syncthreads();
    const long long lo = per_src * slice / slices, hi = per_src * (slice + 1) / slices;
    bool bad = false;
    for (long long e = lo + threadIdx.x; e < hi; e += blockDim.x) {
        const int x = idx[(long long)s * per_src + e];
        if (x < 0) continue;                       // dropped copy
        const int j = x / experts_per_rank;
        if (j >= N) { bad = true; continue; }
        atomicAdd(&cnt[j], 1u);
    }
    __syncthreads();
    const int src = src0 + s;
    for (int j = threadIdx.x; j < N; j += blockDim.x)
        if (cnt[j] && j != src)                    // D_ii = 0: self traffic is handled locally (Section 3)
            atomicAdd((unsigned long long*)&demand_rows[(size_t)s * N + j], (unsigned long long)cnt[j] * (unsigned long long)row_bytes);
    if (bad) atomicOr(status, 1);
}

}  // namespace

extern "C" int vp_plan_time(const vp_catalog* c, int B, int k_max, const int32_t* n_steps, const uint16_t* lane_inst,
                            const int64_t* lane_bytes, int64_t lambda_ns, int64_t* time_xw, void* cuda_stream) {
    if (!c || B <= 0 || k_max <= 0 || !n_steps || !lane_inst || !lane_bytes || !time_xw) return VP_E_BAD_ARG;
    if (lambda_ns < 0 || lambda_ns >= VP_ENTRY_LIMIT) return VP_E_BAD_ARG;
    int prev = -1;
    cudaGetDevice(&prev);
    if (cudaSetDevice(c->device) != cudaSuccess) return VP_E_CUDA;
    const int grid = B < c->sm_count * 8 ? B : c->sm_count * 8;
    plan_time_kernel<<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(c->dc.inst_wdiv, c->dc.n_inst, c->dc.W, c->dc.N, k_max, B,
                                                                  n_steps, lane_inst, lane_bytes, lambda_ns, time_xw);
    g_vp_launches++;
    const int rc = cudaGetLastError() == cudaSuccess ? VP_OK : VP_E_CUDA;
    if (prev >= 0) cudaSetDevice(prev);
    return rc;
}

extern "C" int vp_demand_from_routing(const int32_t* expert_idx, int n_src, int T, int topk, int experts_per_rank, int N,
                                      int src0, int64_t row_bytes, int64_t* demand_rows, int32_t* status,
                                      void* cuda_stream) {
    if (!expert_idx || !demand_rows || !status) return VP_E_BAD_ARG;
    if (n_src <= 0 || T <= 0 || topk <= 0 || experts_per_rank <= 0 || N <= 0 || N > VP_MAX_N || src0 < 0 ||
        src0 + n_src > N || row_bytes <= 0 || row_bytes >= VP_ENTRY_LIMIT)
        return VP_E_BAD_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(demand_rows, 0, (size_t)n_src * N * sizeof(int64_t), stream) != cudaSuccess) return VP_E_CUDA;
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), stream) != cudaSuccess) return VP_E_CUDA;
    const long long per_src = (long long)T * topk;
    int slices = (int)((per_src + 16383) / 16384);
    if (slices < 1) slices = 1;
    if ((long long)n_src * slices > 0x7fffffffLL) return VP_E_UNSUPPORTED;
    demand_kernel<<<n_src * slices, 256, 0, stream>>>(expert_idx, n_src, per_src, experts_per_rank, N, src0, row_bytes, slices,
                                                      demand_rows, status);
    g_vp_launches++;
    return cudaGetLastError() == cudaSuccess ? VP_OK : VP_E_CUDA;
}
