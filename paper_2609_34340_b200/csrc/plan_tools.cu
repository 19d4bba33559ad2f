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
    if (!c || c->device < 0 || B <= 0 || k_max <= 0 || !n_steps || !lane_inst || !lane_bytes || !time_xw) return VP_E_BAD_ARG;
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

// ---- plan-quality sweep: Eq. (2) over a grid of (lambda, K_target) ---------------------------------------------------

namespace {

struct SweepBufs {
    int32_t *n_steps, *chan_id, *status;
    int16_t* lane_dst;
    uint16_t* lane_inst;
    int64_t *lane_bytes, *send_off, *tau;
    void* ws;
    size_t ws_bytes, total;
};

SweepBufs carve_sweep(char* base, const vp_catalog* c, int B, const vp_sched_params* p) {
    const size_t N = (size_t)c->info.N, K = (size_t)p->k_max, b = (size_t)B;
    size_t off = 0;
    auto take = [&](size_t bytes) { char* at = base ? base + off : nullptr; off += vp_align256(bytes); return (void*)at; };
    SweepBufs s;
    s.n_steps = (int32_t*)take(b * 4);
    s.chan_id = (int32_t*)take(b * K * 4);
    s.status = (int32_t*)take(b * 4);
    s.lane_dst = (int16_t*)take(b * K * N * 2);
    s.lane_inst = (uint16_t*)take(b * K * N * 2);
    s.lane_bytes = (int64_t*)take(b * K * N * 8);
    s.send_off = (int64_t*)take(b * (K + 1) * N * 8);
    s.tau = (int64_t*)take(b * 8);
    s.ws_bytes = vp_schedule_workspace_bytes(c, B, p);
    s.ws = take(s.ws_bytes);
    s.total = off;
    return s;
}

}  // namespace

extern "C" size_t vp_sweep_workspace_bytes(const vp_catalog* c, int B, const vp_sched_params* p) {
    if (!c || !p || B <= 0 || p->k_max <= 0) return 0;
    SweepBufs s = carve_sweep(nullptr, c, B, p);
    return s.ws_bytes ? s.total : 0;
}

extern "C" int vp_sweep_plan_time(const vp_catalog* c, const vp_sched_params* p, const int64_t* demand, int B,
                                  const int64_t* lambda_ns, int n_lambda, const int32_t* k_target, int n_k, int64_t* time_xw,
                                  int32_t* n_steps_out, int32_t* status_out, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream) {
    if (!c || !p || !demand || !lambda_ns || !k_target || !time_xw || B <= 0 || n_lambda <= 0 || n_k <= 0 || p->k_max <= 0)
        return VP_E_BAD_ARG;
    if (!workspace || ((uintptr_t)workspace & 255)) return VP_E_WORKSPACE;
    SweepBufs s = carve_sweep((char*)workspace, c, B, p);
    if (!s.ws_bytes) return VP_E_BAD_ARG;
    if (workspace_bytes < s.total) return VP_E_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    for (int i = 0; i < n_lambda; i++)
        for (int j = 0; j < n_k; j++) {
            vp_sched_params q = *p;
            q.lambda_ns = lambda_ns[i];
            q.k_target = k_target[j];
            int rc = vp_schedule_batch(c, &q, demand, nullptr, B, s.n_steps, s.chan_id, s.lane_dst, s.lane_inst, s.lane_bytes, s.send_off,
                                       nullptr, s.tau, s.status, s.ws, s.ws_bytes, cuda_stream);
            if (rc) return rc;
            const size_t at = ((size_t)i * n_k + j) * B;
            rc = vp_plan_time(c, B, p->k_max, s.n_steps, s.lane_inst, s.lane_bytes, q.lambda_ns, time_xw + at, cuda_stream);
            if (rc) return rc;
            if (n_steps_out && cudaMemcpyAsync(n_steps_out + at, s.n_steps, (size_t)B * 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
                return VP_E_CUDA;
            if (status_out && cudaMemcpyAsync(status_out + at, s.status, (size_t)B * 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
                return VP_E_CUDA;
        }
    return VP_OK;
}
