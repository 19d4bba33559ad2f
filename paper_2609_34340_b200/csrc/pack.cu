// vp_pack: stage one rank's routed token rows in activation x destination order
// (Section 5, "Device-resident buffer layout").
//
// Four kernels on the caller's stream:
//   count + plan : per 256-copy chunk, how many copies go to each destination rank; one more
//           block builds, meanwhile, the rank's segment table: for every destination, the
//           activations that send to it, with the stream position they start at and their
//           first staged row (from the plan's send offsets)
//   scan  : exclusive scan of the chunk counts over chunks, one warp per destination
//   map   : stable position of every copy inside its destination's stream ->
//           staged row (binary search in the segment table); writes src_map
//   copy  : token-major: every source row is read ONCE and written to each of
//           its staged rows.  Rows travel global -> shared -> global as bulk
//           asynchronous copies (TMA): one warp per CTA drives a ring of
//           shared-memory stages, an mbarrier per stage signals the load, and
//           the up to topk stores of a token form one bulk group whose read
//           completion frees the stage.
#include <cuda_runtime.h>

#include "row_copy.cuh"
#include "vp_internal.h"

namespace {

constexpr int kItems = 8;                  // 32-copy rounds per warp chunk
constexpr int kChunk = 32 * kItems;        // copies per warp chunk
constexpr int kWarpsPerBlock = 8;

struct PackWs {
    int32_t* flags;      // [0] abort, [1] n_segments
    int32_t* hist;       // [n_chunks][N] copies of each chunk per destination
    int32_t* base;       // [n_chunks][N] copies to that destination in earlier chunks
    int32_t* len;        // [N] routed copies per destination
    int32_t* planned;    // [N] rows the plan sends to each destination
    int32_t* seg_ptr;    // [N+1]
    int32_t* seg_start;  // [k_max] stream position of a segment's first row
    int32_t* seg_row;    // [k_max] staged row of a segment's first row
    int32_t* dst_row;    // [T*topk] staged row of each copy, -1 = not staged
    size_t bytes;
};

PackWs carve(void* base, int N, int T, int topk, int k_max) {
    PackWs w;
    size_t o = 0;
    auto take = [&](size_t n) { size_t at = o; o += vp_align256(n); return (char*)base + at; };
    long long E = (long long)T * topk;
    int n_chunks = (int)((E + kChunk - 1) / kChunk);
    w.flags = (int32_t*)take(256);
    w.hist = (int32_t*)take((size_t)n_chunks * N * 4);
    w.base = (int32_t*)take((size_t)n_chunks * N * 4);
    w.len = (int32_t*)take((size_t)N * 4);
    w.planned = (int32_t*)take((size_t)N * 4);
    w.seg_ptr = (int32_t*)take((size_t)(N + 1) * 4);
    w.seg_start = (int32_t*)take((size_t)k_max * 4);
    w.seg_row = (int32_t*)take((size_t)k_max * 4);
    w.dst_row = (int32_t*)take((size_t)E * 4);
    w.bytes = o;
    return w;
}

__device__ __forceinline__ int dest_of(int x, int experts_per_rank, int N, int rank) {
    // destination rank of a routed copy, or -1 if it is not staged (dropped, local, out of range)
    if (x < 0) return -1;
    int j = x / experts_per_rank;
    return (j >= N || j == rank) ? -1 : j;
}

__device__ __forceinline__ void count_block(const int32_t* __restrict__ idx, long long E, int N, int rank, int experts_per_rank,
                                            int32_t* __restrict__ hist, int32_t* __restrict__ status) {
    __shared__ int wh[kWarpsPerBlock][VP_MAX_N];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long chunk = (long long)blockIdx.x * kWarpsPerBlock + warp;
    const long long e0 = chunk * kChunk;
    if (e0 >= E) return;
    for (int j = lane; j < N; j += 32) wh[warp][j] = 0;
    __syncwarp();
    bool bad = false;
    for (int it = 0; it < kItems; it++) {
        long long e = e0 + it * 32 + lane;
        if (e < E) {
            int x = idx[e];
            int j = dest_of(x, experts_per_rank, N, rank);
            if (x >= 0 && x / experts_per_rank >= N) bad = true;
            if (j >= 0) atomicAdd(&wh[warp][j], 1);
        }
    }
    __syncwarp();
    for (int j = lane; j < N; j += 32) hist[chunk * N + j] = wh[warp][j];
    if (bad) atomicOr(status, VP_ST_PACK_MISMATCH);
}

// One block of VP_MAX_N threads.  Thread j owns destination j; the rank's column of the plan is staged
// through shared memory a tile of steps at a time so that its global loads run in parallel.
__device__ __forceinline__ void segments_block(const int32_t* __restrict__ n_steps_p, const int16_t* __restrict__ lane_dst,
                                               const int64_t* __restrict__ lane_bytes, const int64_t* __restrict__ send_off, int N,
                                               int rank, int k_max, int64_t row_bytes, int64_t capacity_bytes, PackWs w,
                                               int32_t* __restrict__ status) {
    __shared__ int s_cnt[VP_MAX_N + 1];
    __shared__ int16_t t_dst[VP_MAX_N];
    __shared__ int32_t t_rows[VP_MAX_N], t_base[VP_MAX_N];
    const int j = threadIdx.x, NT = blockDim.x;
    int K = *n_steps_p;
    if (K > k_max) K = k_max;
    if (K < 0) K = 0;
    // pass 1: how many activations send to each destination
    int cnt = 0;
    for (int k0 = 0; k0 < K; k0 += NT) {
        const int k = k0 + j;
        t_dst[j] = k < K ? lane_dst[(size_t)k * N + rank] : (int16_t)-1;
        __syncthreads();
        if (j < N) {
            const int n = min(NT, K - k0);
            for (int i = 0; i < n; i++) cnt += (t_dst[i] == j);
        }
        __syncthreads();
    }
    if (j < N) s_cnt[j] = cnt;
    __syncthreads();
    if (j == 0) {
        int run = 0;
        for (int d = 0; d < N; d++) { int v = s_cnt[d]; s_cnt[d] = run; run += v; }
        s_cnt[N] = run;
        w.seg_ptr[N] = run;
        if (send_off[(size_t)K * N + rank] > capacity_bytes) { atomicOr(status, VP_ST_PACK_CAPACITY); w.flags[0] = 1; }
    }
    __syncthreads();
    // pass 2: the segments of each destination: stream position and staged row where each one starts
    int p = j < N ? s_cnt[j] : 0;
    long long cum = 0;
    bool bad = false;
    if (j < N) w.seg_ptr[j] = p;
    for (int k0 = 0; k0 < K; k0 += NT) {
        const int k = k0 + j;
        if (k < K) {
            const int64_t bytes = lane_bytes[(size_t)k * N + rank];
            t_dst[j] = lane_dst[(size_t)k * N + rank];
            t_rows[j] = (int32_t)(bytes / row_bytes);
            t_base[j] = (int32_t)(send_off[(size_t)k * N + rank] / row_bytes);
            if (t_dst[j] >= 0 && bytes % row_bytes) bad = true;
        } else {
            t_dst[j] = -1;
        }
        __syncthreads();
        if (j < N) {
            const int n = min(NT, K - k0);
            for (int i = 0; i < n; i++) {
                if (t_dst[i] != j) continue;
                w.seg_start[p] = (int32_t)cum;
                w.seg_row[p] = t_base[i];
                cum += t_rows[i];
                p++;
            }
        }
        __syncthreads();
    }
    if (j < N) {
        w.planned[j] = (int32_t)cum;
        if (j == rank && cum != 0) bad = true;
    }
    if (bad) atomicOr(status, VP_ST_PACK_MISMATCH);
}

// The count blocks and, as the last block of the grid, the segment table: the two need nothing from each other.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
pack_count_plan_kernel(const int32_t* __restrict__ idx, long long E, int N, int rank, int experts_per_rank,
                       const int32_t* __restrict__ n_steps_p, const int16_t* __restrict__ lane_dst,
                       const int64_t* __restrict__ lane_bytes, const int64_t* __restrict__ send_off, int k_max,
                       int64_t row_bytes, int64_t capacity_bytes, PackWs w, int32_t* __restrict__ status) {
    static_assert(kWarpsPerBlock * 32 == VP_MAX_N, "the segment block has one thread per destination");
    if (blockIdx.x == gridDim.x - 1) segments_block(n_steps_p, lane_dst, lane_bytes, send_off, N, rank, k_max, row_bytes, capacity_bytes, w, status);
    else count_block(idx, E, N, rank, experts_per_rank, w.hist, status);
}

// Exclusive scan of the chunk counts, per destination: one warp per destination, 32 chunks per step; then the
// routed copies of a destination must be as many as the plan sends there.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
pack_scan_kernel(int N, int rank, int n_chunks, PackWs w, int32_t* __restrict__ status) {
    const int lane = threadIdx.x & 31, d = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (d >= N) return;
    int run = 0;
    const int32_t* __restrict__ in = w.hist;
    int32_t* __restrict__ out = w.base;
#pragma unroll 4
    for (int b0 = 0; b0 < n_chunks; b0 += 32) {
        const int c = b0 + lane;
        const int v = c < n_chunks ? in[(size_t)c * N + d] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (c < n_chunks) out[(size_t)c * N + d] = run + incl - v;
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) {
        w.len[d] = run;
        if (d != rank && run != w.planned[d]) atomicOr(status, VP_ST_PACK_MISMATCH);
    }
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
pack_map_kernel(const int32_t* __restrict__ idx, long long E, int N, int rank, int experts_per_rank, PackWs w,
                int32_t* __restrict__ src_map) {
    __shared__ int base[kWarpsPerBlock][VP_MAX_N];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long chunk = (long long)blockIdx.x * kWarpsPerBlock + warp;
    const long long e0 = chunk * kChunk;
    if (e0 >= E) return;
    const bool aborted = w.flags[0] != 0;
    for (int j = lane; j < N; j += 32) base[warp][j] = w.base[chunk * N + j];
    __syncwarp();
    for (int it = 0; it < kItems; it++) {
        long long e = e0 + it * 32 + lane;
        int j = -1;
        if (e < E) j = dest_of(idx[e], experts_per_rank, N, rank);
        const unsigned peers = __match_any_sync(0xffffffffu, j >= 0 ? j : -1 - lane);
        int row = -1;
        if (j >= 0) {
            const int p = base[warp][j] + __popc(peers & ((1u << lane) - 1));   // position in stream_j
            if (!aborted && p < w.planned[j]) {
                int lo = w.seg_ptr[j], hi = w.seg_ptr[j + 1] - 1;              // last segment starting at or before p
                while (lo < hi) {
                    int mid = (lo + hi + 1) >> 1;
                    if (w.seg_start[mid] <= p) lo = mid; else hi = mid - 1;
                }
                row = w.seg_row[lo] + (p - w.seg_start[lo]);
            }
        }
        __syncwarp();
        if (j >= 0 && (peers & ((1u << lane) - 1)) == 0) base[warp][j] += __popc(peers);
        __syncwarp();
        if (e < E) {
            w.dst_row[e] = row;
            if (row >= 0 && src_map) src_map[row] = (int32_t)e;
        }
    }
}

}  // namespace

extern "C" size_t vp_pack_workspace_bytes(int N, int T, int topk, int k_max) {
    if (N <= 0 || N > VP_MAX_N || T <= 0 || topk <= 0 || k_max <= 0) return 0;
    return carve(nullptr, N, T, topk, k_max).bytes;
}

extern "C" int vp_pack(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* lane_bytes_b,
                       const int64_t* send_off_b, int N, int rank, int k_max, const int32_t* expert_idx, int T,
                       int topk, int experts_per_rank, const void* rows, int64_t row_bytes, void* staged,
                       int64_t staged_capacity_bytes, int32_t* src_map, int32_t* status, void* workspace,
                       size_t workspace_bytes, void* cuda_stream) {
    if (!n_steps_b || !lane_dst_b || !lane_bytes_b || !send_off_b || !expert_idx || !rows || !staged || !status)
        return VP_E_BAD_ARG;
    if (N <= 0 || N > VP_MAX_N || rank < 0 || rank >= N || k_max <= 0 || T <= 0 || topk <= 0 || experts_per_rank <= 0 ||
        row_bytes <= 0 || staged_capacity_bytes < 0)
        return VP_E_BAD_ARG;
    if (staged_capacity_bytes / row_bytes >= ((int64_t)1 << 31) || (long long)T * topk >= ((long long)1 << 31))
        return VP_E_UNSUPPORTED;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < vp_pack_workspace_bytes(N, T, topk, k_max))
        return VP_E_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    PackWs w = carve(workspace, N, T, topk, k_max);
    const long long E = (long long)T * topk;
    const int n_chunks = (int)((E + kChunk - 1) / kChunk);
    const int blocks = (n_chunks + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (cudaMemsetAsync(w.flags, 0, 256, stream) != cudaSuccess) return VP_E_CUDA;
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), stream) != cudaSuccess) return VP_E_CUDA;
    vp_prof_mark(1, 0, stream);
    pack_count_plan_kernel<<<blocks + 1, kWarpsPerBlock * 32, 0, stream>>>(expert_idx, E, N, rank, experts_per_rank, n_steps_b,
                                                                         lane_dst_b, lane_bytes_b, send_off_b, k_max, row_bytes,
                                                                         staged_capacity_bytes, w, status);
    pack_scan_kernel<<<(N + kWarpsPerBlock - 1) / kWarpsPerBlock, kWarpsPerBlock * 32, 0, stream>>>(N, rank, n_chunks, w, status);
    pack_map_kernel<<<blocks, kWarpsPerBlock * 32, 0, stream>>>(expert_idx, E, N, rank, experts_per_rank, w, src_map);
    g_vp_launches += 3;
    vp_prof_mark(1, 1, stream);
    vp_prof_mark(2, 0, stream);

    const int rc = launch_row_copy(rows, staged, w.dst_row, w.flags, T, topk, row_bytes, status, stream);
    vp_prof_mark(2, 1, stream);
    return rc;
}

// ---- vp_pack_static: the pack with its scratch built into the library ---------------------------------
//
// Some callers of the pack have no way to obtain device scratch at the moment they call it: they sit inside
// a serving engine's steady-state step, are handed only the input and output buffers, hold no allocator of
// their own, and must not call cudaMalloc there (it synchronises the whole device, it can fail under the
// engine's memory cap, and the engine accounts for every byte itself).  For them the library keeps one
// fixed block of device memory, reserved when the library is loaded on a GPU and held until the process
// exits, and uses it in place of the caller's workspace.
//
// In host code `g_pack_static_scratch` is only a handle for the device array; its device address has to be
// asked for with cudaGetSymbolAddress, once per device, with that device current.
static __device__ __align__(256) unsigned char g_pack_static_scratch[VP_PACK_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the built-in scratch on the current device (looked up on first use).
int static_scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VP_E_CUDA;
    void* p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_pack_static_scratch) != cudaSuccess || !p) return VP_E_CUDA;
        __atomic_store_n(&g_static_scratch_addr[dev], p, __ATOMIC_RELEASE);
    }
    *out = p;
    return VP_OK;
}
}  // namespace

extern "C" int vp_pack_static(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* lane_bytes_b,
                              const int64_t* send_off_b, int N, int rank, int k_max, const int32_t* expert_idx, int T,
                              int topk, int experts_per_rank, const void* rows, int64_t row_bytes, void* staged,
                              int64_t staged_capacity_bytes, int32_t* src_map, int32_t* status, void* cuda_stream) {
    if (N <= 0 || N > VP_MAX_N || T <= 0 || topk <= 0 || k_max <= 0) return VP_E_BAD_ARG;
    // the problem must fit the built-in block; nothing is launched otherwise
    const size_t need = vp_pack_workspace_bytes(N, T, topk, k_max);
    if (need == 0 || need > (size_t)VP_PACK_STATIC_SCRATCH_BYTES) return VP_E_WORKSPACE;
    void* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != VP_OK) return rc;
    // vp_pack zeroes the flags it needs and overwrites every other scratch word it reads, so whatever the
    // previous call left in the block does not matter
    return vp_pack(n_steps_b, lane_dst_b, lane_bytes_b, send_off_b, N, rank, k_max, expert_idx, T, topk,
                   experts_per_rank, rows, row_bytes, staged, staged_capacity_bytes, src_map, status, scratch,
                   (size_t)VP_PACK_STATIC_SCRATCH_BYTES, cuda_stream);
}
