// vp_unpack: the receive side of the buffer layout (Section 5: "the receive kernel unpacks them directly
// into the output layout").
//
// The receive buffer of a rank holds, step after step, the rows its one sender of that step delivered
// (at recv_off[k][rank]).  The output is expert-major: all rows of local expert 0, then 1, ...; inside an
// expert by source rank; inside a source in arrival order.  That is a stable sort of the received rows by
// the key (expert, source), done as a counting sort:
//   plan  : the rank's receive segments (first row, source rank) from the plan
//   count : key of every row (binary search of its segment), per 256-row chunk a histogram of keys
//   scan  : per key an exclusive scan over the chunks; then an exclusive scan over the keys
//   map   : stable position of every row among the rows of its key -> output row
//   copy  : the row copy shared with the pack (each received row read once, written once)
#include <cuda_runtime.h>

#include "row_copy.cuh"
#include "vp_internal.h"

namespace {

constexpr int kItems = 8;                  // 32-row rounds per warp chunk
constexpr int kChunk = 32 * kItems;
constexpr int kWarps = 8;
constexpr int kMaxKeys = 1024;             // experts_per_rank x N

struct UnpackWs {
    int32_t* flags;      // [0] abort, [1] number of segments, [2] rows received
    int32_t* seg_row0;   // [k_max] first receive row of a segment
    int32_t* seg_end;    // [k_max] one past its last receive row
    int32_t* seg_src;    // [k_max] its source rank
    int32_t* hist;       // [n_chunks][keys]
    int32_t* base;       // [n_chunks][keys] rows of that key in earlier chunks
    int32_t* key_total;  // [keys]
    int32_t* key_base;   // [keys + 1] first output row of a key
    int32_t* row_key;    // [capacity] key of a received row, -1 = none
    int32_t* out_row;    // [capacity] output row of a received row, -1 = none
    size_t bytes;
};

UnpackWs carve(void* base, int keys, long long capacity_rows, int k_max) {
    UnpackWs w;
    size_t o = 0;
    auto take = [&](size_t n) { size_t at = o; o += vp_align256(n); return (char*)base + at; };
    const long long n_chunks = (capacity_rows + kChunk - 1) / kChunk;
    w.flags = (int32_t*)take(256);
    w.seg_row0 = (int32_t*)take((size_t)k_max * 4);
    w.seg_end = (int32_t*)take((size_t)k_max * 4);
    w.seg_src = (int32_t*)take((size_t)k_max * 4);
    w.hist = (int32_t*)take((size_t)n_chunks * keys * 4);
    w.base = (int32_t*)take((size_t)n_chunks * keys * 4);
    w.key_total = (int32_t*)take((size_t)keys * 4);
    w.key_base = (int32_t*)take((size_t)(keys + 1) * 4);
    w.row_key = (int32_t*)take((size_t)capacity_rows * 4);
    w.out_row = (int32_t*)take((size_t)capacity_rows * 4);
    w.bytes = o;
    return w;
}

__global__ void __launch_bounds__(256)
unpack_plan_kernel(const int32_t* __restrict__ n_steps_p, const int16_t* __restrict__ lane_dst,
                   const int64_t* __restrict__ recv_off, int N, int rank, int k_max, int64_t row_bytes,
                   long long capacity_rows, UnpackWs w, int32_t* __restrict__ status) {
    __shared__ int t_row0[256], t_src[256], t_rows[256];
    __shared__ int s_n;
    const int tid = threadIdx.x;
    int K = *n_steps_p;
    K = K < 0 ? 0 : (K > k_max ? k_max : K);
    if (tid == 0) {
        s_n = 0;
        const int64_t total = recv_off[(size_t)K * N + rank];
        int st = 0;
        if (total % row_bytes) st |= VP_ST_PACK_MISMATCH;
        if (total / row_bytes > capacity_rows) { st |= VP_ST_PACK_CAPACITY; w.flags[0] = 1; }
        w.flags[2] = (int32_t)(total / row_bytes > capacity_rows ? 0 : total / row_bytes);
        if (st) atomicOr(status, st);
    }
    __syncthreads();
    bool bad = false;
    for (int k0 = 0; k0 < K; k0 += 256) {
        const int k = k0 + tid;
        t_rows[tid] = 0;
        if (k < K) {
            const int64_t lo = recv_off[(size_t)k * N + rank], hi = recv_off[(size_t)(k + 1) * N + rank];
            if (hi > lo && (lo % row_bytes || hi % row_bytes)) bad = true;   // such a segment is left out
            else if (hi > lo) {
                int src = -1;
                for (int i = 0; i < N; i++)
                    if (lane_dst[(size_t)k * N + i] == rank) src = i;
                if (src < 0) bad = true;
                t_row0[tid] = (int)(lo / row_bytes);
                t_rows[tid] = (int)(hi / row_bytes - lo / row_bytes);
                t_src[tid] = src;
            }
        }
        __syncthreads();
        if (tid == 0) {                                    // steps are in receive order: append in order
            int n = s_n;
            for (int i = 0; i < 256 && k0 + i < K; i++)
                if (t_rows[i] > 0) { w.seg_row0[n] = t_row0[i]; w.seg_end[n] = t_row0[i] + t_rows[i]; w.seg_src[n] = t_src[i]; n++; }
            s_n = n;
        }
        __syncthreads();
    }
    if (tid == 0) w.flags[1] = s_n;
    if (bad) atomicOr(status, VP_ST_PACK_MISMATCH);
}

// by_routing = 0: item r is a received row, key = (local expert, source rank of its segment)
// by_routing = 1: item c is a routed copy, key = its global expert id (copies to `rank` itself or dropped: none)
__global__ void __launch_bounds__(kWarps * 32)
unpack_count_kernel(const int32_t* __restrict__ recv_expert, long long capacity_rows, int N, int experts_per_rank,
                    int keys, UnpackWs w, int32_t* __restrict__ status, int by_routing, int rank) {
    __shared__ int wh[kWarps][kMaxKeys];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long chunk = (long long)blockIdx.x * kWarps + warp;
    const long long r0 = chunk * kChunk;
    if (r0 >= capacity_rows) return;
    const int R = w.flags[0] ? 0 : w.flags[2], n_seg = w.flags[1];
    for (int j = lane; j < keys; j += 32) wh[warp][j] = 0;
    __syncwarp();
    bool bad = false;
    for (int it = 0; it < kItems; it++) {
        const long long r = r0 + it * 32 + lane;
        if (r >= capacity_rows) continue;
        int key = -1;
        if (by_routing) {
            const int e = recv_expert[r];
            if (!w.flags[0] && e >= 0 && e < keys && e / experts_per_rank != rank) { key = e; atomicAdd(&wh[warp][key], 1); }
        } else if (r < R) {
            int lo = 0, hi = n_seg - 1;                    // last segment starting at or before r
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (w.seg_row0[mid] <= r) lo = mid; else hi = mid - 1;
            }
            const int e = recv_expert[r];
            const int src = n_seg > 0 && w.seg_row0[lo] <= r && r < w.seg_end[lo] ? w.seg_src[lo] : -1;
            if (e < 0 || e >= experts_per_rank || src < 0) bad = true;
            else { key = e * N + src; atomicAdd(&wh[warp][key], 1); }
        }
        w.row_key[r] = key;
    }
    __syncwarp();
    for (int j = lane; j < keys; j += 32) w.hist[chunk * keys + j] = wh[warp][j];
    if (bad) atomicOr(status, VP_ST_PACK_MISMATCH);
}

// one warp per key: exclusive scan of its counts over the chunks
__global__ void __launch_bounds__(kWarps * 32)
unpack_scan_kernel(int keys, int n_chunks, UnpackWs w) {
    const int lane = threadIdx.x & 31, key = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (key >= keys) return;
    const int32_t* __restrict__ in = w.hist;
    int32_t* __restrict__ out = w.base;
    int run = 0;
#pragma unroll 4
    for (int b0 = 0; b0 < n_chunks; b0 += 32) {
        const int c = b0 + lane;
        const int v = c < n_chunks ? in[(size_t)c * keys + key] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (c < n_chunks) out[(size_t)c * keys + key] = run + incl - v;
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) w.key_total[key] = run;
}

// one block: exclusive scan over the keys (expert-major, then source), expert offsets, consistency check
__global__ void __launch_bounds__(kMaxKeys)
unpack_keys_kernel(int keys, int N, int experts_per_rank, UnpackWs w, int32_t* __restrict__ expert_off,
                   int32_t* __restrict__ status) {
    __shared__ int s[kMaxKeys];
    __shared__ int warp_sum[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int v = tid < keys ? w.key_total[tid] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int ws = warp_sum[lane], wi = ws;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        warp_sum[lane] = wi - ws;
    }
    __syncthreads();
    const int excl = warp_sum[warp] + incl - v;
    s[tid] = excl;
    if (tid < keys) w.key_base[tid] = excl;
    __syncthreads();
    if (expert_off && tid < experts_per_rank) expert_off[tid] = s[tid * N];
    if (tid == kMaxKeys - 1) {
        const int total = excl + v;
        w.key_base[keys] = total;
        if (expert_off) {
            expert_off[experts_per_rank] = total;
            if (!w.flags[0] && total != w.flags[2]) atomicOr(status, VP_ST_PACK_MISMATCH);
        }
    }
}

__global__ void __launch_bounds__(kWarps * 32)
unpack_map_kernel(long long capacity_rows, int N, int keys, UnpackWs w, int32_t* __restrict__ out_src,
                  int32_t* __restrict__ out_map) {
    __shared__ int next[kWarps][kMaxKeys];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long chunk = (long long)blockIdx.x * kWarps + warp;
    const long long r0 = chunk * kChunk;
    if (r0 >= capacity_rows) return;
    for (int j = lane; j < keys; j += 32) next[warp][j] = w.key_base[j] + w.base[chunk * keys + j];
    __syncwarp();
    for (int it = 0; it < kItems; it++) {
        const long long r = r0 + it * 32 + lane;
        const int key = r < capacity_rows ? w.row_key[r] : -1;
        const unsigned peers = __match_any_sync(0xffffffffu, key >= 0 ? key : -1 - lane);
        int o = -1;
        if (key >= 0) o = next[warp][key] + __popc(peers & ((1u << lane) - 1));
        __syncwarp();
        if (key >= 0 && (peers & ((1u << lane) - 1)) == 0) next[warp][key] += __popc(peers);
        __syncwarp();
        if (r < capacity_rows) {
            w.out_row[r] = o;
            if (o >= 0) {
                if (out_src) out_src[o] = key % N;
                if (out_map) out_map[o] = (int32_t)r;
            }
        }
    }
}

}  // namespace

extern "C" size_t vp_unpack_workspace_bytes(int N, int64_t capacity_rows, int experts_per_rank, int k_max) {
    if (N <= 0 || N > VP_MAX_N || capacity_rows <= 0 || experts_per_rank <= 0 || k_max <= 0) return 0;
    if ((long long)N * experts_per_rank > kMaxKeys || capacity_rows >= ((int64_t)1 << 31)) return 0;
    return carve(nullptr, N * experts_per_rank, capacity_rows, k_max).bytes;
}

extern "C" int vp_unpack(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* recv_off_b, int N, int rank,
                         int k_max, const void* recv, int64_t row_bytes, int64_t capacity_rows, const int32_t* recv_expert,
                         int experts_per_rank, void* out, int32_t* expert_off, int32_t* out_src, int32_t* out_map,
                         int32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!n_steps_b || !lane_dst_b || !recv_off_b || !recv || !recv_expert || !out || !expert_off || !status) return VP_E_BAD_ARG;
    if (N <= 0 || N > VP_MAX_N || rank < 0 || rank >= N || k_max <= 0 || row_bytes <= 0 || capacity_rows <= 0 ||
        experts_per_rank <= 0)
        return VP_E_BAD_ARG;
    const int keys = N * experts_per_rank;
    if ((long long)N * experts_per_rank > kMaxKeys || capacity_rows >= ((int64_t)1 << 31)) return VP_E_UNSUPPORTED;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < vp_unpack_workspace_bytes(N, capacity_rows, experts_per_rank, k_max))
        return VP_E_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    UnpackWs w = carve(workspace, keys, capacity_rows, k_max);
    const int n_chunks = (int)((capacity_rows + kChunk - 1) / kChunk);
    const int blocks = (n_chunks + kWarps - 1) / kWarps;
    if (cudaMemsetAsync(w.flags, 0, 256, stream) != cudaSuccess) return VP_E_CUDA;
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), stream) != cudaSuccess) return VP_E_CUDA;
    unpack_plan_kernel<<<1, 256, 0, stream>>>(n_steps_b, lane_dst_b, recv_off_b, N, rank, k_max, row_bytes, capacity_rows, w, status);
    unpack_count_kernel<<<blocks, kWarps * 32, 0, stream>>>(recv_expert, capacity_rows, N, experts_per_rank, keys, w, status, 0, rank);
    unpack_scan_kernel<<<(keys + kWarps - 1) / kWarps, kWarps * 32, 0, stream>>>(keys, n_chunks, w);
    unpack_keys_kernel<<<1, kMaxKeys, 0, stream>>>(keys, N, experts_per_rank, w, expert_off, status);
    unpack_map_kernel<<<blocks, kWarps * 32, 0, stream>>>(capacity_rows, N, keys, w, out_src, out_map);
    g_vp_launches += 5;
    if (cudaGetLastError() != cudaSuccess) return VP_E_CUDA;
    vp_prof_mark(3, 0, stream);
    const int rc = launch_row_copy(recv, out, w.out_row, w.flags, (int)capacity_rows, 1, row_bytes, status, stream);
    vp_prof_mark(3, 1, stream);
    return rc;
}

// ---- return direction: receive buffer -> token layout ---------------------------------------------------

namespace {

struct TokWs {
    UnpackWs u;            // flags, histograms, scans, key of every copy (row_key), inverse map (out_row)
    int32_t* step_sender;  // [k_max] sender of the step's segment for this rank, -1 = none
    int32_t* step_row0;    // [k_max] first receive row of the segment
    int32_t* step_rows;    // [k_max] its rows
    int32_t* sender_ptr;   // [N + 1] segments of sender j are sseg_*[sender_ptr[j] .. sender_ptr[j+1])
    int32_t* sender_total; // [N] rows sender j delivers
    int32_t* sseg_stream0; // [k_max] position of the segment's first row in the sender's stream
    int32_t* sseg_row0;    // [k_max]
    int32_t* sseg_rows;    // [k_max]
    size_t bytes;
};

TokWs carve_tokens(void* base, int N, int keys, long long copies, long long capacity_rows, int k_max) {
    TokWs w;
    size_t o = 0;
    auto take = [&](size_t n) { size_t at = o; o += vp_align256(n); return (char*)base + at; };
    const long long n_chunks = (copies + kChunk - 1) / kChunk;
    w.u.flags = (int32_t*)take(256);
    w.u.seg_row0 = w.u.seg_end = w.u.seg_src = nullptr;
    w.u.hist = (int32_t*)take((size_t)n_chunks * keys * 4);
    w.u.base = (int32_t*)take((size_t)n_chunks * keys * 4);
    w.u.key_total = (int32_t*)take((size_t)keys * 4);
    w.u.key_base = (int32_t*)take((size_t)(keys + 1) * 4);
    w.u.row_key = (int32_t*)take((size_t)copies * 4);
    w.u.out_row = (int32_t*)take((size_t)capacity_rows * 4);
    w.step_sender = (int32_t*)take((size_t)k_max * 4);
    w.step_row0 = (int32_t*)take((size_t)k_max * 4);
    w.step_rows = (int32_t*)take((size_t)k_max * 4);
    w.sender_ptr = (int32_t*)take((size_t)(N + 1) * 4);
    w.sender_total = (int32_t*)take((size_t)N * 4);
    w.sseg_stream0 = (int32_t*)take((size_t)k_max * 4);
    w.sseg_row0 = (int32_t*)take((size_t)k_max * 4);
    w.sseg_rows = (int32_t*)take((size_t)k_max * 4);
    w.bytes = o;
    return w;
}

// One block of VP_MAX_N threads: the segment every step delivers to `rank`, then per sender its segments in step order.
__global__ void __launch_bounds__(VP_MAX_N)
tokens_plan_kernel(const int32_t* __restrict__ n_steps_p, const int16_t* __restrict__ lane_dst,
                   const int64_t* __restrict__ lane_bytes, const int64_t* __restrict__ recv_off, int N, int rank, int k_max,
                   int64_t row_bytes, long long capacity_rows, TokWs w, int32_t* __restrict__ status) {
    __shared__ int s_cnt[VP_MAX_N + 1];
    const int tid = threadIdx.x;
    int K = *n_steps_p;
    K = K < 0 ? 0 : (K > k_max ? k_max : K);
    const bool over = recv_off[(size_t)K * N + rank] > capacity_rows * row_bytes;      // nothing is unpacked then
    if (tid == 0 && over) { atomicOr(status, VP_ST_PACK_CAPACITY); w.u.flags[0] = 1; }
    bool bad = false;
    for (int k = tid; k < K; k += blockDim.x) {
        int sender = -1;
        for (int j = 0; j < N; j++)
            if (lane_dst[(size_t)k * N + j] == rank) sender = j;
        int rows = 0, row0 = 0;
        if (sender >= 0) {
            const int64_t bytes = lane_bytes[(size_t)k * N + sender], at = recv_off[(size_t)k * N + rank];
            if (bytes % row_bytes || at % row_bytes) { bad = true; sender = -1; }       // such a segment is left out
            else { rows = (int)(bytes / row_bytes); row0 = (int)(at / row_bytes); }
        }
        w.step_sender[k] = rows > 0 ? sender : -1;
        w.step_row0[k] = row0;
        w.step_rows[k] = rows;
    }
    if (bad && !over) atomicOr(status, VP_ST_PACK_MISMATCH);
    __syncthreads();
    int cnt = 0;
    if (tid < N)
        for (int k = 0; k < K; k++) cnt += w.step_sender[k] == tid;
    s_cnt[tid] = tid < N ? cnt : 0;
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int j = 0; j < N; j++) { const int c = s_cnt[j]; s_cnt[j] = run; run += c; }
        s_cnt[N] = run;
    }
    __syncthreads();
    if (tid <= N) w.sender_ptr[tid] = s_cnt[tid];
    if (tid < N) {
        int at = s_cnt[tid], stream = 0;
        for (int k = 0; k < K; k++)
            if (w.step_sender[k] == tid) {
                w.sseg_stream0[at] = stream; w.sseg_row0[at] = w.step_row0[k]; w.sseg_rows[at] = w.step_rows[k];
                stream += w.step_rows[k]; at++;
            }
        w.sender_total[tid] = stream;
    }
}

__global__ void __launch_bounds__(kWarps * 32)
tokens_map_kernel(long long copies, int N, int experts_per_rank, int keys, int rank, TokWs w, int32_t* __restrict__ out_map,
                  int32_t* __restrict__ status) {
    __shared__ int next[kWarps][kMaxKeys];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && threadIdx.x < N && threadIdx.x != rank && !w.u.flags[0]) {      // every sender's stream is used up exactly
        const int j = threadIdx.x;
        if (w.u.key_base[(j + 1) * experts_per_rank] - w.u.key_base[j * experts_per_rank] != w.sender_total[j])
            atomicOr(status, VP_ST_PACK_MISMATCH);
    }
    const long long chunk = (long long)blockIdx.x * kWarps + warp;
    const long long c0 = chunk * kChunk;
    if (c0 >= copies) return;
    for (int j = lane; j < keys; j += 32) next[warp][j] = w.u.key_base[j] + w.u.base[chunk * keys + j];
    __syncwarp();
    for (int it = 0; it < kItems; it++) {
        const long long c = c0 + it * 32 + lane;
        const int key = c < copies ? w.u.row_key[c] : -1;
        const unsigned peers = __match_any_sync(0xffffffffu, key >= 0 ? key : -1 - lane);
        int gpos = -1;
        if (key >= 0) gpos = next[warp][key] + __popc(peers & ((1u << lane) - 1));
        __syncwarp();
        if (key >= 0 && (peers & ((1u << lane) - 1)) == 0) next[warp][key] += __popc(peers);
        __syncwarp();
        if (c >= copies) continue;
        int rrow = -1;
        if (key >= 0) {
            const int j = key / experts_per_rank;
            const int pos = gpos - w.u.key_base[j * experts_per_rank];           // position in sender j's stream
            int lo = w.sender_ptr[j], hi = w.sender_ptr[j + 1] - 1;
            if (hi >= lo && pos < w.sender_total[j]) {
                while (lo < hi) {                                                // last segment starting at or before pos
                    const int mid = (lo + hi + 1) >> 1;
                    if (w.sseg_stream0[mid] <= pos) lo = mid; else hi = mid - 1;
                }
                rrow = w.sseg_row0[lo] + pos - w.sseg_stream0[lo];
                w.u.out_row[rrow] = (int32_t)c;
            }
        }
        if (out_map) out_map[c] = rrow;
    }
}

}  // namespace

extern "C" size_t vp_unpack_tokens_workspace_bytes(int N, int T, int topk, int experts_per_rank, int64_t capacity_rows, int k_max) {
    if (N <= 0 || N > VP_MAX_N || T <= 0 || topk <= 0 || capacity_rows <= 0 || experts_per_rank <= 0 || k_max <= 0) return 0;
    if ((long long)N * experts_per_rank > kMaxKeys || capacity_rows >= ((int64_t)1 << 31) || (long long)T * topk >= ((long long)1 << 31)) return 0;
    return carve_tokens(nullptr, N, N * experts_per_rank, (long long)T * topk, capacity_rows, k_max).bytes;
}

extern "C" int vp_unpack_tokens(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* lane_bytes_b,
                                const int64_t* recv_off_b, int N, int rank, int k_max, const int32_t* expert_idx, int T, int topk,
                                int experts_per_rank, const void* recv, int64_t row_bytes, int64_t capacity_rows, void* out,
                                int32_t* out_map, int32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!n_steps_b || !lane_dst_b || !lane_bytes_b || !recv_off_b || !expert_idx || !recv || !out || !status) return VP_E_BAD_ARG;
    if (N <= 0 || N > VP_MAX_N || rank < 0 || rank >= N || k_max <= 0 || T <= 0 || topk <= 0 || row_bytes <= 0 ||
        capacity_rows <= 0 || experts_per_rank <= 0)
        return VP_E_BAD_ARG;
    const size_t need = vp_unpack_tokens_workspace_bytes(N, T, topk, experts_per_rank, capacity_rows, k_max);
    if (!need) return VP_E_UNSUPPORTED;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return VP_E_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const int keys = N * experts_per_rank;
    const long long copies = (long long)T * topk;
    TokWs w = carve_tokens(workspace, N, keys, copies, capacity_rows, k_max);
    const int n_chunks = (int)((copies + kChunk - 1) / kChunk);
    const int blocks = (n_chunks + kWarps - 1) / kWarps;
    if (cudaMemsetAsync(w.u.flags, 0, 256, stream) != cudaSuccess) return VP_E_CUDA;
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), stream) != cudaSuccess) return VP_E_CUDA;
    if (cudaMemsetAsync(w.u.out_row, 0xFF, (size_t)capacity_rows * 4, stream) != cudaSuccess) return VP_E_CUDA;
    tokens_plan_kernel<<<1, VP_MAX_N, 0, stream>>>(n_steps_b, lane_dst_b, lane_bytes_b, recv_off_b, N, rank, k_max, row_bytes,
                                                   capacity_rows, w, status);
    unpack_count_kernel<<<blocks, kWarps * 32, 0, stream>>>(expert_idx, copies, N, experts_per_rank, keys, w.u, status, 1, rank);
    unpack_scan_kernel<<<(keys + kWarps - 1) / kWarps, kWarps * 32, 0, stream>>>(keys, n_chunks, w.u);
    unpack_keys_kernel<<<1, kMaxKeys, 0, stream>>>(keys, N, experts_per_rank, w.u, nullptr, status);
    tokens_map_kernel<<<blocks, kWarps * 32, 0, stream>>>(copies, N, experts_per_rank, keys, rank, w, out_map, status);
    g_vp_launches += 5;
    if (cudaGetLastError() != cudaSuccess) return VP_E_CUDA;
    vp_prof_mark(3, 0, stream);
    const int rc = launch_row_copy(recv, out, w.u.out_row, w.u.flags, (int)capacity_rows, 1, row_bytes, status, stream);
    vp_prof_mark(3, 1, stream);
    return rc;
}
