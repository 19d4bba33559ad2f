// Host-buffer variants of the two entry points: copy in, run the device path, copy out.
#include <cuda_runtime.h>

#include "vp_internal.h"

namespace {

struct Carver {
    char* base;
    size_t off = 0;
    void* take(size_t bytes) {
        size_t at = off;
        off += vp_align256(bytes);
        return base ? base + at : nullptr;
    }
};

struct SchedBufs {
    int64_t *demand, *tau_in, *lane_bytes, *send_off, *recv_off, *tau_out;
    int32_t *n_steps, *chan_id, *status;
    int16_t* lane_dst;
    uint16_t* lane_inst;
    void* ws;
    size_t ws_bytes, total;
};

SchedBufs carve_sched(void* base, const vp_catalog* c, int B, const vp_sched_params* p) {
    vp_info I;
    vp_catalog_info(c, &I);
    const size_t N = (size_t)I.N, K = (size_t)p->k_max, b = (size_t)B;
    Carver cv{(char*)base};
    SchedBufs s;
    s.demand = (int64_t*)cv.take(b * N * N * 8);
    s.tau_in = (int64_t*)cv.take(b * 8);
    s.n_steps = (int32_t*)cv.take(b * 4);
    s.chan_id = (int32_t*)cv.take(b * K * 4);
    s.lane_dst = (int16_t*)cv.take(b * K * N * 2);
    s.lane_inst = (uint16_t*)cv.take(b * K * N * 2);
    s.lane_bytes = (int64_t*)cv.take(b * K * N * 8);
    s.send_off = (int64_t*)cv.take(b * (K + 1) * N * 8);
    s.recv_off = (int64_t*)cv.take(b * (K + 1) * N * 8);
    s.tau_out = (int64_t*)cv.take(b * 8);
    s.status = (int32_t*)cv.take(b * 4);
    s.ws_bytes = vp_schedule_workspace_bytes(c, B, p);
    s.ws = cv.take(s.ws_bytes);
    s.total = cv.off;
    return s;
}

#define VP_COPY(dst, src, bytes, kind)                                                        \
    do {                                                                                      \
        if ((bytes) && cudaMemcpyAsync((dst), (src), (bytes), (kind), stream) != cudaSuccess) \
            return VP_E_CUDA;                                                                 \
    } while (0)

// Makes a device current for the lifetime of a call and puts the caller's device back on every way out.
struct DeviceScope {
    int prev = -1;
    bool ok = true;
    explicit DeviceScope(int device) {
        cudaGetDevice(&prev);
        if (prev != device) ok = cudaSetDevice(device) == cudaSuccess;
    }
    ~DeviceScope() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" size_t vp_schedule_host_scratch_bytes(const vp_catalog* c, int B, const vp_sched_params* p) {
    if (!c || !p || B <= 0 || p->k_max <= 0) return 0;
    SchedBufs s = carve_sched(nullptr, c, B, p);
    return s.ws_bytes ? s.total : 0;
}

namespace {

// Copies of one chunk's results to host memory on `stream`.  With used_only the plan arrays come back only up to each
// matrix's n_steps, which must already be in host memory.
int copy_plan_out(const SchedBufs& s, size_t N, size_t K, size_t lo, size_t n, int32_t* n_steps, int32_t* chan_id,
                  int16_t* lane_dst, uint16_t* lane_inst, int64_t* lane_bytes, int64_t* send_off, int64_t* recv_off,
                  bool used_only, cudaStream_t stream) {
    if (!used_only) {
        VP_COPY(chan_id + lo * K, s.chan_id, n * K * 4, cudaMemcpyDeviceToHost);
        VP_COPY(lane_dst + lo * K * N, s.lane_dst, n * K * N * 2, cudaMemcpyDeviceToHost);
        VP_COPY(lane_inst + lo * K * N, s.lane_inst, n * K * N * 2, cudaMemcpyDeviceToHost);
        VP_COPY(lane_bytes + lo * K * N, s.lane_bytes, n * K * N * 8, cudaMemcpyDeviceToHost);
        VP_COPY(send_off + lo * (K + 1) * N, s.send_off, n * (K + 1) * N * 8, cudaMemcpyDeviceToHost);
        if (recv_off) VP_COPY(recv_off + lo * (K + 1) * N, s.recv_off, n * (K + 1) * N * 8, cudaMemcpyDeviceToHost);
        return VP_OK;
    }
    for (size_t m = 0; m < n; m++) {
        const size_t g = lo + m;
        const size_t k = n_steps[g] < 0 ? 0 : ((size_t)n_steps[g] > K ? K : (size_t)n_steps[g]);
        VP_COPY(chan_id + g * K, s.chan_id + m * K, k * 4, cudaMemcpyDeviceToHost);
        VP_COPY(lane_dst + g * K * N, s.lane_dst + m * K * N, k * N * 2, cudaMemcpyDeviceToHost);
        VP_COPY(lane_inst + g * K * N, s.lane_inst + m * K * N, k * N * 2, cudaMemcpyDeviceToHost);
        VP_COPY(lane_bytes + g * K * N, s.lane_bytes + m * K * N, k * N * 8, cudaMemcpyDeviceToHost);
        VP_COPY(send_off + g * (K + 1) * N, s.send_off + m * (K + 1) * N, (k + 1) * N * 8, cudaMemcpyDeviceToHost);
        if (recv_off) VP_COPY(recv_off + g * (K + 1) * N, s.recv_off + m * (K + 1) * N, (k + 1) * N * 8, cudaMemcpyDeviceToHost);
    }
    return VP_OK;
}

// Batches of at least this many matrices are worked through in chunks, two of them in flight: while one chunk is
// decomposed on the caller's stream, the results of the chunk before it travel to the host on a second stream.
constexpr int kPipeMinBatch = 64;

// Both host-buffer scheduler calls: copy in, run vp_schedule_batch, copy out.
int schedule_host(const vp_catalog* cc, const vp_sched_params* p, const int64_t* demand, const int64_t* tau_ns_in, int B,
                  int32_t* n_steps, int32_t* chan_id, int16_t* lane_dst, uint16_t* lane_inst, int64_t* lane_bytes,
                  int64_t* send_off, int64_t* recv_off, int64_t* tau_ns_out, int32_t* status, void* device_scratch,
                  size_t device_scratch_bytes, void* cuda_stream, bool used_only) {
    vp_catalog* c = const_cast<vp_catalog*>(cc);
    if (!c || !p || B <= 0 || p->k_max <= 0 || !demand || !n_steps || !chan_id || !lane_dst || !lane_inst || !lane_bytes ||
        !send_off || !status)
        return VP_E_BAD_ARG;
    if (!device_scratch || ((uintptr_t)device_scratch & 255)) return VP_E_WORKSPACE;
    SchedBufs whole = carve_sched(nullptr, c, B, p);
    if (!whole.ws_bytes) return VP_E_BAD_ARG;
    if (device_scratch_bytes < whole.total) return VP_E_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const size_t N = (size_t)c->info.N, K = (size_t)p->k_max;
    DeviceScope scope(c->device);
    if (!scope.ok) return VP_E_CUDA;

    // chunks: about one matrix per SM each, at least three, and two chunks' buffers must fit the scratch of the whole batch
    int n_chunks = 1, chunk = B;
    if (B >= kPipeMinBatch) {
        n_chunks = B / (c->sm_count > 0 ? c->sm_count : 128);
        if (n_chunks < 3) n_chunks = 3;
        chunk = (B + n_chunks - 1) / n_chunks;
        n_chunks = (B + chunk - 1) / chunk;
        const SchedBufs one = carve_sched(nullptr, c, chunk, p);
        if (!one.ws_bytes || 2 * one.total > device_scratch_bytes) { n_chunks = 1; chunk = B; }
    }
    if (n_chunks > 1 && !c->host_pipe_ready) {
        if (cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return VP_E_CUDA;
        for (cudaEvent_t& e : c->host_ev)
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return VP_E_CUDA;
        c->host_pipe_ready = 1;
    }
    const size_t slot_bytes = n_chunks > 1 ? carve_sched(nullptr, c, chunk, p).total : 0;
    SchedBufs slot[2];
    slot[0] = carve_sched(device_scratch, c, chunk, p);
    slot[1] = n_chunks > 1 ? carve_sched((char*)device_scratch + slot_bytes, c, chunk, p) : slot[0];
    cudaStream_t copy = n_chunks > 1 ? c->copy_stream : stream;
    cudaEvent_t* done = c->host_ev;          // [0], [1]: chunk decomposed;  [2], [3]: its results copied out
    cudaEvent_t* copied = c->host_ev + 2;

    for (int i = 0; i <= n_chunks; i++) {
        if (i < n_chunks) {                  // ---- chunk i: copy in and decompose, on the caller's stream
            const SchedBufs& s = slot[i & 1];
            const size_t lo = (size_t)i * chunk, n = (size_t)(B - (int)lo < chunk ? B - (int)lo : chunk);
            if (n_chunks > 1 && i >= 2 && cudaStreamWaitEvent(stream, copied[i & 1], 0) != cudaSuccess) return VP_E_CUDA;
            VP_COPY(s.demand, demand + lo * N * N, n * N * N * 8, cudaMemcpyHostToDevice);
            if (tau_ns_in) VP_COPY(s.tau_in, tau_ns_in + lo, n * 8, cudaMemcpyHostToDevice);
            const int rc = vp_schedule_batch(c, p, s.demand, tau_ns_in ? s.tau_in : nullptr, (int)n, s.n_steps, s.chan_id,
                                             s.lane_dst, s.lane_inst, s.lane_bytes, s.send_off, recv_off ? s.recv_off : nullptr,
                                             tau_ns_out ? s.tau_out : nullptr, s.status, s.ws, s.ws_bytes, cuda_stream);
            if (rc) return rc;
            if (n_chunks > 1 && cudaEventRecord(done[i & 1], stream) != cudaSuccess) return VP_E_CUDA;
        }
        if (i >= 1 || n_chunks == 1) {       // ---- chunk i - 1 (the only chunk when there is one): results to the host
            const int j = n_chunks == 1 ? 0 : i - 1;
            if (n_chunks == 1 && i == 1) break;
            const SchedBufs& s = slot[j & 1];
            const size_t lo = (size_t)j * chunk, n = (size_t)(B - (int)lo < chunk ? B - (int)lo : chunk);
            if (n_chunks > 1 && cudaStreamWaitEvent(copy, done[j & 1], 0) != cudaSuccess) return VP_E_CUDA;
            {
                cudaStream_t stream = copy;  // (VP_COPY issues on `stream`)
                VP_COPY(n_steps + lo, s.n_steps, n * 4, cudaMemcpyDeviceToHost);
                if (tau_ns_out) VP_COPY(tau_ns_out + lo, s.tau_out, n * 8, cudaMemcpyDeviceToHost);
                VP_COPY(status + lo, s.status, n * 4, cudaMemcpyDeviceToHost);
                if (used_only && cudaStreamSynchronize(copy) != cudaSuccess) return VP_E_CUDA;   // n_steps is needed on the host now
                const int rc = copy_plan_out(s, N, K, lo, n, n_steps, chan_id, lane_dst, lane_inst, lane_bytes, send_off, recv_off,
                                             used_only, copy);
                if (rc) return rc;
            }
            if (n_chunks > 1 && cudaEventRecord(copied[j & 1], copy) != cudaSuccess) return VP_E_CUDA;
        }
    }
    if (n_chunks > 1 && cudaStreamSynchronize(copy) != cudaSuccess) return VP_E_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return VP_E_CUDA;
    return VP_OK;
}

}  // namespace

extern "C" int vp_schedule_batch_host(const vp_catalog* c, const vp_sched_params* p, const int64_t* demand,
                                      const int64_t* tau_ns_in, int B, int32_t* n_steps, int32_t* chan_id,
                                      int16_t* lane_dst, uint16_t* lane_inst, int64_t* lane_bytes, int64_t* send_off,
                                      int64_t* recv_off, int64_t* tau_ns_out, int32_t* status, void* device_scratch,
                                      size_t device_scratch_bytes, void* cuda_stream) {
    return schedule_host(c, p, demand, tau_ns_in, B, n_steps, chan_id, lane_dst, lane_inst, lane_bytes, send_off, recv_off,
                         tau_ns_out, status, device_scratch, device_scratch_bytes, cuda_stream, false);
}

extern "C" int vp_schedule_batch_host_used(const vp_catalog* c, const vp_sched_params* p, const int64_t* demand,
                                           const int64_t* tau_ns_in, int B, int32_t* n_steps, int32_t* chan_id,
                                           int16_t* lane_dst, uint16_t* lane_inst, int64_t* lane_bytes, int64_t* send_off,
                                           int64_t* recv_off, int64_t* tau_ns_out, int32_t* status, void* device_scratch,
                                           size_t device_scratch_bytes, void* cuda_stream) {
    return schedule_host(c, p, demand, tau_ns_in, B, n_steps, chan_id, lane_dst, lane_inst, lane_bytes, send_off, recv_off,
                         tau_ns_out, status, device_scratch, device_scratch_bytes, cuda_stream, true);
}

namespace {

struct PackBufs {
    int32_t *n_steps, *idx, *src_map, *status;
    int16_t* lane_dst;
    int64_t *lane_bytes, *send_off;
    char *rows, *staged;
    void* ws;
    size_t ws_bytes, total;
};

PackBufs carve_pack(void* base, int N, int T, int topk, int k_max, int64_t row_bytes, int64_t cap) {
    Carver cv{(char*)base};
    PackBufs s;
    const size_t K = (size_t)k_max, n = (size_t)N;
    s.n_steps = (int32_t*)cv.take(4);
    s.lane_dst = (int16_t*)cv.take(K * n * 2);
    s.lane_bytes = (int64_t*)cv.take(K * n * 8);
    s.send_off = (int64_t*)cv.take((K + 1) * n * 8);
    s.idx = (int32_t*)cv.take((size_t)T * topk * 4);
    s.rows = (char*)cv.take((size_t)T * row_bytes);
    s.staged = (char*)cv.take((size_t)cap);
    s.src_map = (int32_t*)cv.take((size_t)(cap / row_bytes + 1) * 4);
    s.status = (int32_t*)cv.take(4);
    s.ws_bytes = vp_pack_workspace_bytes(N, T, topk, k_max);
    s.ws = cv.take(s.ws_bytes);
    s.total = cv.off;
    return s;
}

}  // namespace

extern "C" size_t vp_pack_host_scratch_bytes(int N, int T, int topk, int k_max, int64_t row_bytes, int64_t cap) {
    if (N <= 0 || T <= 0 || topk <= 0 || k_max <= 0 || row_bytes <= 0 || cap < 0) return 0;
    PackBufs s = carve_pack(nullptr, N, T, topk, k_max, row_bytes, cap);
    return s.ws_bytes ? s.total : 0;
}

extern "C" int vp_pack_host(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* lane_bytes_b,
                            const int64_t* send_off_b, int N, int rank, int k_max, const int32_t* expert_idx, int T,
                            int topk, int experts_per_rank, const void* rows, int64_t row_bytes, void* staged,
                            int64_t cap, int32_t* src_map, int32_t* status, void* device_scratch,
                            size_t device_scratch_bytes, void* cuda_stream) {
    if (!n_steps_b || !lane_dst_b || !lane_bytes_b || !send_off_b || !expert_idx || !rows || !staged || !status)
        return VP_E_BAD_ARG;
    if (N <= 0 || T <= 0 || topk <= 0 || k_max <= 0 || row_bytes <= 0 || cap < 0) return VP_E_BAD_ARG;
    if (!device_scratch || ((uintptr_t)device_scratch & 255)) return VP_E_WORKSPACE;
    PackBufs s = carve_pack(device_scratch, N, T, topk, k_max, row_bytes, cap);
    if (!s.ws_bytes) return VP_E_BAD_ARG;
    if (device_scratch_bytes < s.total) return VP_E_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const size_t K = (size_t)k_max, n = (size_t)N;
    VP_COPY(s.n_steps, n_steps_b, 4, cudaMemcpyHostToDevice);
    VP_COPY(s.lane_dst, lane_dst_b, K * n * 2, cudaMemcpyHostToDevice);
    VP_COPY(s.lane_bytes, lane_bytes_b, K * n * 8, cudaMemcpyHostToDevice);
    VP_COPY(s.send_off, send_off_b, (K + 1) * n * 8, cudaMemcpyHostToDevice);
    VP_COPY(s.idx, expert_idx, (size_t)T * topk * 4, cudaMemcpyHostToDevice);
    VP_COPY(s.rows, rows, (size_t)T * row_bytes, cudaMemcpyHostToDevice);
    int rc = vp_pack(s.n_steps, s.lane_dst, s.lane_bytes, s.send_off, N, rank, k_max, s.idx, T, topk, experts_per_rank,
                     s.rows, row_bytes, s.staged, cap, src_map ? s.src_map : nullptr, s.status, s.ws, s.ws_bytes,
                     cuda_stream);
    if (rc) return rc;
    VP_COPY(status, s.status, 4, cudaMemcpyDeviceToHost);
    if (cudaStreamSynchronize(stream) != cudaSuccess) return VP_E_CUDA;
    // only the bytes the plan covers come back: the send volume is send_off[n_steps][rank]
    const int K_used = *n_steps_b < 0 ? 0 : (*n_steps_b > k_max ? k_max : *n_steps_b);
    int64_t used = send_off_b[(size_t)K_used * n + rank];
    if (used < 0) used = 0;
    if (used > cap) used = cap;
    if (!(*status & VP_ST_PACK_CAPACITY)) {
        VP_COPY(staged, s.staged, (size_t)used, cudaMemcpyDeviceToHost);
        if (src_map) VP_COPY(src_map, s.src_map, (size_t)(used / row_bytes) * 4, cudaMemcpyDeviceToHost);
    }
    if (cudaStreamSynchronize(stream) != cudaSuccess) return VP_E_CUDA;
    return VP_OK;
}
