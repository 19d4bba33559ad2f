// vp_schedule_batch: Algorithm 2 (Section 4.2) for a batch of demand matrices.
//
// One CTA decomposes one matrix at a time (persistent CTAs pull matrix indices
// from a counter).  The residual demand D_rem lives in shared memory when
// N <= 64 and in an L2-resident workspace slot otherwise; the group sums D-hat
// are kept in shared memory and updated incrementally after every activation.
// Per iteration: (A) every thread scores shapes (Eq. 6) and a block-wide
// (value, lowest index) arg-max picks M*; (B) every (family, start) pair of
// the bucket is one warp-level task that runs the Alternating Algorithm, one
// lane per rank group, each lane solving its g x g assignment by enumerating
// the g! permutations in lexicographic order (Eq. 7, 8) and then evaluating
// Eq. (9), (10); (C) warp 0 picks the best start per family and the family of
// largest utility by exact 128-bit cross-multiplication; (D) all threads emit
// the activation, subtract it from D_rem / D-hat and advance the running
// send / receive offsets.
#include <cuda_runtime.h>

#include <utility>

#include "vp_internal.h"

namespace {

struct KParams {
    int64_t lambda_ns, granule;
    int k_target, n_start, i_aa, k_max;
    int max_tasks;
};

struct Smem {                 // offsets (bytes) into dynamic shared memory
    int drem, dhat, tbl, send_acc, recv_acc, red, task_f, task_den, bind_src, bind_dst, total;
};

__host__ __device__ inline Smem smem_layout(const DevCat& dc, int max_tasks, bool drem_in_smem) {
    Smem L;
    int o = 0;
    L.drem = o;      o += drem_in_smem ? dc.N * dc.N * 8 : 0;
    L.dhat = o;      o += dc.G * dc.G * 8;
    L.tbl = o;       o += dc.sym ? dc.tbl_size * 8 : 0;
    L.send_acc = o;  o += dc.N * 8;
    L.recv_acc = o;  o += dc.N * 8;
    L.red = o;       o += 64 * 8;
    L.task_f = o;    o += max_tasks * 8;
    L.task_den = o;  o += max_tasks * 8;
    L.bind_src = o;  o += (max_tasks * dc.N + 15) & ~15;
    L.bind_dst = o;  o += (max_tasks * dc.N + 15) & ~15;
    L.total = o;
    return L;
}

__device__ __forceinline__ int64_t min_i64(int64_t a, int64_t b) { return a < b ? a : b; }
__device__ __forceinline__ int64_t max_i64(int64_t a, int64_t b) { return a > b ? a : b; }
__device__ __forceinline__ int64_t ceil_div_i64(int64_t a, int64_t b) { return (a + b - 1) / b; }

// q-th element of the p-th lexicographic permutation of g items (factorial number system)
__host__ __device__ constexpr int perm_entry(int g, int p, int q) {
    int avail[4] = {0, 1, 2, 3};
    int fact[4] = {1, 1, 2, 6};
    int rem = p, out = 0;
    for (int pos = 0; pos <= q; pos++) {
        int f = fact[g - 1 - pos];
        int idx = rem / f;
        rem = rem % f;
        out = avail[idx];
        for (int k = idx; k < 3; k++) avail[k] = avail[k + 1];
    }
    return out;
}
__host__ __device__ constexpr int factorial(int g) { return g <= 1 ? 1 : g * factorial(g - 1); }
__host__ __device__ constexpr unsigned perm_packed(int g, int p) {   // 2 bits per position, position 0 lowest
    unsigned w = 0;
    for (int q = 0; q < g; q++) w |= (unsigned)perm_entry(g, p, q) << (2 * q);
    return w;
}
template <int GS, int P, int Q> struct PermAt { static constexpr int value = perm_entry(GS, P, Q); };
template <int GS, int P> struct PermPacked { static constexpr unsigned value = perm_packed(GS, P); };

template <int GS, int P, int... Q>
__device__ __forceinline__ int64_t perm_value(const int64_t (&c)[GS][GS], std::integer_sequence<int, Q...>) {
    return (c[PermAt<GS, P, Q>::value][Q] + ...);
}
template <int GS, int P>
__device__ __forceinline__ void perm_try(const int64_t (&c)[GS][GS], int64_t& best, unsigned& bpk) {
    const int64_t v = perm_value<GS, P>(c, std::make_integer_sequence<int, GS>{});
    if (v > best) { best = v; bpk = PermPacked<GS, P>::value; }
}
template <int GS, int... P>
__device__ __forceinline__ int64_t best_assignment_impl(const int64_t (&c)[GS][GS], unsigned& bpk,
                                                        std::integer_sequence<int, P...>) {
    int64_t best = -1;
    bpk = 0;
    (perm_try<GS, P>(c, best, bpk), ...);
    return best;
}
// Exact g x g assignment: maximise sum_q c[phi(q)][q] over all g! permutations, enumerated in
// lexicographic order of (phi(0), ..., phi(g-1)); the first maximum wins.
template <int GS>
__device__ __forceinline__ int64_t best_assignment(const int64_t (&c)[GS][GS], int (&phi)[GS]) {
    unsigned bpk;
    const int64_t best = best_assignment_impl<GS>(c, bpk, std::make_integer_sequence<int, factorial(GS)>{});
#pragma unroll
    for (int q = 0; q < GS; q++) phi[q] = (int)((bpk >> (2 * q)) & 3u);
    return best;
}

__device__ __forceinline__ int64_t warp_sum_i64(int64_t v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int64_t warp_max_i64(int64_t v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = max_i64(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// f1/d1 > f2/d2, exactly, by 128-bit cross-multiplication (all four in [0, 2^63)).
__device__ __forceinline__ bool util_greater(int64_t f1, int64_t d1, int64_t f2, int64_t d2) {
    unsigned long long a = (unsigned long long)f1, b = (unsigned long long)d2;
    unsigned long long c = (unsigned long long)f2, d = (unsigned long long)d1;
    unsigned long long hi1 = __umul64hi(a, b), lo1 = a * b, hi2 = __umul64hi(c, d), lo2 = c * d;
    return hi1 > hi2 || (hi1 == hi2 && lo1 > lo2);
}

template <int GS>
__global__ void __launch_bounds__(512)
vp_schedule_kernel(DevCat dc, KParams kp, const int64_t* __restrict__ demand, const int64_t* __restrict__ tau_in, int B,
                   int32_t* __restrict__ n_steps, int32_t* __restrict__ chan_id, int16_t* __restrict__ lane_dst,
                   uint16_t* __restrict__ lane_inst, int64_t* __restrict__ lane_bytes, int64_t* __restrict__ send_off,
                   int64_t* __restrict__ recv_off, int64_t* __restrict__ tau_out, int32_t* __restrict__ status,
                   int64_t* ws_drem, unsigned int* counter, int drem_in_smem) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const Smem L = smem_layout(dc, kp.max_tasks, drem_in_smem != 0);
    const int N = dc.N, G = dc.G, tid = threadIdx.x, NT = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, n_warps = NT >> 5;
    int64_t* Drem = drem_in_smem ? (int64_t*)(smem_raw + L.drem) : ws_drem + (size_t)blockIdx.x * N * N;
    int64_t* Dhat = (int64_t*)(smem_raw + L.dhat);
    int64_t* tbl = dc.sym ? (int64_t*)(smem_raw + L.tbl) : Dhat;
    int64_t* send_acc = (int64_t*)(smem_raw + L.send_acc);
    int64_t* recv_acc = (int64_t*)(smem_raw + L.recv_acc);
    int64_t* red = (int64_t*)(smem_raw + L.red);
    int64_t* task_f = (int64_t*)(smem_raw + L.task_f);
    int64_t* task_den = (int64_t*)(smem_raw + L.task_den);
    uint8_t* bind_src = smem_raw + L.bind_src;
    uint8_t* bind_dst = smem_raw + L.bind_dst;
    __shared__ int s_b, s_flags, s_shape, s_task;
    unsigned long long n_act = 0, n_tasks_done = 0, n_sweeps = 0;     // work counters (per warp / thread 0)
    __shared__ int64_t s_tau, s_left, s_score;
    __shared__ int64_t s_cap[VP_MAX_CLASSES];

    for (;;) {
        if (tid == 0) { s_b = (int)atomicAdd(counter, 1u); s_flags = 0; }
        __syncthreads();
        const int b = s_b;
        if (b >= B) break;
        const int64_t* D = demand + (size_t)b * N * N;
        const size_t lane_base = (size_t)b * kp.k_max * N, off_base = (size_t)b * (kp.k_max + 1) * N;

        // ---- validate, copy D into D_rem
        int flags = 0;
        for (int e = tid; e < N * N; e += NT) {
            int64_t v = D[e];
            if (v < 0) flags |= VP_ST_NEGATIVE;
            else if (v >= VP_ENTRY_LIMIT) flags |= VP_ST_OVERFLOW_RISK;
            else {
                if (e / N == e % N && v != 0) flags |= VP_ST_DIAG_NONZERO;
                if (v % kp.granule) flags |= VP_ST_NOT_GRANULE;
            }
            Drem[e] = v;
        }
        const int64_t tau_given = tau_in ? tau_in[b] : 0;
        if (tid == 0 && (tau_given < 0 || tau_given > VP_ENTRY_LIMIT)) flags |= VP_ST_BAD_TAU;
        if (flags) atomicOr(&s_flags, flags);
        for (int i = tid; i < N; i += NT) {
            send_acc[i] = 0; recv_acc[i] = 0;
            send_off[off_base + i] = 0;
            if (recv_off) recv_off[off_base + i] = 0;
        }
        __syncthreads();
        int st = s_flags;
        int k = 0;
        int64_t tau = 0;
        if (st == 0) {
            // ---- row / column sums, group sums (Eq. 5), quantum (Section 5)
            int64_t est = 0, tot = 0;
            for (int i = tid; i < N; i += NT) {
                int64_t row = 0, col = 0;
                for (int jj = 0; jj < N; jj++) {
                    int j = jj + i; if (j >= N) j -= N;
                    row += Drem[(size_t)i * N + j];
                    col += Drem[(size_t)j * N + i];
                }
                tot += row;
                est = max_i64(est, max_i64(ceil_div_i64(row, dc.bw_max), ceil_div_i64(col, dc.bw_max)));
            }
            for (int cell = tid; cell < G * G; cell += NT) {
                int a = cell / G, d = cell % G;
                int64_t s = 0;
#pragma unroll
                for (int i = 0; i < GS; i++)
#pragma unroll
                    for (int j = 0; j < GS; j++) s += Drem[(size_t)(a * GS + i) * N + d * GS + j];
                Dhat[cell] = s;
            }
            __syncthreads();
            for (int l = tid; l < dc.n_res; l += NT) {
                uint32_t bwl = dc.forced_bw[l];
                if (!bwl) continue;
                int64_t f = 0;
                for (uint32_t e = dc.forced_ptr[l]; e < dc.forced_ptr[l + 1]; e++) f += Dhat[dc.forced_cell[e]];
                est = max_i64(est, ceil_div_i64(f, (int64_t)bwl));
            }
            est = warp_max_i64(est);
            tot = warp_sum_i64(tot);
            if (lane == 0) { red[warp] = est; red[32 + warp] = tot; }
            __syncthreads();
            if (tid == 0) {
                int64_t e = 0, t = 0;
                for (int w = 0; w < n_warps; w++) { e = max_i64(e, red[w]); t += red[32 + w]; }
                int64_t tq = tau_given > 0 ? tau_given : max_i64(1, ceil_div_i64(e, (int64_t)kp.k_target));
                s_tau = tq; s_left = t;
                for (int c = 0; c < dc.n_classes; c++) {
                    int64_t cap = (tq * dc.class_bw[c]) / kp.granule * kp.granule;
                    s_cap[c] = cap < kp.granule ? kp.granule : cap;
                }
            }
            __syncthreads();
            tau = s_tau;

            // ---- Algorithm 2 main loop
            for (;;) {
                if (s_left == 0) break;
                if (k == kp.k_max) { st |= VP_ST_STEP_LIMIT; break; }
                // (A) Eq. (6): shape scores, first maximum
                if (dc.sym) {
                    const int S = dc.S, P = dc.P;
                    for (int e = tid; e < dc.tbl_size; e += NT) {
                        int q2 = e % S, q = (e / S) % S, delta = e / (S * S);
                        int64_t s = 0;
                        for (int n = 0; n < P; n++) {
                            int n2 = n + delta; if (n2 >= P) n2 -= P;
                            s += Dhat[(size_t)(n * S + q) * G + n2 * S + q2];
                        }
                        tbl[e] = s;
                    }
                    __syncthreads();
                }
                int64_t best = -1;
                int best_s = 0x7fffffff;
                for (int s = tid; s < dc.n_shapes; s += NT) {
                    int64_t score = 0;
                    for (uint32_t e = dc.shape_ptr[s]; e < dc.shape_ptr[s + 1]; e++) {
                        uint32_t w = __ldg(&dc.term[e]);
                        score += tbl[w & 0xffffu] * (int64_t)(w >> 16);
                    }
                    if (score > best) { best = score; best_s = s; }     // ascending s: keeps the first maximum
                }
#pragma unroll
                for (int o = 16; o; o >>= 1) {
                    int64_t ov = __shfl_xor_sync(0xffffffffu, best, o);
                    int oi = __shfl_xor_sync(0xffffffffu, best_s, o);
                    if (ov > best || (ov == best && oi < best_s)) { best = ov; best_s = oi; }
                }
                if (lane == 0) { red[warp] = best; red[32 + warp] = best_s; }
                __syncthreads();
                if (tid == 0) {
                    int64_t bv = -1; int bi = 0x7fffffff;
                    for (int w = 0; w < n_warps; w++)
                        if (red[w] > bv || (red[w] == bv && (int)red[32 + w] < bi)) { bv = red[w]; bi = (int)red[32 + w]; }
                    s_score = bv; s_shape = bi;
                }
                __syncthreads();
                if (s_score <= 0) { st |= VP_ST_UNCOVERED; break; }
                const int f0 = (int)dc.bucket_ptr[s_shape], H = (int)dc.bucket_ptr[s_shape + 1] - f0;
                const int n_tasks = H * kp.n_start;

                // (B) MultiStartAA: one warp per (family, start), one lane per rank group
                for (int task = warp; task < n_tasks; task += n_warps) {
                    const int f = f0 + task / kp.n_start, t = task % kp.n_start;
                    const uint32_t* slot = dc.fam_slot + (size_t)f * N;
                    const uint8_t* inslot = dc.fam_inslot + (size_t)f * N;
                    uint8_t* srcb = bind_src + (size_t)task * N;
                    uint8_t* dstb = bind_dst + (size_t)task * N;
                    for (int d = lane; d < G; d += 32)
#pragma unroll
                        for (int q = 0; q < GS; q++) dstb[inslot[d * GS + q]] = (uint8_t)(d * GS + (q + t) % GS);
                    __syncwarp();
                    int64_t F_old = -1, F_new = -1;
                    for (int sweep = 0; sweep < kp.i_aa; sweep++) {
                        for (int a = lane; a < G; a += 32) {            // source half
                            int64_t c[GS][GS];
                            int phi[GS];
#pragma unroll
                            for (int q = 0; q < GS; q++) {
                                const int r = a * GS + q;
                                const int64_t cap = s_cap[(__ldg(&slot[r]) >> 24) & 0xf];
                                const int dq = dstb[r];
#pragma unroll
                                for (int i = 0; i < GS; i++) c[i][q] = min_i64(Drem[(size_t)(a * GS + i) * N + dq], cap);
                            }
                            best_assignment<GS>(c, phi);
#pragma unroll
                            for (int q = 0; q < GS; q++) srcb[a * GS + q] = (uint8_t)(a * GS + phi[q]);
                        }
                        __syncwarp();
                        int64_t part = 0;
                        for (int d = lane; d < G; d += 32) {            // destination half
                            int64_t c[GS][GS];
                            int phi[GS], rq[GS];
#pragma unroll
                            for (int q = 0; q < GS; q++) {
                                rq[q] = inslot[d * GS + q];
                                const int64_t cap = s_cap[(__ldg(&slot[rq[q]]) >> 24) & 0xf];
                                const int sq = srcb[rq[q]];
#pragma unroll
                                for (int j = 0; j < GS; j++) c[j][q] = min_i64(Drem[(size_t)sq * N + d * GS + j], cap);
                            }
                            part += best_assignment<GS>(c, phi);
#pragma unroll
                            for (int q = 0; q < GS; q++) dstb[rq[q]] = (uint8_t)(d * GS + phi[q]);
                        }
                        __syncwarp();
                        F_new = warp_sum_i64(part);                      // Eq. (8), in bytes
                        n_sweeps++;
                        if (F_new <= F_old) break;
                        F_old = F_new;
                    }
                    int64_t tmax = 0;                                    // Eq. (9), slowest lane of Eq. (10)
                    for (int r = lane; r < N; r += 32) {
                        const int cls = (__ldg(&slot[r]) >> 24) & 0xf;
                        const int64_t x = min_i64(s_cap[cls], Drem[(size_t)srcb[r] * N + dstb[r]]);
                        tmax = max_i64(tmax, x * dc.class_wdiv[cls]);
                    }
                    tmax = warp_max_i64(tmax);
                    n_tasks_done++;
                    if (lane == 0) {
                        task_f[task] = F_new;
                        task_den[task] = F_new > 0 ? kp.lambda_ns * dc.W + tmax : 1;
                    }
                }
                __syncthreads();

                // (C) best start per family (largest F, lowest t), then largest utility, lowest family
                if (warp == 0) {
                    int64_t bf = -1, bd = 1;
                    int bt = 0x7fffffff;
                    for (int h = lane; h < H; h += 32) {
                        int64_t ff = -1; int tt = 0;
                        for (int t = 0; t < kp.n_start; t++)
                            if (task_f[h * kp.n_start + t] > ff) { ff = task_f[h * kp.n_start + t]; tt = h * kp.n_start + t; }
                        if (bt == 0x7fffffff || util_greater(ff, task_den[tt], bf, bd)) { bf = ff; bd = task_den[tt]; bt = tt; }
                    }
#pragma unroll
                    for (int o = 16; o; o >>= 1) {
                        int64_t of = __shfl_xor_sync(0xffffffffu, bf, o), od = __shfl_xor_sync(0xffffffffu, bd, o);
                        int ot = __shfl_xor_sync(0xffffffffu, bt, o);
                        bool take = false;
                        if (ot != 0x7fffffff) {
                            if (bt == 0x7fffffff) take = true;
                            else if (util_greater(of, od, bf, bd)) take = true;
                            else if (!util_greater(bf, bd, of, od) && ot < bt) take = true;
                        }
                        if (take) { bf = of; bd = od; bt = ot; }
                    }
                    if (lane == 0) { s_task = bt; red[0] = bf; }
                }
                __syncthreads();
                const int wtask = s_task;
                const int64_t wF = red[0];
                if (wF <= 0) { st |= VP_ST_NO_PROGRESS; break; }

                // (D) emit activation k, D_rem -= X(E), update D-hat and the running offsets
                {
                    const int f = f0 + wtask / kp.n_start;
                    const uint32_t* slot = dc.fam_slot + (size_t)f * N;
                    const uint8_t* srcb = bind_src + (size_t)wtask * N;
                    const uint8_t* dstb = bind_dst + (size_t)wtask * N;
                    const size_t row = lane_base + (size_t)k * N;
                    for (int r = tid; r < N; r += NT) {
                        const uint32_t w = __ldg(&slot[r]);
                        const int i = srcb[r], j = dstb[r];
                        const int64_t x = min_i64(s_cap[(w >> 24) & 0xf], Drem[(size_t)i * N + j]);
                        if (x > 0) {
                            lane_dst[row + i] = (int16_t)j;
                            lane_inst[row + i] = (uint16_t)(w & 0xffffu);
                            lane_bytes[row + i] = x;
                            Drem[(size_t)i * N + j] -= x;
                            atomicAdd((unsigned long long*)&Dhat[(i / GS) * G + (j / GS)], (unsigned long long)(-x));
                            send_acc[i] += x;
                            recv_acc[j] += x;
                        } else {
                            lane_dst[row + i] = -1;
                            lane_inst[row + i] = 0xFFFF;
                            lane_bytes[row + i] = 0;
                        }
                    }
                    if (tid == 0) { chan_id[(size_t)b * kp.k_max + k] = f; s_left -= wF; }
                }
                __syncthreads();
                k++;
                for (int i = tid; i < N; i += NT) {
                    send_off[off_base + (size_t)k * N + i] = send_acc[i];
                    if (recv_off) recv_off[off_base + (size_t)k * N + i] = recv_acc[i];
                }
            }
        }
        __syncthreads();
        // ---- idle rows beyond n_steps; offset rows repeat the totals
        for (size_t e = (size_t)k * N + tid; e < (size_t)kp.k_max * N; e += NT) {
            lane_dst[lane_base + e] = -1;
            lane_inst[lane_base + e] = 0xFFFF;
            lane_bytes[lane_base + e] = 0;
            const int i = (int)(e % N);
            send_off[off_base + N + e] = send_acc[i];
            if (recv_off) recv_off[off_base + N + e] = recv_acc[i];
        }
        for (int kk = k + tid; kk < kp.k_max; kk += NT) chan_id[(size_t)b * kp.k_max + kk] = -1;
        if (tid == 0) {
            n_act += (unsigned long long)k;
            n_steps[b] = k;
            status[b] = st;
            if (tau_out) tau_out[b] = tau;
        }
        __syncthreads();
    }
    unsigned long long* stats = (unsigned long long*)(counter + 4);
    if (tid == 0 && n_act) atomicAdd(&stats[0], n_act);
    if (lane == 0 && n_tasks_done) { atomicAdd(&stats[1], n_tasks_done); atomicAdd(&stats[2], n_sweeps); }
}

struct Launch {
    int threads, grid, drem_in_smem, max_tasks;
    size_t smem;
};

template <int GS>
int plan_launch(const vp_catalog* c, int B, const KParams& kp, Launch* out) {
    const DevCat& dc = c->dc;
    Launch L;
    L.max_tasks = kp.max_tasks;
    L.threads = dc.N <= 16 ? 128 : (dc.N <= 64 ? 256 : 512);
    L.drem_in_smem = dc.N <= 64;
    L.smem = (size_t)smem_layout(dc, kp.max_tasks, L.drem_in_smem).total;
    if (L.smem + 1024 > (size_t)c->max_smem_optin) return VP_E_UNSUPPORTED;
    if (cudaFuncSetAttribute(vp_schedule_kernel<GS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.smem) != cudaSuccess)
        return VP_E_CUDA;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, vp_schedule_kernel<GS>, L.threads, L.smem) != cudaSuccess || per_sm < 1)
        return VP_E_CUDA;
    long long cap = (long long)per_sm * c->sm_count;
    L.grid = (int)(B < cap ? B : cap);
    *out = L;
    return VP_OK;
}

int resolve_params(const vp_catalog* c, const vp_sched_params* p, KParams* kp) {
    if (!c || !p) return VP_E_BAD_ARG;
    if (p->k_max <= 0 || p->granule_bytes <= 0 || p->lambda_ns < 0 || p->lambda_ns >= VP_ENTRY_LIMIT) return VP_E_BAD_ARG;
    if (p->k_target < 0 || p->n_start < 0 || p->i_aa < 0 || p->n_start > 64) return VP_E_BAD_ARG;
    kp->lambda_ns = p->lambda_ns; kp->granule = p->granule_bytes;
    kp->k_target = p->k_target ? p->k_target : 2 * c->dc.N;
    kp->n_start = p->n_start ? p->n_start : c->dc.g;
    kp->i_aa = p->i_aa ? p->i_aa : 3;
    kp->k_max = p->k_max;
    kp->max_tasks = c->dc.max_bucket * kp->n_start;
    return VP_OK;
}

int plan_any(const vp_catalog* c, int B, const KParams& kp, Launch* L) {
    switch (c->dc.g) {
        case 1: return plan_launch<1>(c, B, kp, L);
        case 2: return plan_launch<2>(c, B, kp, L);
        case 3: return plan_launch<3>(c, B, kp, L);
        case 4: return plan_launch<4>(c, B, kp, L);
    }
    return VP_E_UNSUPPORTED;
}

size_t workspace_bytes(const vp_catalog* c, const Launch& L) {
    size_t drem = L.drem_in_smem ? 0 : (size_t)L.grid * c->dc.N * c->dc.N * 8;
    return vp_align256(256 + drem);
}

}  // namespace

extern "C" size_t vp_schedule_workspace_bytes(const vp_catalog* c, int B, const vp_sched_params* p) {
    KParams kp;
    Launch L;
    if (B <= 0 || resolve_params(c, p, &kp) != VP_OK) return 0;
    int prev = -1;
    cudaGetDevice(&prev);
    cudaSetDevice(c->device);
    int rc = plan_any(c, B, kp, &L);
    if (prev >= 0) cudaSetDevice(prev);
    return rc == VP_OK ? workspace_bytes(c, L) : 0;
}

extern "C" int vp_schedule_batch(const vp_catalog* c, const vp_sched_params* p, const int64_t* demand,
                                 const int64_t* tau_ns_in, int B, int32_t* n_steps, int32_t* chan_id,
                                 int16_t* lane_dst, uint16_t* lane_inst, int64_t* lane_bytes, int64_t* send_off,
                                 int64_t* recv_off, int64_t* tau_ns_out, int32_t* status, void* workspace,
                                 size_t workspace_bytes_given, void* cuda_stream) {
    KParams kp;
    int rc = resolve_params(c, p, &kp);
    if (rc) return rc;
    if (B <= 0 || !demand || !n_steps || !chan_id || !lane_dst || !lane_inst || !lane_bytes || !send_off || !status)
        return VP_E_BAD_ARG;
    int prev = -1;
    cudaGetDevice(&prev);
    if (cudaSetDevice(c->device) != cudaSuccess) return VP_E_CUDA;
    Launch L;
    rc = plan_any(c, B, kp, &L);
    if (!rc && (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes_given < workspace_bytes(c, L))) rc = VP_E_WORKSPACE;
    if (!rc) {
        cudaStream_t stream = (cudaStream_t)cuda_stream;
        unsigned int* counter = (unsigned int*)workspace;
        int64_t* ws_drem = (int64_t*)((char*)workspace + 256);
        if (cudaMemsetAsync(counter, 0, 256, stream) != cudaSuccess) rc = VP_E_CUDA;
#define VP_LAUNCH(GS)                                                                                           \
    vp_schedule_kernel<GS><<<L.grid, L.threads, L.smem, stream>>>(c->dc, kp, demand, tau_ns_in, B, n_steps,     \
        chan_id, lane_dst, lane_inst, lane_bytes, send_off, recv_off, tau_ns_out, status, ws_drem, counter,     \
        L.drem_in_smem)
        if (!rc) {
            vp_prof_mark(0, 0, stream);
            switch (c->dc.g) {
                case 1: VP_LAUNCH(1); break;
                case 2: VP_LAUNCH(2); break;
                case 3: VP_LAUNCH(3); break;
                case 4: VP_LAUNCH(4); break;
            }
            g_vp_launches++;
            if (cudaGetLastError() != cudaSuccess) rc = VP_E_CUDA;
            vp_prof_mark(0, 1, stream);
        }
#undef VP_LAUNCH
    }
    if (prev >= 0) cudaSetDevice(prev);
    return rc;
}

extern "C" int vp_schedule_read_stats(const void* workspace, void* cuda_stream, uint64_t* out3) {
    if (!workspace || !out3) return VP_E_BAD_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(out3, (const char*)workspace + 16, 24, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return VP_E_CUDA;
    return cudaStreamSynchronize(stream) == cudaSuccess ? VP_OK : VP_E_CUDA;
}
