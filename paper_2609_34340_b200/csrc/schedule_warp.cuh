// Algorithm 2 with ONE WARP per demand matrix, for catalogs of at most four groups of four ranks (N <= 16).
//
// A matrix this small has too little work per phase for a whole CTA: with several warps per matrix most of an
// iteration is spent in block barriers and in hand-overs through shared memory.  Here a warp owns a matrix from
// the first to the last activation and nothing but __syncwarp orders its phases:
//  (A) each lane scores every 32nd shape (Eq. 6); a butterfly of shuffles leaves the first maximum in all lanes;
//  (B) the (family, start) tasks of the bucket run four at a time IN THE SAME WARP as independent instruction
//      streams: the lanes keep their role (a team of eight lanes per rank group, three permutations per lane) and
//      issue every step of the Alternating Algorithm (Eq. 7, 8) for the four tasks back to back, so the four
//      dependent chains overlap; a task that stops improving is frozen (its stores are predicated off) while
//      the others finish; Evaluate (Eq. 9, 10) and the best start / best family follow in registers;
//  (D) sixteen lanes emit the activation and subtract it; D-hat is then re-summed from D_rem by all lanes
//      (two lanes per cell), which needs no atomics.
// A CTA is one to four such warps that share only the staged catalog.  Included by schedule.cu.
#pragma once

namespace {

constexpr int kWT = 4;                      // tasks in flight per warp

struct WarpSmem {                           // byte offsets; the per-warp block comes first, once per warp
    int drem, dhat, send_acc, recv_acc, cred, cap64, tscale, cap32, bind_src, bind_dst, per_warp;
    int term, fam_in, fam_cls, fam_slot, bucket, lut, total;
};

__host__ __device__ inline WarpSmem warp_smem_layout(const DevCat& dc, const KParams& kp, int n_warps) {
    WarpSmem L;
    int o = 0;
    L.drem = o;      o += align16(dc.N * (dc.N + 1) * 8);      // rows padded by one element: no bank conflicts down a column
    L.dhat = o;      o += align16(dc.G * dc.G * 8);
    L.send_acc = o;  o += dc.N * 8;
    L.recv_acc = o;  o += dc.N * 8;
    L.cred = o;      o += kWT * 4 * 17 * 8;
    L.cap64 = o;     o += VP_MAX_CLASSES * 8;
    L.tscale = o;    o += VP_MAX_CLASSES * 8;
    L.cap32 = o;     o += VP_MAX_CLASSES * 4;
    L.bind_src = o;  o += align16(kp.max_tasks * dc.N);
    L.bind_dst = o;  o += align16(kp.max_tasks * dc.N);
    L.per_warp = align16(o);
    o = L.per_warp * n_warps;
    L.term = o;      o += ((dc.n_shapes + 31) & ~31) * dc.max_terms * 4;
    L.fam_slot = o;  o += align16(dc.n_families * dc.N * 4);
    L.fam_in = o;    o += align16(dc.n_families * dc.N * 2);
    L.fam_cls = o;   o += align16(dc.n_families * dc.N);
    L.bucket = o;    o += align16((dc.n_shapes + 1) * 4);
    L.lut = o;       o += 32;
    L.total = o;
    return L;
}


extern __shared__ __align__(16) unsigned char vp_wsmem[];   // the CTA's dynamic shared memory

// Shared-memory byte offsets (into vp_wsmem) and output pointers of one warp's matrix.  Offsets rather than
// pointers: every access is then provably a shared-memory access with a 32-bit address.
struct WCtx {
    int N, G, lane;
    unsigned o_drem, o_dhat, o_send_acc, o_recv_acc, o_cred, o_cap, o_tscale, o_bind_src, o_bind_dst;
    unsigned o_term, o_fam_slot, o_fam_in, o_fam_cls, o_bucket, o_lut;
    int32_t* chan_id_b;
    int16_t* lane_dst_b;
    uint16_t* lane_inst_b;
    int64_t *lane_bytes_b, *send_off_b, *recv_off_b;
};

template <typename T> __device__ __forceinline__ T* ws(unsigned off) { return (T*)(vp_wsmem + off); }

// team_best for kWT credit tiles at once, written level by level so that the shuffles of the four tasks are
// issued back to back (shuffles are not reordered by the compiler).
__device__ __forceinline__ void team_best_x(const unsigned (&tile)[kWT], int tl, const uint8_t (&pidx)[3][4], unsigned o_lut,
                                            unsigned (&bpk)[kWT], uint32_t (&val)[kWT]) {
    const Reg8Lane L = reg8_lane(tl);
    uint32_t key[kWT];
#pragma unroll
    for (int t = 0; t < kWT; t++) key[t] = reg8_key(ws<uint32_t>(tile[t]), L);
#pragma unroll
    for (int o = 4; o; o >>= 1) {
        uint32_t other[kWT];
#pragma unroll
        for (int t = 0; t < kWT; t++) other[t] = __shfl_xor_sync(0xffffffffu, key[t], o);
#pragma unroll
        for (int t = 0; t < kWT; t++) key[t] = max_v(key[t], other[t]);
    }
#pragma unroll
    for (int t = 0; t < kWT; t++) { bpk[t] = ~key[t] & 255u; val[t] = key[t] >> 8; }      // the permutation byte, the sum
}
__device__ __forceinline__ void team_best_x(const unsigned (&tile)[kWT], int tl, const uint8_t (&pidx)[3][4], unsigned o_lut,
                                            unsigned (&bpk)[kWT], int64_t (&val)[kWT]) {
    int bp[kWT];
#pragma unroll
    for (int t = 0; t < kWT; t++) {
        const int64_t* cred = ws<int64_t>(tile[t]);
        val[t] = -1; bp[t] = 0;
#pragma unroll
        for (int pp = 0; pp < 3; pp++) {
            const int64_t v = cred[pidx[pp][0]] + cred[pidx[pp][1]] + cred[pidx[pp][2]] + cred[pidx[pp][3]];
            if (v > val[t]) { val[t] = v; bp[t] = tl * 3 + pp; }
        }
    }
#pragma unroll
    for (int o = 4; o; o >>= 1) {
        int64_t ov[kWT];
        int op[kWT];
#pragma unroll
        for (int t = 0; t < kWT; t++) { ov[t] = __shfl_xor_sync(0xffffffffu, val[t], o); op[t] = __shfl_xor_sync(0xffffffffu, bp[t], o); }
#pragma unroll
        for (int t = 0; t < kWT; t++)
            if (ov[t] > val[t] || (ov[t] == val[t] && op[t] < bp[t])) { val[t] = ov[t]; bp[t] = op[t]; }
    }
#pragma unroll
    for (int t = 0; t < kWT; t++) bpk[t] = ws<uint8_t>(o_lut)[31 - bp[t]];
}

// Eq. (8): sum over the teams of a per-team value (held by every lane of the team); every lane gets the totals.
__device__ __forceinline__ void team_totals(const uint32_t (&v)[kWT], bool first_lane_of_active_team, int64_t (&F)[kWT]) {
#pragma unroll
    for (int t = 0; t < kWT; t++) F[t] = (int64_t)__reduce_add_sync(0xffffffffu, first_lane_of_active_team ? v[t] : 0u);
}
__device__ __forceinline__ void team_totals(const int64_t (&v)[kWT], bool first_lane_of_active_team, int64_t (&F)[kWT]) {
#pragma unroll
    for (int t = 0; t < kWT; t++) F[t] = first_lane_of_active_team ? v[t] : 0;
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        int64_t other[kWT];
#pragma unroll
        for (int t = 0; t < kWT; t++) other[t] = __shfl_xor_sync(0xffffffffu, F[t], o);
#pragma unroll
        for (int t = 0; t < kWT; t++) F[t] += other[t];
    }
}
__device__ __forceinline__ void warp_max_x(int64_t (&v)[kWT]) {
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        int64_t other[kWT];
#pragma unroll
        for (int t = 0; t < kWT; t++) other[t] = __shfl_xor_sync(0xffffffffu, v[t], o);
#pragma unroll
        for (int t = 0; t < kWT; t++) v[t] = max_v(v[t], other[t]);
    }
}

template <typename V>
__device__ __forceinline__ void decompose_warp(const DevCat& dc, const KParams& kp, const WCtx& c, int64_t unit, int64_t left,
                                               int& k, int& st, Counters& cnt) {
    const int N = c.N, G = c.G, lane = c.lane;
    const int ld = N + 1;                                // row stride of D_rem
    const int ns_pad = (dc.n_shapes + 31) & ~31;         // row stride of the transposed term table
    const int team = lane >> 3, tl = lane & 7;
    const bool active = team < G;
    const int a = active ? team : G - 1;                 // the team's group (spare teams repeat the last group on their own tiles)
    const int q = tl & 3, i0 = tl >> 2, i1 = i0 + 2;     // the lane's credit elements: (i0, q) and (i1, q)
    const bool ns4 = kp.n_start == 4;
    V* const Drem = ws<V>(c.o_drem);
    const V* const cap = ws<V>(c.o_cap);
    int64_t* const Dhat = ws<int64_t>(c.o_dhat);
    uint8_t pidx[3][4];
#pragma unroll
    for (int pp = 0; pp < 3; pp++) {
        const unsigned pk = perm4_packed_rt(tl * 3 + pp);
#pragma unroll
        for (int qq = 0; qq < 4; qq++) pidx[pp][qq] = (uint8_t)(((pk >> (2 * qq)) & 3) * 4 + qq);
    }
    unsigned tile[kWT];                                  // this team's credit tile of each task in flight
#pragma unroll
    for (int t = 0; t < kWT; t++) tile[t] = c.o_cred + (unsigned)((t * 4 + team) * 17 * sizeof(V));

    for (;;) {
        if (left == 0) break;
        if (k == kp.k_max) { st |= VP_ST_STEP_LIMIT; break; }
        // (A) Eq. (6): shape scores, four shapes per lane in flight, first maximum
        int64_t best = -1;
        int best_s = 0x7fffffff;
        for (int s0 = lane; s0 < dc.n_shapes; s0 += 128) {
            int64_t score[4] = {0, 0, 0, 0};
            const uint32_t* tp = ws<uint32_t>(c.o_term) + s0;     // term e of shape s is at [e][s]: lanes read neighbours
            const int last = dc.n_shapes - 1 - s0;               // shapes beyond the catalog re-read the last one
            int du[4];
#pragma unroll
            for (int u = 0; u < 4; u++) du[u] = min(32 * u, last);
#pragma unroll 4
            for (int e = 0; e < dc.max_terms; e++) {
#pragma unroll
                for (int u = 0; u < 4; u++) {
                    const uint32_t w = tp[e * ns_pad + du[u]];
                    score[u] += *(const int64_t*)((const char*)Dhat + (w & 0xffffu)) * (int64_t)(w >> 16);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; u++)
                if (s0 + 32 * u < dc.n_shapes && score[u] > best) { best = score[u]; best_s = s0 + 32 * u; }
        }
        warp_argmax_first(best, best_s);
        if (best <= 0) { st |= VP_ST_UNCOVERED; break; }
        const int f0 = (int)ws<uint32_t>(c.o_bucket)[best_s], H = (int)ws<uint32_t>(c.o_bucket)[best_s + 1] - f0;
        const int n_tasks = H * kp.n_start;

        // (B) MultiStartAA, four (family, start) tasks at a time; (C) best start per family, best family
        int64_t bf = -1, bd = 1, ff = -1, fd = 1;        // best family so far; best start of the current family
        int bt = -1, ft = -1, cur_h = -1;
        for (int task0 = 0; task0 < n_tasks; task0 += kWT) {
            unsigned alive = 0;
            V cap_out[kWT], cap_in[kWT];
            int cls_in[kWT];
            unsigned o_src[kWT], o_dst[kWT], o_rin_s[kWT], o_rin_d[kWT];
            // initial destination binding: start t rotates the in-slots of every group by t
            for (int e = lane; e < kWT * 16; e += 32) {
                const int t = e >> 4, d = (e >> 2) & 3, qq = e & 3, task = task0 + t;
                if (task < n_tasks && d < G) {
                    const int h = ns4 ? task >> 2 : task / kp.n_start, tt = task - h * kp.n_start;
                    ws<uint8_t>(c.o_bind_dst)[task * N + (ws<uint16_t>(c.o_fam_in)[(f0 + h) * N + d * 4 + qq] & 0xff)] =
                        (uint8_t)(d * 4 + ((qq + tt) & 3));
                }
            }
#pragma unroll
            for (int t = 0; t < kWT; t++) {
                const int task = task0 + t < n_tasks ? task0 + t : n_tasks - 1;
                if (task0 + t < n_tasks) alive |= 1u << t;
                const int f = f0 + (ns4 ? task >> 2 : task / kp.n_start);
                const unsigned w = ws<uint16_t>(c.o_fam_in)[f * N + a * 4 + q];
                cap_out[t] = cap[ws<uint8_t>(c.o_fam_cls)[f * N + a * 4 + q]];
                cls_in[t] = (int)(w >> 8);
                cap_in[t] = cap[cls_in[t]];
                o_src[t] = c.o_bind_src + (unsigned)(task * N);
                o_dst[t] = c.o_bind_dst + (unsigned)(task * N);
                o_rin_s[t] = o_src[t] + (w & 0xff);          // binding entries of the in-slot this lane serves
                o_rin_d[t] = o_dst[t] + (w & 0xff);
            }
            const unsigned valid = alive;
            __syncwarp();
            int64_t F_old[kWT], F_new[kWT];
            unsigned bpk_fin[kWT];
#pragma unroll
            for (int t = 0; t < kWT; t++) { F_old[t] = -1; F_new[t] = -1; bpk_fin[t] = 0; }
            for (int sweep = 0; sweep < kp.i_aa && alive; sweep++) {
                V v0[kWT], v1[kWT], val[kWT];
                unsigned bpk[kWT];
                // source half: credits of source group a towards the current destinations of its out-slots
#pragma unroll
                for (int t = 0; t < kWT; t++) {
                    const int dq = ws<uint8_t>(o_dst[t])[a * 4 + q];
                    v0[t] = min_v(Drem[(a * 4 + i0) * ld + dq], cap_out[t]);
                    v1[t] = min_v(Drem[(a * 4 + i1) * ld + dq], cap_out[t]);
                }
#pragma unroll
                for (int t = 0; t < kWT; t++)
                    if (alive >> t & 1) { ws<V>(tile[t])[i0 * 4 + q] = v0[t]; ws<V>(tile[t])[i1 * 4 + q] = v1[t]; }
                __syncwarp();
                team_best_x(tile, tl, pidx, c.o_lut, bpk, val);
#pragma unroll
                for (int t = 0; t < kWT; t++)
                    if (alive >> t & 1) ws<uint8_t>(o_src[t])[a * 4 + q] = (uint8_t)(a * 4 + perm_pos<V>(bpk[t], q));
                __syncwarp();
                // destination half: credits into destination group a from the current sources of its in-slots
#pragma unroll
                for (int t = 0; t < kWT; t++) {
                    const int sq = *ws<uint8_t>(o_rin_s[t]);
                    v0[t] = min_v(Drem[sq * ld + a * 4 + i0], cap_in[t]);
                    v1[t] = min_v(Drem[sq * ld + a * 4 + i1], cap_in[t]);
                }
#pragma unroll
                for (int t = 0; t < kWT; t++)
                    if (alive >> t & 1) { ws<V>(tile[t])[i0 * 4 + q] = v0[t]; ws<V>(tile[t])[i1 * 4 + q] = v1[t]; }
                __syncwarp();
                team_best_x(tile, tl, pidx, c.o_lut, bpk, val);
#pragma unroll
                for (int t = 0; t < kWT; t++)
                    if (alive >> t & 1) *ws<uint8_t>(o_rin_d[t]) = (uint8_t)(a * 4 + perm_pos<V>(bpk[t], q));
                int64_t Fn[kWT];
                team_totals(val, active && tl == 0, Fn);                                  // Eq. (8)
#pragma unroll
                for (int t = 0; t < kWT; t++) {
                    if (alive >> t & 1) {
                        F_new[t] = Fn[t];
                        bpk_fin[t] = bpk[t];
                        cnt.sweeps++;
                        if (Fn[t] <= F_old[t]) alive &= ~(1u << t);       // frozen: bindings and credits stay
                        else F_old[t] = Fn[t];
                    }
                }
                __syncwarp();
            }
            // Evaluate: Eq. (9) volumes are the chosen credits of the task's last destination half; Eq. (10)
            int64_t den[kWT];
            {
                V x[kWT];
#pragma unroll
                for (int t = 0; t < kWT; t++) {
                    x[t] = 0;
                    if (valid >> t & 1) x[t] = ws<V>(tile[t])[perm_pos<V>(bpk_fin[t], q) * 4 + q];
                }
                if (sizeof(V) == 4 && dc.n_classes == 1) {      // one path rate: the slowest lane carries the largest volume
                    const int64_t ts = ws<int64_t>(c.o_tscale)[0];
#pragma unroll
                    for (int t = 0; t < kWT; t++) den[t] = (int64_t)__reduce_max_sync(0xffffffffu, (uint32_t)x[t]) * ts;
                } else {
#pragma unroll
                    for (int t = 0; t < kWT; t++) den[t] = (int64_t)x[t] * ws<int64_t>(c.o_tscale)[cls_in[t]];
                    warp_max_x(den);
                }
#pragma unroll
                for (int t = 0; t < kWT; t++) den[t] = F_new[t] > 0 ? kp.lambda_ns * dc.W + den[t] : 1;
            }
#pragma unroll
            for (int t = 0; t < kWT; t++) {
                if (!(valid >> t & 1)) continue;
                const int task = task0 + t, h = ns4 ? task >> 2 : task / kp.n_start;
                cnt.tasks++;
                if (h != cur_h) {                          // a new family starts: settle the previous one
                    if (cur_h >= 0 && (bt < 0 || util_greater(ff, fd, bf, bd))) { bf = ff; bd = fd; bt = ft; }
                    cur_h = h; ff = -1; fd = 1; ft = -1;
                }
                if (F_new[t] > ff) { ff = F_new[t]; fd = den[t]; ft = task; }    // largest F, lowest start
            }
        }
        if (cur_h >= 0 && (bt < 0 || util_greater(ff, fd, bf, bd))) { bf = ff; bd = fd; bt = ft; }   // lowest family on ties
        if (bf <= 0) { st |= VP_ST_NO_PROGRESS; break; }

        // (D) emit activation k, D_rem -= X(E), write offset row k+1, re-sum D-hat
        {
            const int h = ns4 ? bt >> 2 : bt / kp.n_start;
            const size_t row = (size_t)k * N, orow = (size_t)(k + 1) * N;
            if (lane < N) {
                const int r = lane;
                const uint32_t w = ws<uint32_t>(c.o_fam_slot)[(f0 + h) * N + r];
                const int i = ws<uint8_t>(c.o_bind_src)[bt * N + r], j = ws<uint8_t>(c.o_bind_dst)[bt * N + r];
                const V x = min_v(cap[(w >> 24) & 0xf], Drem[i * ld + j]);
                // straight-line: an idle lane (x = 0) writes the idle values and adds zero
                const bool busy = x > 0;
                const int64_t bytes = (int64_t)x * unit;
                const int64_t sa = ws<int64_t>(c.o_send_acc)[i] + bytes, ra = ws<int64_t>(c.o_recv_acc)[j] + bytes;
                c.lane_dst_b[row + i] = busy ? (int16_t)j : (int16_t)-1;
                c.lane_inst_b[row + i] = busy ? (uint16_t)(w & 0xffffu) : (uint16_t)0xFFFF;
                c.lane_bytes_b[row + i] = bytes;
                Drem[i * ld + j] -= x;
                ws<int64_t>(c.o_send_acc)[i] = sa;
                ws<int64_t>(c.o_recv_acc)[j] = ra;
                c.send_off_b[orow + i] = sa;
                if (c.recv_off_b) c.recv_off_b[orow + j] = ra;
            }
            if (lane == 0) c.chan_id_b[k] = f0 + h;
            left -= bf;
            __syncwarp();
            {   // Eq. (5): two lanes per cell, eight entries each
                const int cell = lane >> 1, half = lane & 1;
                int64_t s = 0;
                if (cell < G * G) {
                    const int ga = cell / G, gd = cell - ga * G;
#pragma unroll
                    for (int ii = 0; ii < 2; ii++)
#pragma unroll
                        for (int jj = 0; jj < 4; jj++) s += (int64_t)Drem[(ga * 4 + half * 2 + ii) * ld + gd * 4 + jj];
                }
                s += __shfl_xor_sync(0xffffffffu, s, 1);
                if (cell < G * G && half == 0) Dhat[cell] = s;
            }
        }
        k++;
        __syncwarp();
    }
}

#ifndef VP_WARP_MIN_BLOCKS
#define VP_WARP_MIN_BLOCKS 3
#endif
__global__ void __launch_bounds__(128, VP_WARP_MIN_BLOCKS)
vp_schedule_warp_kernel(DevCat dc, KParams kp, const int64_t* __restrict__ demand, const int64_t* __restrict__ tau_in, int B,
                        int32_t* __restrict__ n_steps, int32_t* __restrict__ chan_id, int16_t* __restrict__ lane_dst,
                        uint16_t* __restrict__ lane_inst, int64_t* __restrict__ lane_bytes, int64_t* __restrict__ send_off,
                        int64_t* __restrict__ recv_off, int64_t* __restrict__ tau_out, int32_t* __restrict__ status,
                        unsigned int* counter) {
    unsigned char* const smem_raw = vp_wsmem;
    const int N = dc.N, G = dc.G, tid = threadIdx.x, NT = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, n_warps = NT >> 5;
    const int ld = N + 1;
    const WarpSmem L = warp_smem_layout(dc, kp, n_warps);
    if (tid < 32) smem_raw[L.lut + tid] = (uint8_t)(31 - tid < 24 ? perm4_packed_rt(31 - tid) : 0);
    // ---- stage the catalog (shared by the warps of the CTA): bulk asynchronous copies (TMA) of whole arrays onto one
    // mbarrier; plain loads if the bounded wait gives up
    {
        const int ns_pad = (dc.n_shapes + 31) & ~31;
        const unsigned b_term = (unsigned)(ns_pad * dc.max_terms * 4), b_slot = (unsigned)align16(dc.n_families * N * 4),
                       b_fin = (unsigned)align16(dc.n_families * N * 2), b_fcls = (unsigned)align16(dc.n_families * N),
                       b_bucket = (unsigned)align16((dc.n_shapes + 1) * 4);
        const unsigned total = b_term + b_slot + b_fin + b_fcls + b_bucket;
        __shared__ __align__(8) unsigned long long s_stage_bar;
        bool landed = false;
        if (total < (1u << 20)) {
            const unsigned bar = smem_u32(&s_stage_bar);
            if (tid == 0) {
                mbar_init(bar, 1);
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                mbar_expect_tx(bar, total);
                bulk_load(smem_u32(smem_raw + L.term), dc.term_t, b_term, bar);
                bulk_load(smem_u32(smem_raw + L.fam_slot), dc.fam_slot, b_slot, bar);
                bulk_load(smem_u32(smem_raw + L.fam_in), dc.fam_in, b_fin, bar);
                bulk_load(smem_u32(smem_raw + L.fam_cls), dc.fam_cls, b_fcls, bar);
                bulk_load(smem_u32(smem_raw + L.bucket), dc.bucket_ptr, b_bucket, bar);
            }
            __syncthreads();
            landed = __syncthreads_and(mbar_wait_bounded(bar, 0, 1u << 20)) != 0;
        }
        if (!landed) {
            uint32_t* t_term = (uint32_t*)(smem_raw + L.term);
            for (int e = tid; e < ns_pad * dc.max_terms; e += NT) t_term[e] = dc.term_t[e];
            uint32_t* t_slot = (uint32_t*)(smem_raw + L.fam_slot);
            uint16_t* t_in = (uint16_t*)(smem_raw + L.fam_in);
            uint8_t* t_cls = smem_raw + L.fam_cls;
            for (int e = tid; e < dc.n_families * N; e += NT) {
                t_slot[e] = dc.fam_slot[e]; t_in[e] = dc.fam_in[e]; t_cls[e] = dc.fam_cls[e];
            }
            uint32_t* t_bp = (uint32_t*)(smem_raw + L.bucket);
            for (int e = tid; e <= dc.n_shapes; e += NT) t_bp[e] = dc.bucket_ptr[e];
        }
    }
    __syncthreads();
    WCtx c;
    c.N = N; c.G = G; c.lane = lane;
    const unsigned base = (unsigned)warp * (unsigned)L.per_warp;
    c.o_drem = base + L.drem; c.o_dhat = base + L.dhat; c.o_send_acc = base + L.send_acc; c.o_recv_acc = base + L.recv_acc;
    c.o_cred = base + L.cred; c.o_tscale = base + L.tscale; c.o_bind_src = base + L.bind_src; c.o_bind_dst = base + L.bind_dst;
    c.o_cap = base + L.cap64;
    c.o_term = L.term; c.o_fam_slot = L.fam_slot; c.o_fam_in = L.fam_in; c.o_fam_cls = L.fam_cls; c.o_bucket = L.bucket;
    c.o_lut = L.lut;
    int64_t* const Drem = ws<int64_t>(c.o_drem);
    int64_t* const Dhat = ws<int64_t>(c.o_dhat);
    int64_t* const send_acc = ws<int64_t>(c.o_send_acc);
    int64_t* const recv_acc = ws<int64_t>(c.o_recv_acc);
    int64_t* const cap64 = ws<int64_t>(base + L.cap64);
    int64_t* const tscale = ws<int64_t>(c.o_tscale);
    uint32_t* const cap32 = ws<uint32_t>(base + L.cap32);
    unsigned long long n_act = 0;
    Counters cnt;
    cnt.tasks = 0; cnt.sweeps = 0; cnt.t_mark = 0;

    for (;;) {
        int b = 0;
        if (lane == 0) b = (int)atomicAdd(counter, 1u);
        b = __shfl_sync(0xffffffffu, b, 0);
        if (b >= B) break;
        const int64_t* D = demand + (size_t)b * N * N;
        const size_t lane_base = (size_t)b * kp.k_max * N, off_base = (size_t)b * (kp.k_max + 1) * N;
        c.chan_id_b = chan_id + (size_t)b * kp.k_max;
        c.lane_dst_b = lane_dst + lane_base;
        c.lane_inst_b = lane_inst + lane_base;
        c.lane_bytes_b = lane_bytes + lane_base;
        c.send_off_b = send_off + off_base;
        c.recv_off_b = recv_off ? recv_off + off_base : nullptr;

        // ---- validate, copy D into D_rem
        int flags = 0;
        for (int e = lane; e < N * N; e += 32) {
            const int64_t v = D[e];
            if (v < 0) flags |= VP_ST_NEGATIVE;
            else if (v >= VP_ENTRY_LIMIT) flags |= VP_ST_OVERFLOW_RISK;
            else {
                if (e / N == e % N && v != 0) flags |= VP_ST_DIAG_NONZERO;
                if (v % kp.granule) flags |= VP_ST_NOT_GRANULE;
            }
            Drem[(e / N) * ld + e % N] = v;
        }
        const int64_t tau_given = tau_in ? tau_in[b] : 0;
        if (tau_given < 0 || tau_given > VP_ENTRY_LIMIT) flags |= VP_ST_BAD_TAU;
        flags = (int)__reduce_or_sync(0xffffffffu, (unsigned)flags);
        for (int i = lane; i < N; i += 32) {
            send_acc[i] = 0; recv_acc[i] = 0;
            c.send_off_b[i] = 0;
            if (c.recv_off_b) c.recv_off_b[i] = 0;
        }
        __syncwarp();
        int st = flags, k = 0;
        int64_t tau = 0;
        if (st == 0) {
            // ---- row / column sums, group sums (Eq. 5), quantum (Section 5)
            int64_t est = 0, tot = 0;
            for (int i = lane; i < N; i += 32) {
                int64_t row = 0, col = 0;
                for (int jj = 0; jj < N; jj++) {
                    int j = jj + i; if (j >= N) j -= N;
                    row += Drem[i * ld + j];
                    col += Drem[j * ld + i];
                }
                tot += row;
                est = max_v(est, max_v(ceil_div_i64(row, dc.bw_max), ceil_div_i64(col, dc.bw_max)));
            }
            for (int cell = lane; cell < G * G; cell += 32) {
                const int ga = cell / G, gd = cell % G;
                int64_t s = 0;
#pragma unroll
                for (int i = 0; i < 4; i++)
#pragma unroll
                    for (int j = 0; j < 4; j++) s += Drem[(ga * 4 + i) * ld + gd * 4 + j];
                Dhat[cell] = s;
            }
            __syncwarp();
            for (int l = lane; l < dc.n_res; l += 32) {
                const uint32_t bwl = dc.forced_bw[l];
                if (!bwl) continue;
                int64_t f = 0;
                for (uint32_t e = dc.forced_ptr[l]; e < dc.forced_ptr[l + 1]; e++) f += Dhat[dc.forced_cell[e]];
                est = max_v(est, ceil_div_i64(f, (int64_t)bwl));
            }
            est = warp_max_i64(est);
            tot = warp_sum_i64(tot);
            const int64_t tq = tau_given > 0 ? tau_given : max_v((int64_t)1, ceil_div_i64(est, (int64_t)kp.k_target));
            int64_t cap_max = 0;
            for (int cl = 0; cl < dc.n_classes; cl++) {
                int64_t cp = (tq * dc.class_bw[cl]) / kp.granule * kp.granule;
                cp = cp < kp.granule ? kp.granule : cp;
                cap_max = max_v(cap_max, cp);
                if (lane == 0) cap64[cl] = cp;
            }
            // granule units: capacities below 2^22 granules (four credits and a permutation byte share 32 bits)
            const bool units = cap_max / kp.granule < ((int64_t)1 << 22) && kp.granule >= 256;
            __syncwarp();
            if (lane < dc.n_classes) {
                cap32[lane] = (uint32_t)(units ? cap64[lane] / kp.granule : 0);
                tscale[lane] = dc.class_wdiv[lane] * (units ? kp.granule : 1);
            }
            tau = tq;
            __syncwarp();
            if (units) {
                // the byte copy is no longer needed: overwrite it with the demand in granules
                uint32_t* Drem32 = (uint32_t*)Drem;
                for (int e = lane; e < N * N; e += 32) Drem32[(e / N) * ld + e % N] = (uint32_t)(D[e] / kp.granule);
                for (int cell = lane; cell < G * G; cell += 32) Dhat[cell] /= kp.granule;
                __syncwarp();
                c.o_cap = base + L.cap32;
                decompose_warp<uint32_t>(dc, kp, c, kp.granule, tot / kp.granule, k, st, cnt);
            } else {
                c.o_cap = base + L.cap64;
                decompose_warp<int64_t>(dc, kp, c, 1, tot, k, st, cnt);
            }
        }
        __syncwarp();
        // ---- idle rows beyond n_steps; offset rows repeat the totals
        for (size_t e = (size_t)k * N + lane; e < (size_t)kp.k_max * N; e += 32) {
            c.lane_dst_b[e] = -1;
            c.lane_inst_b[e] = 0xFFFF;
            c.lane_bytes_b[e] = 0;
            const int i = (int)(e % N);
            c.send_off_b[N + e] = send_acc[i];
            if (c.recv_off_b) c.recv_off_b[N + e] = recv_acc[i];
        }
        for (int kk = k + lane; kk < kp.k_max; kk += 32) c.chan_id_b[kk] = -1;
        if (lane == 0) {
            n_act += (unsigned long long)k;
            n_steps[b] = k;
            status[b] = st;
            if (tau_out) tau_out[b] = tau;
        }
        __syncwarp();
    }
    unsigned long long* stats = (unsigned long long*)(counter + 4);
    if (lane == 0) {
        if (n_act) atomicAdd(&stats[0], n_act);
        if (cnt.tasks) { atomicAdd(&stats[1], cnt.tasks); atomicAdd(&stats[2], cnt.sweeps); }
    }
}

}  // namespace
