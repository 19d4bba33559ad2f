// Algorithm 2 with ONE WARP per demand matrix, for catalogs of at most four groups of four ranks (N <= 16).
//
// A matrix this small has too little work per phase for a whole CTA: with several warps per matrix most of an
// iteration is spent in block barriers and in hand-overs through shared memory.  Here a warp owns a matrix from
// the first to the last activation and nothing but __syncwarp orders its phases:
//  (A) each lane scores every 32nd shape (Eq. 6); a butterfly of shuffles leaves the first maximum in all lanes;
//  (B) the (family, start) tasks of the bucket run eight at a time: a team of four lanes per task, one lane per rank
//      group, and every lane solves its group's exact 4 x 4 assignments (Eq. 7) by itself; the two halves of a sweep
//      exchange nothing but the bindings; a task that stops improving (Eq. 8) is frozen while the others finish;
//      Evaluate (Eq. 9, 10) runs when several families compete; best start / best family follow in registers;
//  (D) sixteen lanes emit the activation and subtract it; D-hat is then re-summed from D_rem by all lanes
//      (two lanes per cell), which needs no atomics.
// A CTA is one to four such warps that share only the staged catalog.  Included by schedule.cu.
#pragma once

namespace {


struct WarpSmem {                           // byte offsets; the per-warp block comes first, once per warp
    int drem, dremT, dhat, send_acc, recv_acc, cred, cap64, tscale, cap32, bind_src, bind_dst, per_warp;
    int term, fam_in, fam_cls, fam_slot, bucket, lut, total;
};

__host__ __device__ inline WarpSmem warp_smem_layout(const DevCat& dc, const KParams& kp, int n_warps) {
    WarpSmem L;
    int o = 0;
    L.drem = o;      o += align16(dc.N * (dc.N + 1) * 8);      // rows padded by one element: no bank conflicts down a column
    L.dremT = o;     o += align16(dc.N * dc.N * 4);            // 32-bit granules: the transpose (a column's four credits of a group in 16 bytes)
    L.dhat = o;      o += align16(dc.G * dc.G * 8);
    L.send_acc = o;  o += dc.N * 8;
    L.recv_acc = o;  o += dc.N * 8;
    L.cred = o;
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
    unsigned o_drem, o_dremT, o_dhat, o_send_acc, o_recv_acc, o_cred, o_cap, o_tscale, o_bind_src, o_bind_dst;
    unsigned o_term, o_fam_slot, o_fam_in, o_fam_cls, o_bucket, o_lut;
    int32_t* chan_id_b;
    int16_t* lane_dst_b;
    uint16_t* lane_inst_b;
    int64_t *lane_bytes_b, *send_off_b, *recv_off_b;
};

template <typename T> __device__ __forceinline__ T* ws(unsigned off) { return (T*)(vp_wsmem + off); }

// Sum over the four lanes of a team (lane & ~3 .. lane | 3); every lane gets it.
__device__ __forceinline__ uint32_t team_sum(uint32_t v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v + __shfl_xor_sync(0xffffffffu, v, 2);
}
__device__ __forceinline__ int64_t team_sum(int64_t v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v + __shfl_xor_sync(0xffffffffu, v, 2);
}
__device__ __forceinline__ int64_t team_max(int64_t v) {
    v = max_v(v, __shfl_xor_sync(0xffffffffu, v, 1));
    return max_v(v, __shfl_xor_sync(0xffffffffu, v, 2));
}

// Eq. (6) for the R shapes of a lane (shape lane + 32 u) from their lane counts, four bits per D-hat cell (cells 0..7 in
// the first word, 8..15 in the second), against the cells themselves; S is the score type (32 bits while scores stay
// below 2^31).  Cells are taken four at a time (a table has 1, 4, 9 or 16 of them; a cell beyond the table has count 0
// in every shape, so what is read there does not matter).  Leaves the lane's first maximum in (best, best_s).
template <int R, typename S>
__device__ __forceinline__ void score_dense(const int64_t* Dhat, int tbl_size, const uint32_t (&smask)[4][2], int lane, int n_shapes,
                                            int64_t& best, int& best_s) {
    S sc[R];
#pragma unroll
    for (int u = 0; u < R; u++) sc[u] = 0;
#pragma unroll
    for (int quad = 0; quad < 4; quad++) {
        if (quad * 4 < tbl_size) {
#pragma unroll
            for (int m = 0; m < 4; m++) {
                const int cell = quad * 4 + m;
                const S d = (S)Dhat[cell];
#pragma unroll
                for (int u = 0; u < R; u++) sc[u] += d * (S)((smask[u][cell >> 3] >> (4 * (cell & 7))) & 15u);
            }
        }
    }
#pragma unroll
    for (int u = 0; u < R; u++)
        if (lane + 32 * u < n_shapes && (int64_t)sc[u] > best) { best = (int64_t)sc[u]; best_s = lane + 32 * u; }
}

template <typename V>
__device__ __forceinline__ void decompose_warp(const DevCat& dc, const KParams& kp, const WCtx& c, int64_t unit, int64_t left,
                                               int& k, int& st, Counters& cnt) {
    const int N = c.N, G = c.G, lane = c.lane;
    // row stride of D_rem: N for 32-bit granules (a row's four credits of a group are one 16-byte load), N + 1 for bytes
    const int ld = sizeof(V) == 4 ? N : N + 1;
    const int ns_pad = (dc.n_shapes + 31) & ~31;         // row stride of the transposed term table
    // Step 2 runs eight (family, start) tasks at a time: a team of four lanes per task, one lane per rank group, which
    // solves its group's exact 4 x 4 assignments on its own (best_assignment) -- no credit tiles, no hand-overs
    // between lanes except the bindings themselves.
    const int team = lane >> 2, a = lane & 3;
    const bool active = a < G;
    const int ns_shift = (kp.n_start & (kp.n_start - 1)) == 0 ? 31 - __clz(kp.n_start) : -1;
    V* const Drem = ws<V>(c.o_drem);
    uint32_t* const DremT = ws<uint32_t>(c.o_dremT);      // (32-bit granules only) DremT[j * N + i] = Drem[i * N + j]
    const V* const cap = ws<V>(c.o_cap);
    int64_t* const Dhat = ws<int64_t>(c.o_dhat);
    // Plain score tables of at most 16 D-hat cells and at most 128 shapes: a lane keeps the lane counts of its (up to
    // four) shapes in registers, four bits per cell, and scoring needs no term loads.
    const bool dense = dc.tbl_size <= 16 && dc.n_shapes <= 128;
    const int n_rounds = (dc.n_shapes + 31) >> 5;         // shapes per lane (dense: at most four)
    uint32_t smask[4][2] = {{0u, 0u}, {0u, 0u}, {0u, 0u}, {0u, 0u}};     // cells 0..7, cells 8..15
    if (dense)
        for (int u = 0; u < 4; u++) {
            const int s = lane + 32 * u;
            if (s < dc.n_shapes)
                for (int e = 0; e < dc.max_terms; e++) {
                    const uint32_t w = ws<uint32_t>(c.o_term)[e * ns_pad + s];
                    const uint32_t cell = (w & 0xffffu) >> 3;
                    smask[u][cell >> 3] |= (w >> 16) << (4 * (cell & 7));
                }
        }

    for (;;) {
        if (left == 0) break;
        if (k == kp.k_max) { st |= VP_ST_STEP_LIMIT; break; }
        // (A) Eq. (6): shape scores, first maximum
        int64_t best = -1;
        int best_s = 0x7fffffff;
        const bool narrow_now = left < ((int64_t)1 << 31);       // every D-hat cell fits 32 bits
        if (dense) {
            const bool narrow = left * 4 < ((int64_t)1 << 31);   // a score is at most g x (what is left)
            switch (n_rounds * 2 + (narrow ? 1 : 0)) {
                case 3: score_dense<1, uint32_t>(Dhat, dc.tbl_size, smask, lane, dc.n_shapes, best, best_s); break;
                case 5: score_dense<2, uint32_t>(Dhat, dc.tbl_size, smask, lane, dc.n_shapes, best, best_s); break;
                case 7: score_dense<3, uint32_t>(Dhat, dc.tbl_size, smask, lane, dc.n_shapes, best, best_s); break;
                case 9: score_dense<4, uint32_t>(Dhat, dc.tbl_size, smask, lane, dc.n_shapes, best, best_s); break;
                case 2: score_dense<1, int64_t>(Dhat, dc.tbl_size, smask, lane, dc.n_shapes, best, best_s); break;
                case 4: score_dense<2, int64_t>(Dhat, dc.tbl_size, smask, lane, dc.n_shapes, best, best_s); break;
                case 6: score_dense<3, int64_t>(Dhat, dc.tbl_size, smask, lane, dc.n_shapes, best, best_s); break;
                default: score_dense<4, int64_t>(Dhat, dc.tbl_size, smask, lane, dc.n_shapes, best, best_s); break;
            }
        } else {
            for (int s0 = lane; s0 < dc.n_shapes; s0 += 128) {     // four shapes per lane in flight
                int64_t score[4] = {0, 0, 0, 0};
                const uint32_t* tp = ws<uint32_t>(c.o_term) + s0;  // term e of shape s is at [e][s]: lanes read neighbours
                const int last = dc.n_shapes - 1 - s0;             // shapes beyond the catalog re-read the last one
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
        }
        VP_TICK(0);
        warp_argmax_first(best, best_s);
        if (best <= 0) { st |= VP_ST_UNCOVERED; break; }
        const int f0 = (int)ws<uint32_t>(c.o_bucket)[best_s], H = (int)ws<uint32_t>(c.o_bucket)[best_s + 1] - f0;
        const int n_tasks = H * kp.n_start;
        VP_TICK(1);

        // (B) MultiStartAA, eight (family, start) tasks at a time; (C) best start per family, best family
        int64_t bf = -1, bd = 1, ff = -1, fd = 1;        // best family so far; best start of the current family
        int bt = -1, ft = -1, cur_h = -1;
        for (int task0 = 0; task0 < n_tasks; task0 += 8) {
            const int task = min(task0 + team, n_tasks - 1);
            const bool has = task0 + team < n_tasks && active;
            const int h = ns_shift >= 0 ? task >> ns_shift : task / kp.n_start, tt = task - h * kp.n_start, f = f0 + h;
            uint8_t* const srcb = ws<uint8_t>(c.o_bind_src) + task * N;
            uint8_t* const dstb = ws<uint8_t>(c.o_bind_dst) + task * N;
            V cap_out[4], cap_in[4];
            int rq[4], cls_in[4];
            const int ag = active ? a : 0;                   // (spare lanes read group 0's tables and write nothing)
            const uint2 fin4 = *(const uint2*)(ws<uint16_t>(c.o_fam_in) + f * N + ag * 4);        // four in-slots, 16 bits each
            const uint32_t fcls4 = *(const uint32_t*)(ws<uint8_t>(c.o_fam_cls) + f * N + ag * 4);  // four out-slot classes
#pragma unroll
            for (int q = 0; q < 4; q++) {
                const unsigned w = ((q < 2 ? fin4.x : fin4.y) >> (16 * (q & 1))) & 0xffffu;
                cap_out[q] = cap[(fcls4 >> (8 * q)) & 0xffu];
                rq[q] = (int)(w & 0xffu);
                cls_in[q] = (int)(w >> 8);
                cap_in[q] = cap[cls_in[q]];
                if (has) dstb[rq[q]] = (uint8_t)(a * 4 + ((q + tt) & 3));     // start t rotates the in-slots of every group
            }
            __syncwarp();
            VP_TICK(2);
            int64_t F_old = -1, F_new = -1;
            bool alive = has;
            for (int sweep = 0; sweep < kp.i_aa && __any_sync(0xffffffffu, alive); sweep++) {
                if (alive) {                                  // source half: credits of group a towards its out-slots' destinations
                    const uint32_t d4 = *(const uint32_t*)(dstb + a * 4);
                    V cm[4][4];
#pragma unroll
                    for (int q = 0; q < 4; q++) {
                        const int dq = (int)((d4 >> (8 * q)) & 0xffu);
                        if constexpr (sizeof(V) == 4) {
                            const uint4 c4 = *(const uint4*)(DremT + dq * N + a * 4);
                            cm[0][q] = min_v((V)c4.x, cap_out[q]); cm[1][q] = min_v((V)c4.y, cap_out[q]);
                            cm[2][q] = min_v((V)c4.z, cap_out[q]); cm[3][q] = min_v((V)c4.w, cap_out[q]);
                        } else {
                            const V* col = Drem + (a * 4) * ld + dq;
#pragma unroll
                            for (int i = 0; i < 4; i++) cm[i][q] = min_v(col[i * ld], cap_out[q]);
                        }
                    }
                    uint32_t rows4;                          // the row bound to position q, in byte q
                    if constexpr (sizeof(V) == 4) {
                        uint32_t v[4][4];
#pragma unroll
                        for (int i = 0; i < 4; i++)
#pragma unroll
                            for (int q = 0; q < 4; q++) v[i][q] = (uint32_t)cm[i][q] * 256u + big_tag(i, q);
                        const uint32_t pb = ~big_best_key(v) & 255u;      // position 0 in the two highest bits
                        rows4 = ((pb >> 6) & 3u) | ((pb << 4) & 0x300u) | ((pb << 14) & 0x30000u) | ((pb << 24) & 0x3000000u);
                    } else {
                        unsigned bpk;
                        best_assignment<4, V>(cm, bpk);
                        rows4 = (bpk & 3u) | ((bpk >> 2) & 3u) << 8 | ((bpk >> 4) & 3u) << 16 | ((bpk >> 6) & 3u) << 24;
                    }
                    *(uint32_t*)(srcb + a * 4) = (uint32_t)(a * 4) * 0x01010101u + rows4;
                }
                __syncwarp();
                V part = 0;
                if (alive) {                                  // destination half: credits into group a from its in-slots' sources
                    V cm[4][4];
#pragma unroll
                    for (int q = 0; q < 4; q++) {
                        const V* row = Drem + (int)srcb[rq[q]] * ld + a * 4;
                        if constexpr (sizeof(V) == 4) {
                            const uint4 r4 = *(const uint4*)row;
                            cm[0][q] = min_v((V)r4.x, cap_in[q]); cm[1][q] = min_v((V)r4.y, cap_in[q]);
                            cm[2][q] = min_v((V)r4.z, cap_in[q]); cm[3][q] = min_v((V)r4.w, cap_in[q]);
                        } else {
#pragma unroll
                            for (int i = 0; i < 4; i++) cm[i][q] = min_v(row[i], cap_in[q]);
                        }
                    }
                    if constexpr (sizeof(V) == 4) {
                        uint32_t v[4][4];
#pragma unroll
                        for (int i = 0; i < 4; i++)
#pragma unroll
                            for (int q = 0; q < 4; q++) v[i][q] = (uint32_t)cm[i][q] * 256u + big_tag(i, q);
                        const uint32_t key = big_best_key(v), pb = ~key & 255u;
                        part = (V)(key >> 8);
#pragma unroll
                        for (int q = 0; q < 4; q++) dstb[rq[q]] = (uint8_t)(a * 4 + ((pb >> (6 - 2 * q)) & 3u));
                    } else {
                        unsigned bpk;
                        part = best_assignment<4, V>(cm, bpk);
#pragma unroll
                        for (int q = 0; q < 4; q++) dstb[rq[q]] = (uint8_t)(a * 4 + ((bpk >> (2 * q)) & 3u));
                    }
                }
                const int64_t Fn = (int64_t)team_sum(part);   // Eq. (8)
                if (alive) {
                    F_new = Fn;
                    if (a == 0) cnt.sweeps++;
                    if (Fn <= F_old) alive = false;           // the run ends; its bindings stay as this sweep left them
                    else F_old = Fn;
                }
                __syncwarp();
            }
            VP_TICK(3);
            // Evaluate (Eq. 9, 10), needed only when several families compete: the volume of every in-slot of this
            // lane's group under the final bindings, the slowest lane over the team
            int64_t den = 1;
            if (H > 1) {
                int64_t tmax = 0;
                if (has) {
#pragma unroll
                    for (int q = 0; q < 4; q++) {
                        const V x = min_v(Drem[(int)srcb[rq[q]] * ld + (int)dstb[rq[q]]], cap_in[q]);
                        tmax = max_v(tmax, (int64_t)x * ws<int64_t>(c.o_tscale)[cls_in[q]]);
                    }
                }
                tmax = team_max(tmax);
                den = F_new > 0 ? kp.lambda_ns * dc.W + tmax : 1;
            }
            if (has && a == 0) cnt.tasks++;
            if (H == 1 && n_tasks <= 8) {
                // one family, one round: the best start is the largest F, the lowest start among equals -- one maximum of
                // F << 3 | (7 - start) over the warp (F is below 2^42)
                const uint64_t key = has && a == 0 ? (uint64_t)F_new << 3 | (uint64_t)(7 - team) : 0ull;
                const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key;
                const uint32_t mhi = __reduce_max_sync(0xffffffffu, hi);
                const uint32_t mlo = __reduce_max_sync(0xffffffffu, hi == mhi ? lo : 0u);
                const uint64_t mkey = (uint64_t)mhi << 32 | mlo;
                bf = (int64_t)(mkey >> 3); bd = 1; bt = 7 - (int)(mkey & 7u);
                cur_h = -1;                                       // (settled)
                break;
            }
            // the teams' results in task order (every lane follows along)
            const int in_round = min(8, n_tasks - task0);
            for (int t = 0; t < in_round; t++) {
                const int64_t Ft = __shfl_sync(0xffffffffu, F_new, t * 4), dt = __shfl_sync(0xffffffffu, den, t * 4);
                const int tk = task0 + t, ht = ns_shift >= 0 ? tk >> ns_shift : tk / kp.n_start;
                if (ht != cur_h) {                             // a new family starts: settle the previous one
                    if (cur_h >= 0 && (bt < 0 || util_greater(ff, fd, bf, bd))) { bf = ff; bd = fd; bt = ft; }
                    cur_h = ht; ff = -1; fd = 1; ft = -1;
                }
                if (Ft > ff) { ff = Ft; fd = dt; ft = tk; }    // largest F, lowest start
            }
        }
        if (cur_h >= 0 && (bt < 0 || util_greater(ff, fd, bf, bd))) { bf = ff; bd = fd; bt = ft; }   // lowest family on ties
        if (bf <= 0) { st |= VP_ST_NO_PROGRESS; break; }
        VP_TICK(4);

        // (D) emit activation k, D_rem -= X(E), write offset row k+1, re-sum D-hat
        {
            const int h = ns_shift >= 0 ? bt >> ns_shift : bt / kp.n_start;
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
                if constexpr (sizeof(V) == 4) DremT[j * N + i] -= (uint32_t)x;
                if (busy) {                                   // Eq. (5): the volume leaves its group pair's cell of D-hat
                    int64_t* cell = &Dhat[(i >> 2) * G + (j >> 2)];
                    if (narrow_now) atomicSub((unsigned int*)cell, (unsigned int)x);     // high word is zero, low word >= x
                    else atomicAdd((unsigned long long*)cell, (unsigned long long)(-(int64_t)x));
                }
                ws<int64_t>(c.o_send_acc)[i] = sa;
                ws<int64_t>(c.o_recv_acc)[j] = ra;
                c.send_off_b[orow + i] = sa;
                if (c.recv_off_b) c.recv_off_b[orow + j] = ra;
            }
            if (lane == 0) c.chan_id_b[k] = f0 + h;
            left -= bf;
            __syncwarp();
        }
        k++;
        __syncwarp();
        VP_TICK(5);
    }
}

#ifndef VP_WARP_MIN_BLOCKS
#define VP_WARP_MIN_BLOCKS 4
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
    c.o_drem = base + L.drem; c.o_dremT = base + L.dremT; c.o_dhat = base + L.dhat; c.o_send_acc = base + L.send_acc; c.o_recv_acc = base + L.recv_acc;
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
    for (int i = 0; i < 6; i++) cnt.cyc[i] = 0;

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
#ifdef VP_PHASE_TIMING
        cnt.t_mark = clock64();
#endif
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
                uint32_t* DremT32 = ws<uint32_t>(c.o_dremT);
                for (int e = lane; e < N * N; e += 32) {                                            // (row stride N, and the transpose)
                    const uint32_t v = (uint32_t)(D[e] / kp.granule);
                    const int i = e / N, j = e - i * N;
                    Drem32[e] = v;
                    DremT32[j * N + i] = v;
                }
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
    cnt.tasks = (unsigned long long)warp_sum_i64((int64_t)cnt.tasks);      // (counted by the first lane of every team)
    cnt.sweeps = (unsigned long long)warp_sum_i64((int64_t)cnt.sweeps);
    if (lane == 0) {
        if (n_act) atomicAdd(&stats[0], n_act);
        if (cnt.tasks) { atomicAdd(&stats[1], cnt.tasks); atomicAdd(&stats[2], cnt.sweeps); }
#ifdef VP_PHASE_TIMING
        for (int i = 0; i < 6; i++) atomicAdd(&stats[3 + i], (unsigned long long)cnt.cyc[i]);
#endif
    }
}

}  // namespace
