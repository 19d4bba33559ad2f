// Algorithm 2 (Section 4.2) for large node-symmetric catalogs: groups of four ranks, more than sixteen groups
// (N = 68 .. 256), shapes invariant under a shift of the node index.  Included by schedule.cu.
//
// One CTA decomposes one matrix at a time.  What differs from the general kernel is where the state lives:
//
//  * Credits.  Step 2 only ever looks at min(D_rem[i][j], cap_r) (Eq. 7).  When every lane capacity is below 2^16
//    granules, a 16-bit copy of the residual that saturates at 65,535 granules gives exactly the same credits, and
//    N x N of those fit shared memory (128 KB at N = 256) where the residual itself (256 KB in 32-bit granules) does
//    not.  The exact residual of a cell is kept in an L2-resident workspace slot and is touched only while the cell
//    is still saturated; once a cell has dropped below 65,535 granules the 16-bit copy *is* the residual.
//  * Scores.  Eq. (6) on a node-symmetric catalog is a sum of at most max_terms products count x C[e], where
//    C[delta][q][q'] = sum_n D-hat[(n,q)][(n+delta,q')] (the same integer as the full sum over D-hat).  The table C
//    (P S S entries, 32-bit granules) is kept in shared memory and every activation subtracts its lane volumes from
//    the entries they fall in, so D-hat itself is needed only once, for the quantum rule and the first table.
//    The terms of a shape are split by source rail into S rows, and the catalog has few distinct rows (127 per rail
//    for 4,095 shapes): an iteration first scores every row pattern (a few hundred sums of at most three products),
//    then every shape is the sum of S looked-up row scores -- two loads and an addition instead of six
//    multiply-adds.  The row scores are kept in eight copies so that the lanes of a warp rarely meet in a bank.
//
// A matrix that does not meet the conditions (granule below 256 bytes, a capacity of 2^16 granules or more, 2^32
// granules or more in total) is appended to a list that the general kernel works through afterwards.
#pragma once

namespace {

// Scoring reads the row scores at data-dependent positions; with one copy per lane class (lane mod 8) the lanes of a
// warp meet in a bank only when they share a class and read different patterns of equal parity.
constexpr int BIG_RS_COPIES = 8;

struct BigSmem {
    int cs, tbl, rs, pat, gnode, send_acc, recv_acc, red, pair, task_f, task_den, slotw, bind_src, bind_dst, term, bucket, total;
    int cs_stride;            // credits per row of the 16-bit matrix (N + 2: rows start in different banks)
    int pat_words;            // 32-bit words of row-pattern ids per shape (two ids per word)
};

__host__ __device__ inline BigSmem big_smem_layout(const DevCat& dc, const KParams& kp) {
    BigSmem L;
    int o = 0;
    L.cs_stride = dc.N + 2;
    const int cs_bytes = dc.N * L.cs_stride * 2, dhat_bytes = dc.G * dc.G * 8 + dc.N * 16;
    L.cs = o;        o += align16(cs_bytes > dhat_bytes ? cs_bytes : dhat_bytes);   // set-up: D-hat, row and column sums
    L.tbl = o;       o += align16(dc.tbl_size * 4);
    L.rs = o;        o += dc.n_patterns * 8 * BIG_RS_COPIES;      // row scores, one copy per lane class
    L.pat = o;       o += align16(dc.n_patterns * dc.max_row_terms * 4);
    L.gnode = o;     o += align16(dc.G * 2);
    L.send_acc = o;  o += dc.N * 8;
    L.recv_acc = o;  o += dc.N * 8;
    L.red = o;       o += 64 * 8;
    L.pair = o;      o += 16 * 6 * 8;
    L.task_f = o;    o += align16(kp.max_tasks * 8);
    L.task_den = o;  o += align16(kp.max_tasks * 8);
    L.slotw = o;     o += align16(dc.max_bucket * dc.N * 4);
    L.bind_src = o;  o += align16(kp.max_tasks * dc.N);
    L.bind_dst = o;  o += align16(kp.max_tasks * dc.N);
    L.pat_words = (dc.S + 1) / 2;
    L.term = o;      o += ((dc.n_shapes + 31) & ~31) * L.pat_words * 4;
    L.bucket = o;    o += align16((dc.n_shapes + 1) * 4);
    L.total = o;
    return L;
}

// Exact 4 x 4 assignment on credits that arrive shifted left by eight bits (a sum of four stays below 2^26):
// maximise key = 255 + sum_q (c[phi(q)][q] - (phi(q) << (6 - 2q))) over the permutations phi.  The subtracted part is
// the permutation written as a byte (position 0 in the two highest bits), so the largest key belongs to the largest
// credit sum and, among equal sums, to the first permutation in lexicographic order, exactly as an enumeration in
// that order that keeps the first maximum.  Because the key is a sum over positions it is maximised by dynamic
// programming over the set of rows already placed (positions 0, 1, 2, 3 in turn): 28 additions and 17 maxima
// instead of 24 sums of four.  The permutation byte is ~key & 255, the credit sum key >> 8.
__device__ __forceinline__ uint32_t big_best_key(const uint32_t (&c)[4][4]) {
#define VP_V(r, q) ((int32_t)c[r][q] - ((r) << (6 - 2 * (q))))
    const int32_t a0 = 255 + VP_V(0, 0), a1 = 255 + VP_V(1, 0), a2 = 255 + VP_V(2, 0), a3 = 255 + VP_V(3, 0);
    const int32_t b01 = max_v(a0 + VP_V(1, 1), a1 + VP_V(0, 1)), b02 = max_v(a0 + VP_V(2, 1), a2 + VP_V(0, 1));
    const int32_t b03 = max_v(a0 + VP_V(3, 1), a3 + VP_V(0, 1)), b12 = max_v(a1 + VP_V(2, 1), a2 + VP_V(1, 1));
    const int32_t b13 = max_v(a1 + VP_V(3, 1), a3 + VP_V(1, 1)), b23 = max_v(a2 + VP_V(3, 1), a3 + VP_V(2, 1));
    const int32_t c012 = max_v(max_v(b01 + VP_V(2, 2), b02 + VP_V(1, 2)), b12 + VP_V(0, 2));
    const int32_t c013 = max_v(max_v(b01 + VP_V(3, 2), b03 + VP_V(1, 2)), b13 + VP_V(0, 2));
    const int32_t c023 = max_v(max_v(b02 + VP_V(3, 2), b03 + VP_V(2, 2)), b23 + VP_V(0, 2));
    const int32_t c123 = max_v(max_v(b12 + VP_V(3, 2), b13 + VP_V(2, 2)), b23 + VP_V(1, 2));
    return (uint32_t)max_v(max_v(c012 + VP_V(3, 3), c013 + VP_V(2, 3)), max_v(c023 + VP_V(1, 3), c123 + VP_V(0, 3)));
#undef VP_V
}

// W = warps per (family, start) task: one lane per rank group, 32 W >= G.
template <int W>
__global__ void __launch_bounds__(512, 1)
vp_schedule_big_kernel(DevCat dc, KParams kp, const int64_t* __restrict__ demand, const int64_t* __restrict__ tau_in, int B,
                       int32_t* __restrict__ n_steps, int32_t* __restrict__ chan_id, int16_t* __restrict__ lane_dst,
                       uint16_t* __restrict__ lane_inst, int64_t* __restrict__ lane_bytes, int64_t* __restrict__ send_off,
                       int64_t* __restrict__ recv_off, int64_t* __restrict__ tau_out, int32_t* __restrict__ status,
                       int64_t* ws_drem, unsigned int* counter, int* __restrict__ todo) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int N = dc.N, G = dc.G, tid = threadIdx.x, NT = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, n_warps = NT >> 5;
    const BigSmem L = big_smem_layout(dc, kp);
    const int CS = L.cs_stride;
    uint16_t* Cs = (uint16_t*)(smem_raw + L.cs);
    uint32_t* tbl = (uint32_t*)(smem_raw + L.tbl);
    uint64_t* rs = (uint64_t*)(smem_raw + L.rs);
    uint32_t* pat = (uint32_t*)(smem_raw + L.pat);
    uint8_t* gnode = smem_raw + L.gnode;                 // per group: node index, then (at G) rail index
    int64_t* send_acc = (int64_t*)(smem_raw + L.send_acc);
    int64_t* recv_acc = (int64_t*)(smem_raw + L.recv_acc);
    int64_t* red = (int64_t*)(smem_raw + L.red);
    int64_t* pairs = (int64_t*)(smem_raw + L.pair);
    int64_t* task_f = (int64_t*)(smem_raw + L.task_f);
    int64_t* task_den = (int64_t*)(smem_raw + L.task_den);
    uint32_t* slotw = (uint32_t*)(smem_raw + L.slotw);
    uint8_t* bind_src = smem_raw + L.bind_src;
    uint8_t* bind_dst = smem_raw + L.bind_dst;
    uint32_t* spat = (uint32_t*)(smem_raw + L.term);      // row-pattern ids per shape
    uint32_t* bucket = (uint32_t*)(smem_raw + L.bucket);
    uint32_t* Dg = (uint32_t*)(ws_drem + (size_t)blockIdx.x * N * N);      // exact residual, granules
    __shared__ int s_b, s_flags, s_ok;
    __shared__ int64_t s_tau, s_left;
    __shared__ int64_t s_tscale[VP_MAX_CLASSES];
    __shared__ uint32_t s_cap[VP_MAX_CLASSES];
    __shared__ __align__(8) unsigned long long s_stage_bar;
    unsigned long long n_act = 0, n_tasks_done = 0, n_sweeps = 0;
    Counters cnt;                                        // phase cycle counts (only with VP_PHASE_TIMING)
    cnt.t_mark = 0;
    for (int i = 0; i < 6; i++) cnt.cyc[i] = 0;
    const int ns_pad = (dc.n_shapes + 31) & ~31;
    const int S = dc.S, P = dc.P;

    // ---- stage the catalog once per CTA: packed terms and bucket pointers by bulk asynchronous copies (TMA) onto one
    // mbarrier; should the bounded wait give up, plain loads fetch the same arrays
    {
        const unsigned b_term = (unsigned)(ns_pad * L.pat_words * 4), b_bucket = (unsigned)align16((dc.n_shapes + 1) * 4);
        const unsigned b_pat = (unsigned)align16(dc.n_patterns * dc.max_row_terms * 4);
        bool landed = false;
        if (b_term + b_bucket + b_pat < (1u << 20)) {
            const unsigned bar = smem_u32(&s_stage_bar);
            if (tid == 0) {
                mbar_init(bar, 1);
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                mbar_expect_tx(bar, b_term + b_bucket + b_pat);
                bulk_load(smem_u32(spat), dc.shape_pat, b_term, bar);
                bulk_load(smem_u32(bucket), dc.bucket_ptr, b_bucket, bar);
                bulk_load(smem_u32(pat), dc.pat_term, b_pat, bar);
            }
            __syncthreads();
            landed = __syncthreads_and(mbar_wait_bounded(bar, 0, 1u << 20)) != 0;
        }
        if (!landed) {
            for (int e = tid; e < ns_pad * L.pat_words; e += NT) spat[e] = dc.shape_pat[e];
            for (int e = tid; e <= dc.n_shapes; e += NT) bucket[e] = dc.bucket_ptr[e];
            for (int e = tid; e < dc.n_patterns * dc.max_row_terms; e += NT) pat[e] = dc.pat_term[e];
        }
        for (int a = tid; a < G; a += NT) { gnode[a] = (uint8_t)(a / S); gnode[G + a] = (uint8_t)(a % S); }
        __syncthreads();
    }
    const int ns_shift = (kp.n_start & (kp.n_start - 1)) == 0 ? 31 - __clz(kp.n_start) : -1;
    const int n_score_warps = min(n_warps, (dc.n_shapes + 31) >> 5);

    for (;;) {
        if (tid == 0) { s_b = (int)atomicAdd(counter, 1u); s_flags = 0; }
        __syncthreads();
        const int b = s_b;
        if (b >= B) break;
#ifdef VP_PHASE_TIMING
        cnt.t_mark = clock64();
#endif
        const int64_t* D = demand + (size_t)b * N * N;
        const size_t lane_base = (size_t)b * kp.k_max * N, off_base = (size_t)b * (kp.k_max + 1) * N;
        int32_t* chan_id_b = chan_id + (size_t)b * kp.k_max;
        int16_t* lane_dst_b = lane_dst + lane_base;
        uint16_t* lane_inst_b = lane_inst + lane_base;
        int64_t* lane_bytes_b = lane_bytes + lane_base;
        int64_t* send_off_b = send_off + off_base;
        int64_t* recv_off_b = recv_off ? recv_off + off_base : nullptr;

        // ---- pass 1 over D: validate; row sums, column sums and group sums (Eq. 5) into the set-up area
        int64_t* Dhat = (int64_t*)(smem_raw + L.cs);
        int64_t* rowsum = Dhat + G * G;
        int64_t* colsum = rowsum + N;
        for (int i = tid; i < N; i += NT) { colsum[i] = 0; send_acc[i] = 0; recv_acc[i] = 0; }
        __syncthreads();
        int flags = 0;
        for (int a = warp; a < G; a += n_warps) {            // one warp per source group: four rows, eight columns per lane
            int64_t cell0 = 0, cell1 = 0, col[8];
#pragma unroll
            for (int m = 0; m < 8; m++) col[m] = 0;
#pragma unroll
            for (int i4 = 0; i4 < 4; i4++) {
                const int i = a * 4 + i4;
                int64_t rs = 0;
#pragma unroll
                for (int m = 0; m < 8; m++) {
                    const int j = lane * 8 + m;
                    int64_t v = 0;
                    if (j < N) {
                        v = D[(size_t)i * N + j];
                        if (v < 0) flags |= VP_ST_NEGATIVE;
                        else if (v >= VP_ENTRY_LIMIT) flags |= VP_ST_OVERFLOW_RISK;
                        else {
                            if (i == j && v != 0) flags |= VP_ST_DIAG_NONZERO;
                            if (v % kp.granule) flags |= VP_ST_NOT_GRANULE;
                        }
                    }
                    rs += v;
                    col[m] += v;
                    if (m < 4) cell0 += v; else cell1 += v;
                }
                rs = warp_sum_i64(rs);
                if (lane == 0) rowsum[i] = rs;
            }
            if (lane * 2 < G) Dhat[a * G + lane * 2] = cell0;
            if (lane * 2 + 1 < G) Dhat[a * G + lane * 2 + 1] = cell1;
#pragma unroll
            for (int m = 0; m < 8; m++)
                if (lane * 8 + m < N) atomicAdd((unsigned long long*)&colsum[lane * 8 + m], (unsigned long long)col[m]);
        }
        const int64_t tau_given = tau_in ? tau_in[b] : 0;
        if (tid == 0 && (tau_given < 0 || tau_given > VP_ENTRY_LIMIT)) flags |= VP_ST_BAD_TAU;
        if (flags) atomicOr(&s_flags, flags);
        for (int i = tid; i < N; i += NT) {
            send_off_b[i] = 0;
            if (recv_off_b) recv_off_b[i] = 0;
        }
        __syncthreads();
        int st = s_flags;
        int k = 0;
        int64_t tau = 0;
        bool deferred = false;
        if (st == 0) {
            // ---- quantum (Section 5) and capacities
            int64_t est = 0, tot = 0;
            for (int i = tid; i < N; i += NT) {
                tot += rowsum[i];
                est = max_v(est, max_v(ceil_div_i64(rowsum[i], dc.bw_max), ceil_div_i64(colsum[i], dc.bw_max)));
            }
            for (int l = tid; l < dc.n_res; l += NT) {
                const uint32_t bwl = dc.forced_bw[l];
                if (!bwl) continue;
                int64_t f = 0;
                for (uint32_t e = dc.forced_ptr[l]; e < dc.forced_ptr[l + 1]; e++) f += Dhat[dc.forced_cell[e]];
                est = max_v(est, ceil_div_i64(f, (int64_t)bwl));
            }
            est = warp_max_i64(est);
            tot = warp_sum_i64(tot);
            if (lane == 0) { red[warp] = est; red[32 + warp] = tot; }
            __syncthreads();
            if (tid == 0) {
                int64_t e = 0, t = 0;
                for (int w = 0; w < n_warps; w++) { e = max_v(e, red[w]); t += red[32 + w]; }
                const int64_t tq = tau_given > 0 ? tau_given : max_v((int64_t)1, ceil_div_i64(e, (int64_t)kp.k_target));
                int64_t cap_max = 0;
                for (int cl = 0; cl < dc.n_classes; cl++) {
                    int64_t cp = (tq * dc.class_bw[cl]) / kp.granule * kp.granule;
                    if (cp < kp.granule) cp = kp.granule;
                    cap_max = max_v(cap_max, cp);
                    s_cap[cl] = (uint32_t)min_v(cp / kp.granule, (int64_t)0xffffffffll);
                    s_tscale[cl] = dc.class_wdiv[cl] * kp.granule;
                }
                // 16-bit credits need capacities below 2^16 granules; the 32-bit table needs fewer than 2^32 granules in all
                s_ok = kp.granule >= 256 && cap_max / kp.granule < 65535 && t / kp.granule < ((int64_t)1 << 32);
                s_tau = tq; s_left = t / kp.granule;
            }
            __syncthreads();
            tau = s_tau;
            deferred = !s_ok;
        }
        if (deferred) {
            // the general kernel takes this matrix (it validates and derives the quantum again)
            if (tid == 0) todo[atomicAdd(counter + 1, 1u)] = b;
            __syncthreads();
            continue;
        }
        if (st == 0) {
            // ---- first score table from D-hat, in granules
            for (int e = tid; e < dc.tbl_size; e += NT) {
                const int q2 = e % S, q = (e / S) % S, delta = e / (S * S);
                int64_t s = 0;
                for (int n = 0; n < P; n++) {
                    int n2 = n + delta; if (n2 >= P) n2 -= P;
                    s += Dhat[(size_t)(n * S + q) * G + n2 * S + q2];
                }
                tbl[e] = (uint32_t)(s / kp.granule);
            }
            __syncthreads();
            // ---- pass 2 over D: the residual in granules (workspace slot) and its saturating 16-bit copy
            for (int e = tid; e < N * N; e += NT) {
                const uint32_t v = (uint32_t)(D[e] / kp.granule);
                const int i = e / N, j = e - i * N;
                Dg[e] = v;
                Cs[i * CS + j] = (uint16_t)min_v(v, 65535u);
            }
            __syncthreads();
            int64_t left = s_left;
            VP_TICK(0);

            for (;;) {
                if (left == 0) break;
                if (k == kp.k_max) { st |= VP_ST_STEP_LIMIT; break; }
                // (A) Eq. (6): shape scores on the table, first maximum
                for (int p = tid; p < dc.n_patterns; p += NT) {       // row scores: at most max_row_terms products each
                    uint64_t v = 0;
                    for (int t = 0; t < dc.max_row_terms; t++) {
                        const uint32_t tw = pat[p * dc.max_row_terms + t];
                        v += (uint64_t)tbl[tw & 0xffffu] * (tw >> 16);
                    }
#pragma unroll
                    for (int r = 0; r < BIG_RS_COPIES; r++) rs[p * BIG_RS_COPIES + r] = v;
                }
                __syncthreads();
                if (warp < n_score_warps) {
                    int64_t best = -1;
                    int best_s = 0x7fffffff;
                    const uint64_t* rl = rs + (lane & (BIG_RS_COPIES - 1));
                    for (int s = tid; s < dc.n_shapes; s += NT) {
                        uint64_t score = 0;
                        for (int w = 0; w < L.pat_words; w++) {
                            const uint32_t pw = spat[w * ns_pad + s];
                            score += rl[(pw & 0xffffu) * BIG_RS_COPIES];
                            if (2 * w + 1 < S) score += rl[(pw >> 16) * BIG_RS_COPIES];
                        }
                        if ((int64_t)score > best) { best = (int64_t)score; best_s = s; }
                    }
                    warp_argmax_first(best, best_s);
                    if (lane == 0) { red[warp] = best; red[32 + warp] = best_s; }
                }
                __syncthreads();
                int64_t best = lane < n_score_warps ? red[lane] : -1;
                int best_s = lane < n_score_warps ? (int)red[32 + lane] : 0x7fffffff;
                warp_argmax_first(best, best_s);
                if (best <= 0) { st |= VP_ST_UNCOVERED; break; }
                const int f0 = (int)bucket[best_s], H = (int)bucket[best_s + 1] - f0;
                const int n_tasks = H * kp.n_start;
                VP_TICK(1);

                // (B) MultiStartAA: W warps per (family, start), one lane per rank group
                const int sub = W == 2 ? (warp & 1) : 0, wgroup = W == 2 ? (warp >> 1) : warp;
                const int a = sub * 32 + lane;                   // this lane's group: source group, then destination group
                const bool active = a < G;
                auto task_sync = [&]() {
                    if (W == 2) asm volatile("bar.sync %0, 64;" ::"r"(1 + wgroup) : "memory");
                    else __syncwarp();
                };
                for (int task = wgroup; task < n_tasks; task += n_warps / W) {
                    const int h = ns_shift >= 0 ? task >> ns_shift : task / kp.n_start, f = f0 + h, t = task - h * kp.n_start;
                    uint8_t* srcb = bind_src + (size_t)task * N;
                    uint8_t* dstb = bind_dst + (size_t)task * N;
                    uint32_t cap_out[4], cap_in[4];
                    int rq[4], cls_in[4];
                    if (active) {
                        const uint32_t co = __ldg((const uint32_t*)(dc.fam_cls + (size_t)f * N) + a);
                        const uint2 fi = __ldg((const uint2*)(dc.fam_in + (size_t)f * N) + a);
                        const uint32_t fw[4] = {fi.x & 0xffffu, fi.x >> 16, fi.y & 0xffffu, fi.y >> 16};
#pragma unroll
                        for (int q = 0; q < 4; q++) {
                            cap_out[q] = s_cap[(co >> (8 * q)) & 0xffu] << 8;
                            rq[q] = (int)(fw[q] & 0xffu);
                            cls_in[q] = (int)(fw[q] >> 8);
                            cap_in[q] = s_cap[cls_in[q]] << 8;
                            dstb[rq[q]] = (uint8_t)(a * 4 + ((q + t) & 3));      // start t rotates the in-slots
                        }
                        if (t == 0) {                             // the family's slot words, parked for step (D)
                            const uint4 sw = __ldg((const uint4*)(dc.fam_slot + (size_t)f * N) + a);
                            *((uint4*)(slotw + h * N) + a) = sw;
                        }
                    }
                    task_sync();
                    int64_t F_old = -1, F_new = -1;
                    uint32_t xmax = 0;
                    int64_t tmax = 0;
                    int64_t* pair = pairs + wgroup * 6;
                    for (int sweep = 0; sweep < kp.i_aa; sweep++) {
                        if (active) {                             // source half: one exact assignment per source group
                            const uint32_t d4 = *((const uint32_t*)dstb + a);
                            uint32_t cr[4][4];
#pragma unroll
                            for (int q = 0; q < 4; q++) {
                                const uint16_t* colp = Cs + (a * 4) * CS + ((d4 >> (8 * q)) & 0xffu);
#pragma unroll
                                for (int i = 0; i < 4; i++) cr[i][q] = min_v((uint32_t)colp[i * CS] << 8, cap_out[q]);
                            }
                            const uint32_t pb = ~big_best_key(cr) & 255u;
                            *((uint32_t*)srcb + a) = (uint32_t)(a * 4) * 0x01010101u +
                                                     (((pb >> 6) & 3u) | (((pb >> 4) & 3u) << 8) | (((pb >> 2) & 3u) << 16) | ((pb & 3u) << 24));
                        }
                        task_sync();
                        uint32_t part = 0;
                        if (active) {                             // destination half
                            uint32_t cr[4][4];
#pragma unroll
                            for (int q = 0; q < 4; q++) {
                                const uint32_t* rowp = (const uint32_t*)(Cs + (int)srcb[rq[q]] * CS + a * 4);
                                const uint32_t lo = rowp[0], hi = rowp[1];
                                cr[0][q] = min_v(__byte_perm(lo, 0, 0x4104), cap_in[q]);     // (low half) << 8
                                cr[1][q] = min_v(__byte_perm(lo, 0, 0x4324), cap_in[q]);     // (high half) << 8
                                cr[2][q] = min_v(__byte_perm(hi, 0, 0x4104), cap_in[q]);
                                cr[3][q] = min_v(__byte_perm(hi, 0, 0x4324), cap_in[q]);
                            }
                            const uint32_t key = big_best_key(cr);
                            const uint32_t pb = ~key & 255u;
                            part = key >> 8;                      // key = (sum of credits) << 8 | tag
#pragma unroll
                            for (int q = 0; q < 4; q++) dstb[rq[q]] = (uint8_t)(a * 4 + ((pb >> (6 - 2 * q)) & 3u));
                        }
                        F_new = (int64_t)__reduce_add_sync(0xffffffffu, part);          // Eq. (8); at most 2^8 lanes of < 2^16
                        if (W == 2) {                             // add the partner warp's half (slots alternate by sweep)
                            if (lane == 0) pair[(sweep & 1) * 2 + sub] = F_new;
                            task_sync();
                            F_new = pair[(sweep & 1) * 2] + pair[(sweep & 1) * 2 + 1];
                        } else {
                            __syncwarp();
                        }
                        if (sub == 0 && lane == 0) n_sweeps++;
                        if (F_new <= F_old) break;
                        F_old = F_new;
                    }
                    // Eq. (9) volumes of the binding as it stands: the credit of every in-slot; slowest lane of Eq. (10)
                    if (active) {
#pragma unroll
                        for (int q = 0; q < 4; q++) {
                            const uint32_t x = min_v((uint32_t)Cs[(int)srcb[rq[q]] * CS + (int)dstb[rq[q]]], cap_in[q] >> 8);
                            xmax = max_v(xmax, x);
                            if (dc.n_classes > 1) tmax = max_v(tmax, (int64_t)x * s_tscale[cls_in[q]]);
                        }
                    }
                    if (dc.n_classes == 1) tmax = (int64_t)__reduce_max_sync(0xffffffffu, xmax) * s_tscale[0];
                    else tmax = warp_max_i64(tmax);
                    if (W == 2) {
                        if (lane == 0) pair[4 + sub] = tmax;
                        task_sync();
                        tmax = max_v(pair[4], pair[5]);
                    }
                    if (lane == 0 && sub == 0) {
                        n_tasks_done++;
                        task_f[task] = F_new;
                        task_den[task] = F_new > 0 ? kp.lambda_ns * dc.W + tmax : 1;
                    }
                }
                __syncthreads();
                VP_TICK(2);

                // (C) best start per family (largest F, lowest t), then largest utility, lowest family
                int wtask;
                int64_t wF;
                if (H == 1 && kp.n_start <= 32) {
                    int64_t ff = lane < kp.n_start ? task_f[lane] : -1;
                    int tt = lane;
                    warp_argmax_first(ff, tt);
                    wtask = tt; wF = ff;
                } else {
                    int64_t bf = -1, bd = 1;
                    int bt = 0x7fffffff;
                    for (int h = lane; h < H; h += 32) {
                        int64_t ff = -1; int tt = 0;
                        for (int t = 0; t < kp.n_start; t++)
                            if (task_f[h * kp.n_start + t] > ff) { ff = task_f[h * kp.n_start + t]; tt = h * kp.n_start + t; }
                        if (bt == 0x7fffffff || util_greater(ff, task_den[tt], bf, bd)) { bf = ff; bd = task_den[tt]; bt = tt; }
                    }
                    for (int o = 16; o; o >>= 1) {
                        const int64_t of = __shfl_xor_sync(0xffffffffu, bf, o), od = __shfl_xor_sync(0xffffffffu, bd, o);
                        const int ot = __shfl_xor_sync(0xffffffffu, bt, o);
                        bool take = false;
                        if (ot != 0x7fffffff) {
                            if (bt == 0x7fffffff) take = true;
                            else if (util_greater(of, od, bf, bd)) take = true;
                            else if (!util_greater(bf, bd, of, od) && ot < bt) take = true;
                        }
                        if (take) { bf = of; bd = od; bt = ot; }
                    }
                    wtask = __shfl_sync(0xffffffffu, bt, 0);
                    wF = __shfl_sync(0xffffffffu, bf, 0);
                }
                if (wF <= 0) { st |= VP_ST_NO_PROGRESS; break; }
                VP_TICK(3);

                // (D) emit activation k: volumes off the residual and off the score table, next offset row
                {
                    const int h = ns_shift >= 0 ? wtask >> ns_shift : wtask / kp.n_start;
                    const uint32_t* slot = slotw + h * N;
                    const uint8_t* srcb = bind_src + (size_t)wtask * N;
                    const uint8_t* dstb = bind_dst + (size_t)wtask * N;
                    const size_t row = (size_t)k * N, orow = (size_t)(k + 1) * N;
                    for (int r0 = warp * 32; r0 < N; r0 += NT) {  // whole warps: the sums below need every lane
                        const int r = r0 + lane;
                        const bool live = r < N;
                        uint32_t x = 0, mine = 0xffffffffu;
                        if (live) {
                            const uint32_t w = slot[r];
                            const int i = srcb[r], j = dstb[r];
                            uint16_t* cell = Cs + i * CS + j;
                            const uint32_t c = *cell;
                            x = min_v(s_cap[(w >> 24) & 0xf], c);
                            const bool busy = x > 0;
                            const int64_t bytes = (int64_t)x * kp.granule;
                            const int64_t sa = send_acc[i] + bytes, ra = recv_acc[j] + bytes;
                            lane_dst_b[row + i] = busy ? (int16_t)j : (int16_t)-1;
                            lane_inst_b[row + i] = busy ? (uint16_t)(w & 0xffffu) : (uint16_t)0xFFFF;
                            lane_bytes_b[row + i] = bytes;
                            send_acc[i] = sa;
                            recv_acc[j] = ra;
                            send_off_b[orow + i] = sa;            // src and dst are permutations: every rank is written once
                            if (recv_off_b) recv_off_b[orow + j] = ra;
                            if (busy) {
                                uint32_t nv = c - x;
                                if (c == 65535u) {                // saturated: the exact residual is in the workspace slot
                                    nv = atomicSub(&Dg[(size_t)i * N + j], x) - x;
                                    nv = min_v(nv, 65535u);
                                }
                                *cell = (uint16_t)nv;
                                const int ga = i >> 2, gd = j >> 2;
                                int delta = (int)gnode[gd] - (int)gnode[ga];
                                if (delta < 0) delta += P;
                                mine = (uint32_t)((delta * S + gnode[G + ga]) * S + gnode[G + gd]);
                            }
                        }
                        // the volumes leave the table entries of their group pairs: the lanes of an activation fall into
                        // the entries of the chosen shape's terms, so one warp sum per such entry, then one atomic each
                        for (int q = 0; q < S; q++) {
                            const uint32_t pid = (spat[(q >> 1) * ns_pad + best_s] >> (16 * (q & 1))) & 0xffffu;
                            for (int t = 0; t < dc.max_row_terms; t++) {
                                const uint32_t tw = pat[pid * dc.max_row_terms + t];
                                if (!(tw >> 16)) continue;                // (the same word in every thread)
                                const uint32_t sum = __reduce_add_sync(0xffffffffu, mine == (tw & 0xffffu) ? x : 0u);
                                if (lane == 0 && sum) atomicSub(&tbl[tw & 0xffffu], sum);
                            }
                        }
                    }
                    if (tid == 0) chan_id_b[k] = f0 + h;
                    left -= wF;
                }
                k++;
                __syncthreads();
                VP_TICK(4);
            }
        }
        __syncthreads();
        // ---- idle rows beyond n_steps; offset rows repeat the totals
        for (size_t e = (size_t)k * N + tid; e < (size_t)kp.k_max * N; e += NT) {
            lane_dst_b[e] = -1;
            lane_inst_b[e] = 0xFFFF;
            lane_bytes_b[e] = 0;
            const int i = (int)(e % N);
            send_off_b[N + e] = send_acc[i];
            if (recv_off_b) recv_off_b[N + e] = recv_acc[i];
        }
        for (int kk = k + tid; kk < kp.k_max; kk += NT) chan_id_b[kk] = -1;
        if (tid == 0) {
            n_act += (unsigned long long)k;
            n_steps[b] = k;
            status[b] = st;
            if (tau_out) tau_out[b] = tau;
        }
        __syncthreads();
        VP_TICK(5);
    }
    unsigned long long* stats = (unsigned long long*)(counter + 4);
    if (tid == 0 && n_act) atomicAdd(&stats[0], n_act);
    if (lane == 0 && n_tasks_done) { atomicAdd(&stats[1], n_tasks_done); atomicAdd(&stats[2], n_sweeps); }
#ifdef VP_PHASE_TIMING
    if (tid == 0) for (int i = 0; i < 6; i++) atomicAdd(&stats[3 + i], (unsigned long long)cnt.cyc[i]);
#endif
}

}  // namespace
