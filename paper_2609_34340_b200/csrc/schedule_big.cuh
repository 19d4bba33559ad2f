// Algorithm 2 (Section 4.2) for large node-symmetric catalogs: groups of four ranks, more than sixteen groups
// (N = 68 .. 256), shapes invariant under a shift of the node index.  Included by schedule.cu.
//
// One CTA decomposes one matrix at a time.  What differs from the general kernel is where the state lives:
//
//  * Credits.  Step 2 only ever looks at min(D_rem[i][j], cap_r) (Eq. 7).  N x N 16-bit cells fit shared memory (128 KB
//    at N = 256) where the residual in 32-bit granules (256 KB) does not.  A cell below F = 65,536 - M granules is
//    kept as it is; a cell of F granules or more holds F + (its index in a side list of M = 4,096 exact 32-bit
//    values).  As long as every lane capacity is below F, such a cell yields the same credit as its exact value
//    (the capacity), and the emit step keeps the side list exact until the cell drops below F and becomes ordinary.
//  * Scores.  Eq. (6) on a node-symmetric catalog is a sum of at most max_terms products count x C[e], where
//    C[delta][q][q'] = sum_n D-hat[(n,q)][(n+delta,q')] (the same integer as the full sum over D-hat).  The table C
//    (P S S entries, 32-bit granules) is kept in shared memory and every activation subtracts its lane volumes from
//    the entries they fall in, so D-hat itself is needed only once, for the quantum rule and the first table.
//    The terms of a shape are split by source rail into S rows, and the catalog has few distinct rows (127 per rail
//    for 4,095 shapes): an iteration first scores every row pattern (a few hundred sums of at most three products),
//    then every shape is the sum of S looked-up row scores -- two loads and an addition instead of six
//    multiply-adds.  The row scores are kept in eight copies so that the lanes of a warp rarely meet in a bank.
//
//  * Large capacities.  When a lane capacity reaches 2^16 granules (skewed MoE matrices with many tokens), the few
//    columns that hold cells of 65,535 granules or more -- the destinations of the popular experts -- become "hot
//    columns": their cells are kept exactly, low 16 bits in the credit matrix and high 16 bits in a side array of up
//    to 32 columns, and the credits that touch them are patched after the ordinary 16-bit pass.  Every other cell of
//    such a matrix is below 65,535 granules, so its 16-bit copy is exact.  No L2 traffic is needed in this mode.
//
// A matrix that does not meet the conditions (granule below 256 bytes, a capacity of 2^22 granules or more, 2^32
// granules or more in total, more than 32 hot columns, more big cells than the side list holds) is appended to a list that the general kernel works through
// afterwards.
#pragma once

namespace {

// Scoring reads the row scores at data-dependent positions; with one copy per lane class (lane mod 8) the lanes of a
// warp meet in a bank only when they share a class and read different patterns of equal parity.
constexpr int BIG_RS_COPIES = 1;
#ifndef BIG_FILL_LANES
#define BIG_FILL_LANES 8              // bulk copies of the fill issued per iteration of the main loop (32 measured 2 % slower)
#endif
constexpr int BIG_HOT_MAX = 32;       // columns whose cells are kept beyond 16 bits
constexpr int BIG_SMEM_LIMIT = 227 * 1024 - 2048;   // dynamic shared memory of one CTA, less room for the static variables

struct BigSmem {
    int cs, tbl, rs, pat, bnd, dec, hi, colmap, gnode, send_acc, recv_acc, red, pair, task_f, task_den, slotw, bind_src, bind_dst, term, bucket, total;
    int emit, fill, fill_rows;      // source buffers of the asynchronous fill, offset rows per buffer (0: plain stores)
    int cs_stride;            // credits per row of the 16-bit matrix (N + 2: rows start in different banks)
    int pat_words;            // 32-bit words of row-pattern ids per shape (two ids per word)
};

// The arg-max is taken class by class when the catalog allows it and has enough shapes for that to pay: a few hundred
// shapes are scanned faster than two rounds of class maxima.
#ifndef BIG_DEC_MIN_SHAPES
#define BIG_DEC_MIN_SHAPES 1024
#endif
__host__ __device__ inline bool big_use_dec(const DevCat& dc) { return dc.dec != nullptr && dc.n_shapes >= BIG_DEC_MIN_SHAPES; }

__host__ __device__ inline BigSmem big_smem_layout(const DevCat& dc, const KParams& kp) {
    BigSmem L;
    const bool dec = big_use_dec(dc);
    int o = 0;
    L.cs_stride = dc.N + 2;
    const int cs_bytes = dc.N * L.cs_stride * 2, dhat_bytes = dc.G * dc.G * 8 + dc.N * 24;
    L.cs = o;        o += align16(cs_bytes > dhat_bytes ? cs_bytes : dhat_bytes);   // set-up: D-hat, row and column sums
    L.hi = o;        o += BIG_HOT_MAX * dc.N * 2;                  // high halves of the hot columns' cells
    L.colmap = o;    o += align16(dc.N);                          // hot-column index of every rank, 0xFF = none
    L.tbl = o;       o += align16(dc.tbl_size * 4);
    L.rs = o;        o += dc.n_patterns * 8 * BIG_RS_COPIES;      // row scores, one copy per lane class
    L.pat = o;       o += align16(dc.n_patterns * dc.max_row_terms * 4);
    L.bnd = o;       o += dec ? 0 : ((dc.n_shapes + 31) & ~31) * 4;     // upper bounds on (score >> 2) of every shape
    L.dec = o;       o += dec ? align16(dc.dec_words * 4) : 0;     // class decomposition of the arg-max, if any
    L.gnode = o;     o += align16(dc.G * 2);
    L.send_acc = o;  o += dc.N * 8;
    L.recv_acc = o;  o += dc.N * 8;
    L.red = o;       o += 64 * 8;
    L.pair = o;      o += 16 * 8 * 8;
    L.task_f = o;    o += align16(kp.max_tasks * 8);
    L.task_den = o;  o += align16(kp.max_tasks * 8);
    L.slotw = o;     o += align16(dc.max_bucket * dc.N * 4);
    L.bind_src = o;  o += align16(kp.max_tasks * dc.N);
    L.bind_dst = o;  o += align16(kp.max_tasks * dc.N);
    L.pat_words = (dc.S + 1) / 2;
    L.term = o;      o += dec ? 0 : ((dc.n_shapes + 31) & ~31) * L.pat_words * 4;
    L.bucket = o;    o += align16((dc.n_shapes + 1) * 4);
    // Staging row of the emit step (lane_dst, lane_inst, lane_bytes, send_off, recv_off of one activation: 28 N bytes)
    L.emit = o;      o += dc.N % 8 == 0 ? 28 * dc.N : 0;
    // Source buffers of the asynchronous fill: all ones, zeros (written once per CTA), the send totals and the receive
    // totals repeated fill_rows times (per matrix); the idle rows of a plan are written from them by bulk asynchronous
    // copies while the next matrix is decomposed.  Only for the one-CTA-per-SM shape (more than 32 groups), in
    // whatever shared memory is left, and not below 4 KB per buffer.
    L.fill = o;
    L.fill_rows = dc.G > 32 ? (BIG_SMEM_LIMIT - o) / 4 / (dc.N * 8) : 0;
    if (L.fill_rows > 8) L.fill_rows = 8;
    if (L.fill_rows * dc.N * 8 < 4096) L.fill_rows = 0;
    o += 4 * L.fill_rows * dc.N * 8;
    L.total = o;
    return L;
}

// Tag of row r at position q of a 4 x 4 assignment: (3 - r) in the two bits that position q owns in a byte whose
// two highest bits belong to position 0.  The four tags of a permutation add up to 255 minus the permutation written
// as a byte, so a credit sum carried as (sum << 8) + tags is largest for the largest sum and, among equal sums, for
// the first permutation in lexicographic order -- the same winner as an enumeration that keeps the first maximum.
__host__ __device__ constexpr uint32_t big_tag(int r, int q) { return (uint32_t)(3 - r) << (6 - 2 * q); }

__device__ __forceinline__ uint32_t add_max(uint32_t a, uint32_t b, uint32_t c) { return __viaddmax_u32(a, b, c); }   // max(a + b, c)

// Exact 4 x 4 assignment: v[r][q] = (credit of row r at position q) << 8 | big_tag(r, q).  Returns the largest
// sum_q v[phi(q)][q] over the permutations phi, by dynamic programming over the set of rows placed so far (positions
// 0, 1, 2, 3 in turn), 28 add / add-max operations.  The permutation byte is ~key & 255, the credit sum key >> 8.
__device__ __forceinline__ uint32_t big_best_key(const uint32_t (&v)[4][4]) {
    const uint32_t b01 = add_max(v[0][0], v[1][1], v[1][0] + v[0][1]), b02 = add_max(v[0][0], v[2][1], v[2][0] + v[0][1]);
    const uint32_t b03 = add_max(v[0][0], v[3][1], v[3][0] + v[0][1]), b12 = add_max(v[1][0], v[2][1], v[2][0] + v[1][1]);
    const uint32_t b13 = add_max(v[1][0], v[3][1], v[3][0] + v[1][1]), b23 = add_max(v[2][0], v[3][1], v[3][0] + v[2][1]);
    const uint32_t c012 = add_max(b01, v[2][2], add_max(b02, v[1][2], b12 + v[0][2]));
    const uint32_t c013 = add_max(b01, v[3][2], add_max(b03, v[1][2], b13 + v[0][2]));
    const uint32_t c023 = add_max(b02, v[3][2], add_max(b03, v[2][2], b23 + v[0][2]));
    const uint32_t c123 = add_max(b12, v[3][2], add_max(b13, v[2][2], b23 + v[1][2]));
    return add_max(c012, v[3][3], add_max(c013, v[2][3], add_max(c023, v[1][3], c123 + v[0][3])));
}

// Maximum of distinct 64-bit keys over the warp: the largest high word, then the largest low word among its holders.
__device__ __forceinline__ uint64_t big_warp_max64(uint64_t key) {
    const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key;
    const uint32_t mhi = __reduce_max_sync(0xffffffffu, hi);
    const uint32_t mlo = __reduce_max_sync(0xffffffffu, hi == mhi ? lo : 0u);
    return (uint64_t)mhi << 32 | mlo;
}

// Fills bytes [lo, hi) of dst with a repeated byte, by 16-byte stores where the address allows (all threads of the CTA).
__device__ __forceinline__ void big_fill_bytes(unsigned char* dst, size_t lo, size_t hi, unsigned char byte, int tid, int NT) {
    if (lo >= hi) return;
    const size_t head = min((size_t)((16 - ((uintptr_t)(dst + lo) & 15)) & 15), hi - lo);
    for (size_t e = lo + tid; e < lo + head; e += NT) dst[e] = byte;
    const size_t vlo = lo + head, nvec = (hi - vlo) / 16;
    const uint32_t w = 0x01010101u * byte;
    uint4* v = (uint4*)(dst + vlo);
    for (size_t e = tid; e < nvec; e += NT) v[e] = make_uint4(w, w, w, w);
    for (size_t e = vlo + nvec * 16 + tid; e < hi; e += NT) dst[e] = byte;
}

// (out of line: 64-bit division is long, and granules are powers of two in practice)
__device__ __noinline__ bool big_not_multiple(int64_t x, int64_t granule) { return x % granule != 0; }
__device__ __noinline__ uint32_t big_div_granule(int64_t x, int64_t granule) { return (uint32_t)(x / granule); }

// Step 3 when several families compete (kept out of line: most shapes have one family, and the main loop should
// stay small for the instruction cache): best start per family (largest F, lowest start), then the family of largest
// utility F / duration by exact cross-multiplication, lowest family first among equals.  Whole warp.
__device__ __noinline__ void big_select_family(const int64_t* task_f, const int64_t* task_den, int H, int n_start, int lane,
                                               int& wtask, int64_t& wF) {
    int64_t bf = -1, bd = 1;
    int bt = 0x7fffffff;
    for (int h = lane; h < H; h += 32) {
        int64_t ff = -1; int tt = 0;
        for (int t = 0; t < n_start; t++)
            if (task_f[h * n_start + t] > ff) { ff = task_f[h * n_start + t]; tt = h * n_start + t; }
        if (bt == 0x7fffffff || util_greater(ff, task_den[tt], bf, bd)) { bf = ff; bd = task_den[tt]; bt = tt; }
    }
#pragma unroll 1
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

// Eq. (9) volumes of a binding as it stands (the credit of every in-slot of this lane's group) and the slowest lane of
// Eq. (10) over the warp, in rate-lcm time units.  Only needed when several families compete.  Whole warp.
__device__ __noinline__ int64_t big_slowest_lane(const uint16_t* Cs, int CS, const uint16_t* Hi, const uint8_t* colmap, int N,
                                                 bool hot_mode, const uint8_t* srcb, const uint8_t* dstb,
                                                 const int (&rq)[4], const uint32_t (&cap_in)[4], const int (&cls_in)[4],
                                                 const int64_t* tscale, int n_classes, bool active) {
    int64_t tmax = 0;
    uint32_t xmax = 0;
    if (active) {
#pragma unroll 1
        for (int q = 0; q < 4; q++) {
            const int sq = srcb[rq[q]], dq = dstb[rq[q]];
            uint32_t val = Cs[sq * CS + dq];
            if (hot_mode && colmap[dq] != 0xFF) val |= (uint32_t)Hi[(int)colmap[dq] * N + sq] << 16;
            const uint32_t x = min_v(val, cap_in[q]);
            xmax = max_v(xmax, x);
            if (n_classes > 1) tmax = max_v(tmax, (int64_t)x * tscale[cls_in[q]]);
        }
    }
    if (n_classes == 1) return (int64_t)__reduce_max_sync(0xffffffffu, xmax) * tscale[0];
    return warp_max_i64(tmax);
}

// Work order for a batch whose matrices differ a lot in length: the number of non-zero cells predicts the number of
// activations well (dense cross-node MoE demand takes several times as many as block-diagonal sequence-parallel
// demand), and CTAs that take the long matrices first leave a short tail.  One warp counts one matrix ...
__global__ void __launch_bounds__(256) big_count_nonzero_kernel(const int64_t* __restrict__ demand, int B, int cells, int* __restrict__ key) {
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (b >= B) return;
    const int64_t* D = demand + (size_t)b * cells;
    int n = 0;
    for (int e = lane; e < cells; e += 32) n += D[e] != 0;
    n = __reduce_add_sync(0xffffffffu, n);
    if (lane == 0) key[b] = n;
}
// ... and every matrix finds its place by counting the matrices that go before it (more non-zero cells, or as many
// and a lower index): B^2 comparisons over the whole grid, a few microseconds for a few thousand matrices.
__global__ void __launch_bounds__(256) big_rank_kernel(const int* __restrict__ key, int B, int* __restrict__ order) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int mine = key[b];
    int before = 0;
    for (int o = 0; o < B; o++) {
        const int other = __ldg(&key[o]);
        before += other > mine || (other == mine && o < b);
    }
    order[before] = b;
}

// W = warps per (family, start) task: one lane per rank group, 32 W >= G.  With at most sixteen groups two tasks share a
// warp (W = 1, launched with two warps per CTA); with 17 to 32 groups a CTA is four warps, a task each; with more, W = 2
// and a CTA is twelve warps, eight of which hold the four tasks of Step 2.
#ifndef VP_BIG_W1_CTAS
#define VP_BIG_W1_CTAS 2
#endif
// DEC: the arg-max of Eq. (6) is taken class by class (see big_use_dec).
template <int W, bool DEC>
#ifndef BIG_W2_THREADS
#define BIG_W2_THREADS 384             // 8 task warps + 4 others; 512 (8 others) measured 6 % slower, 320 5 % slower
#endif
#ifndef BIG_W1_MAXT
#define BIG_W1_MAXT 256
#endif
__global__ void __launch_bounds__(W == 2 ? BIG_W2_THREADS : BIG_W1_MAXT, W == 2 ? 1 : VP_BIG_W1_CTAS)
vp_schedule_big_kernel(DevCat dc, KParams kp, const int64_t* __restrict__ demand, const int64_t* __restrict__ tau_in, int B,
                       int32_t* __restrict__ n_steps, int32_t* __restrict__ chan_id, int16_t* __restrict__ lane_dst,
                       uint16_t* __restrict__ lane_inst, int64_t* __restrict__ lane_bytes, int64_t* __restrict__ send_off,
                       int64_t* __restrict__ recv_off, int64_t* __restrict__ tau_out, int32_t* __restrict__ status,
                       unsigned int* counter, int* __restrict__ todo, const int* __restrict__ order) {
    // `order` (may be null) lists the matrices in the order in which the CTAs should take them: longest first.
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int N = dc.N, G = dc.G, tid = threadIdx.x, NT = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, n_warps = NT >> 5;
    const BigSmem L = big_smem_layout(dc, kp);
    const int CS = L.cs_stride;
    uint16_t* Cs = (uint16_t*)(smem_raw + L.cs);
    uint32_t* tbl = (uint32_t*)(smem_raw + L.tbl);
    uint16_t* Hi = (uint16_t*)(smem_raw + L.hi);
    uint8_t* colmap = smem_raw + L.colmap;
    uint64_t* rs = (uint64_t*)(smem_raw + L.rs);
    uint32_t* pat = (uint32_t*)(smem_raw + L.pat);
    uint32_t* bnd = (uint32_t*)(smem_raw + L.bnd);
    const uint32_t* decs = (const uint32_t*)(smem_raw + L.dec);
    const int dec_n = DEC ? dc.dec_classes : 0;
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
    // Big cells (16-bit mode): a cell of big_floor granules or more holds big_floor + its index in the side list, where
    // its exact value is kept.  Every capacity is below big_floor, so such a cell gives the same credit as its value.
    uint32_t* side = (uint32_t*)(smem_raw + L.hi);
    const int big_max = min(BIG_HOT_MAX * N / 2, 4096), big_floor = 65536 - big_max;
    __shared__ int s_b, s_flags, s_mode, s_nhot, s_nbig;           // s_mode: 0 leave to the general kernel, 1 plain, 2 hot columns
    __shared__ int64_t s_tau, s_left;
    __shared__ int64_t s_tscale[VP_MAX_CLASSES];
    __shared__ uint32_t s_cap[VP_MAX_CLASSES];
    __shared__ __align__(8) unsigned long long s_stage_bar;
    // Pending fill: the idle rows of the last finished matrix.  Arrays 0 and 1 (lane_dst, lane_inst) take 4 fill_rows rows
    // per bulk copy, arrays 2 to 4 (lane_bytes, send_off, recv_off) fill_rows rows; copies are numbered array by array.
    __shared__ unsigned char* s_job_ptr[5];
    __shared__ int s_job_rows, s_job_next, s_job_total;
    constexpr int FILL_WARP = 8;                         // issues the copies, a batch per iteration of the main loop
    unsigned long long n_act = 0, n_tasks_done = 0, n_sweeps = 0;
    Counters cnt;                                        // phase cycle counts (only with VP_PHASE_TIMING)
    cnt.t_mark = 0;
    for (int i = 0; i < 6; i++) cnt.cyc[i] = 0;
    const int ns_pad = (dc.n_shapes + 31) & ~31;
    const int S = dc.S, P = dc.P;

    // ---- stage the catalog once per CTA: packed terms and bucket pointers by bulk asynchronous copies (TMA) onto one
    // mbarrier; should the bounded wait give up, plain loads fetch the same arrays
    {
        const unsigned b_term = DEC ? 0u : (unsigned)(ns_pad * L.pat_words * 4), b_bucket = (unsigned)align16((dc.n_shapes + 1) * 4);
        const unsigned b_pat = (unsigned)align16(dc.n_patterns * dc.max_row_terms * 4);
        bool landed = false;
        if (b_term + b_bucket + b_pat < (1u << 20)) {
            const unsigned bar = smem_u32(&s_stage_bar);
            if (tid == 0) {
                mbar_init(bar, 1);
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                mbar_expect_tx(bar, b_term + b_bucket + b_pat);
                if (b_term) bulk_load(smem_u32(spat), dc.shape_pat, b_term, bar);
                bulk_load(smem_u32(bucket), dc.bucket_ptr, b_bucket, bar);
                bulk_load(smem_u32(pat), dc.pat_term, b_pat, bar);
            }
            __syncthreads();
            landed = __syncthreads_and(mbar_wait_bounded(bar, 0, 1u << 20)) != 0;
        }
        if (!landed) {
            for (int e = tid; e < ns_pad * L.pat_words && !DEC; e += NT) spat[e] = dc.shape_pat[e];
            for (int e = tid; e <= dc.n_shapes; e += NT) bucket[e] = dc.bucket_ptr[e];
            for (int e = tid; e < dc.n_patterns * dc.max_row_terms; e += NT) pat[e] = dc.pat_term[e];
        }
        for (int a = tid; a < G; a += NT) { gnode[a] = (uint8_t)(a / S); gnode[G + a] = (uint8_t)(a % S); }
        for (int e = tid; e < L.fill_rows * N * 8 / 16; e += NT) {       // fill buffers: all ones, then zeros
            ((uint4*)(smem_raw + L.fill))[e] = make_uint4(0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu);
            ((uint4*)(smem_raw + L.fill + L.fill_rows * N * 8))[e] = make_uint4(0u, 0u, 0u, 0u);
        }
        for (int e = tid; e < dc.dec_words && DEC; e += NT) ((uint32_t*)(smem_raw + L.dec))[e] = dc.dec[e];
        __syncthreads();
        // pattern ids become byte offsets into the row scores (fewer than 1,024 patterns, so they still fit 16 bits)
        for (int e = tid; e < ns_pad * L.pat_words && !DEC; e += NT) {
            const uint32_t w = spat[e];
            spat[e] = (w & 0xffffu) * (8 * BIG_RS_COPIES) | ((w >> 16) * (8 * BIG_RS_COPIES)) << 16;
        }
        __syncthreads();
    }
    const int ns_shift = (kp.n_start & (kp.n_start - 1)) == 0 ? 31 - __clz(kp.n_start) : -1;
    const bool tpw2 = W == 1 && G <= 16;                 // two tasks per warp in Step 2 (see there)
    // Issues up to `batches` x 32 of the pending copies (one per lane) and commits them; FILL_WARP only.
    auto fill_step = [&](int batches) {
        const int R = L.fill_rows, rows = s_job_rows, total = s_job_total;
        const int na = (rows + 4 * R - 1) / (4 * R), nb = (rows + R - 1) / R;
        const unsigned chunk = (unsigned)(R * N * 8), buf = smem_u32(smem_raw + L.fill);
        int next = s_job_next;
        for (int bt = 0; bt < batches && next < total; bt++, next += BIG_FILL_LANES) {
            const int op = next + lane;
            if (lane < BIG_FILL_LANES && op < total) {
                int arr, r0, cnt, width;
                if (op < 2 * na) { arr = op >= na; r0 = (op - arr * na) * 4 * R; cnt = min(4 * R, rows - r0); width = 2; }
                else { const int o2 = op - 2 * na; arr = 2 + o2 / nb; r0 = (o2 - (arr - 2) * nb) * R; cnt = min(R, rows - r0); width = 8; }
                unsigned char* base = s_job_ptr[arr];
                if (base) bulk_store(base + (size_t)r0 * N * width, buf + (arr < 2 ? 0u : (unsigned)(arr - 1) * chunk), (unsigned)(cnt * N * width));
            }
            bulk_commit();
        }
        __syncwarp();
        if (lane == 0) s_job_next = next;
        __syncwarp();
    };
    if (tid == 0) { s_job_next = 0; s_job_total = 0; s_job_rows = 0; }

    for (;;) {
        if (tid == 0) {
            const unsigned at = atomicAdd(counter, 1u);
            s_b = at < (unsigned)B ? (order ? order[at] : (int)at) : B;
            s_flags = 0;
        }
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
        int64_t* colmax = colsum + N;
        for (int i = tid; i < N; i += NT) { colsum[i] = 0; colmax[i] = 0; rowsum[i] = 0; send_acc[i] = 0; recv_acc[i] = 0; colmap[i] = 0xFF; }
        if (tid == 0) { s_nhot = 0; s_nbig = 0; }
        for (int e = tid; e < G * G; e += NT) Dhat[e] = 0;
        __syncthreads();
        int flags = 0;
        // One warp per source group.  A row is read 32 columns per load instruction, its loads (up to eight) all in
        // flight at once; row sums need one warp reduction per row, column figures are carried over the group's four rows.
        const int64_t gmask = (kp.granule & (kp.granule - 1)) == 0 ? kp.granule - 1 : -1;     // power-of-two granule
        for (int a = warp; a < G; a += n_warps) {
            int64_t colv[8], colm[8];
#pragma unroll
            for (int m = 0; m < 8; m++) { colv[m] = 0; colm[m] = 0; }
#pragma unroll 1
            for (int i4 = 0; i4 < 4; i4++) {
                const int i = a * 4 + i4;
                const int64_t* row = D + (size_t)i * N;
                int64_t v[8];
#pragma unroll
                for (int m = 0; m < 8; m++) v[m] = m * 32 + lane < N ? row[m * 32 + lane] : 0;
                int64_t rsum = 0;
#pragma unroll
                for (int m = 0; m < 8; m++) {
                    const int64_t x = v[m];
                    if (x < 0) flags |= VP_ST_NEGATIVE;
                    else if (x >= VP_ENTRY_LIMIT) flags |= VP_ST_OVERFLOW_RISK;
                    else {
                        if (m * 32 + lane == i && x != 0) flags |= VP_ST_DIAG_NONZERO;
                        if (gmask >= 0 ? (x & gmask) != 0 : big_not_multiple(x, kp.granule)) flags |= VP_ST_NOT_GRANULE;
                    }
                    rsum += x;
                    colv[m] += x;
                    colm[m] = max_v(colm[m], x);
                }
                rsum = warp_sum_i64(rsum);
                if (lane == 0) rowsum[i] = rsum;             // (rows of this group belong to this warp alone)
            }
#pragma unroll
            for (int m = 0; m < 8; m++) {
                const int j = m * 32 + lane;
                if (j < N) {
                    atomicAdd((unsigned long long*)&colsum[j], (unsigned long long)colv[m]);
                    atomicMax((long long*)&colmax[j], (long long)colm[m]);
                    atomicAdd((unsigned long long*)&Dhat[a * G + (j >> 2)], (unsigned long long)colv[m]);
                }
            }
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
                // 16-bit credits need capacities below 2^16 granules, hot columns capacities below 2^22 (four credits and
                // a tag share 32 bits); the 32-bit table needs fewer than 2^32 granules in all
                const bool fits = kp.granule >= 256 && t / kp.granule < ((int64_t)1 << 32);
                s_mode = !fits ? 0 : (cap_max / kp.granule < big_floor ? 1 : (cap_max / kp.granule < ((int64_t)1 << 22) ? 2 : 0));
                s_tau = tq; s_left = t / kp.granule;
            }
            __syncthreads();
            tau = s_tau;
            if (s_mode == 2) {                               // hot columns: those with a cell of 65,535 granules or more
                for (int j = tid; j < N; j += NT)
                    if (colmax[j] / kp.granule >= 65535) {
                        const int at = atomicAdd(&s_nhot, 1);
                        if (at < BIG_HOT_MAX) colmap[j] = (uint8_t)at;
                    }
                __syncthreads();
                if (tid == 0 && s_nhot > BIG_HOT_MAX) s_mode = 0;
                __syncthreads();
            }
            deferred = s_mode == 0;
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
            // ---- pass 2 over D: the residual in granules as 16-bit cells (big cells through the side list)
            const bool hot_mode = s_mode == 2;
            if (DEC && tid < 2 * dec_n) red[tid] = 0;        // the units' best keys (see step A)
            const int gshift = gmask >= 0 ? 63 - __clzll(kp.granule) : -1;
#pragma unroll 1
            for (int e0 = tid; e0 < N * N; e0 += 4 * NT) {       // four loads in flight per thread
                int64_t raw[4];
#pragma unroll
                for (int u = 0; u < 4; u++) raw[u] = e0 + u * NT < N * N ? D[e0 + u * NT] : 0;
#pragma unroll 1
                for (int u = 0; u < 4; u++) {
                const int e = e0 + u * NT;
                if (e >= N * N) break;
                const uint32_t v = gshift >= 0 ? (uint32_t)(raw[u] >> gshift) : big_div_granule(raw[u], kp.granule);
                const int i = e / N, j = e - i * N;
                if (!hot_mode) {
                    uint32_t code = v;
                    if (v >= (uint32_t)big_floor) {             // a big cell: exact value in the side list, its index in the matrix
                        const int at = atomicAdd(&s_nbig, 1);
                        code = (uint32_t)big_floor + (uint32_t)min_v(at, big_max - 1);
                        if (at < big_max) side[at] = v;
                    }
                    Cs[i * CS + j] = (uint16_t)code;
                } else {                                     // exact: 32 bits in a hot column, below 65,535 elsewhere
                    Cs[i * CS + j] = (uint16_t)v;
                    if (colmap[j] != 0xFF) Hi[(int)colmap[j] * N + i] = (uint16_t)(v >> 16);
                }
                }
            }
            __syncthreads();
            if (s_nbig > big_max) {                          // more big cells than the side list holds: the general kernel's
                if (tid == 0) todo[atomicAdd(counter + 1, 1u)] = b;
                __syncthreads();
                continue;
            }
            int64_t left = s_left;
            int last_s = -1;                                 // shape chosen in the last iteration
            for (int s = tid; s < dc.n_shapes && !DEC; s += NT) bnd[s] = 0xffffffffu;
            int f_cached = -1;                               // family whose tables this lane still holds (first task only)
            uint32_t c_co = 0;
            uint2 c_fi = make_uint2(0u, 0u);
            VP_TICK(0);
            // Emit rows through shared memory: the five rows of an activation are staged there, and the upper half of the
            // warps, which has no task in Step 2 as a rule, copies them out during Step 2 of the next iteration.  (Plain
            // stores to global memory by the emitting warps, just before a CTA-wide barrier, made every iteration wait
            // for them: 6 % of the run time.)
            // first warp with neither a task nor a slot to emit
            const int copy_warp0 = max(tpw2 ? (kp.n_start + 1) >> 1 : kp.n_start * W, (N + 31) >> 5);
            const bool rows_async = N % 8 == 0 && copy_warp0 < n_warps &&
                (((uintptr_t)lane_dst_b | (uintptr_t)lane_inst_b | (uintptr_t)lane_bytes_b | (uintptr_t)send_off_b |
                  (uintptr_t)(recv_off_b ? recv_off_b : send_off_b)) & 15) == 0;
            int copied = 0;                                  // activations copied out (upper warps)
            auto copy_row = [&](int kk) {
                const unsigned char* sb = smem_raw + L.emit;
                for (int e = tid - copy_warp0 * 32; e < 28 * N / 16; e += NT - copy_warp0 * 32) {
                    const int at = e * 16;
                    unsigned char* dst;
                    if (at < 4 * N) dst = at < 2 * N ? (unsigned char*)(lane_dst_b + (size_t)kk * N) + at
                                                     : (unsigned char*)(lane_inst_b + (size_t)kk * N) + (at - 2 * N);
                    else if (at < 12 * N) dst = (unsigned char*)(lane_bytes_b + (size_t)kk * N) + (at - 4 * N);
                    else if (at < 20 * N) dst = (unsigned char*)(send_off_b + (size_t)(kk + 1) * N) + (at - 12 * N);
                    else dst = recv_off_b ? (unsigned char*)(recv_off_b + (size_t)(kk + 1) * N) + (at - 20 * N) : nullptr;
                    if (dst) *(uint4*)dst = *(const uint4*)(sb + at);
                }
            };

            for (;;) {
                if (left == 0) break;
                if (k == kp.k_max) { st |= VP_ST_STEP_LIMIT; break; }
                // (A) Eq. (6).  Row scores first: at most max_row_terms products each, stored shifted left by 16 bits.
                if (!DEC) {
                    for (int p = tid; p < dc.n_patterns; p += NT) {
                        uint64_t v = 0;
#pragma unroll 1
                        for (int t = 0; t < dc.max_row_terms; t++) {
                            const uint32_t tw = pat[p * dc.max_row_terms + t];
                            v += (uint64_t)tbl[tw & 0xffffu] * (tw >> 16);
                        }
                        rs[p] = v << 16;
                    }
                    __syncthreads();
                }
                // A score is below 2^34 (g x fewer than 2^32 granules) and there are fewer than 2^16 shapes, so
                // key = score << 16 | (65535 - shape) orders by score first and lower shape index second: the first
                // maximum of Eq. (6) is a plain maximum of keys.
                //
                // Lazy evaluation.  Table entries only ever shrink while a matrix is decomposed, so the score a shape had
                // when it was last computed bounds its score now.  The shape chosen last time, scored again, is a lower
                // bound on the maximum; a shape whose old score lies below that bound (both compared after dropping their
                // two lowest bits, so that they fit 32 bits) cannot be the maximum, nor tie with it, and is skipped.
                auto score_key = [&](int s) {
                    uint64_t key = (uint64_t)(65535 - s);
                    for (int w = 0; w < L.pat_words; w++) {
                        const uint32_t pw = spat[w * ns_pad + s];              // two byte offsets into the row scores
                        key += *(const uint64_t*)((const char*)rs + (pw & 0xffffu));
                        if (2 * w + 1 < S) key += *(const uint64_t*)((const char*)rs + (pw >> 16));
                    }
                    return key;
                };
                uint64_t best = 0;
                if (DEC) {
                    // Class by class (two rails).  A shape is a first row p0 and a second row p1 from the list of p0's
                    // class, and its index grows with p0's place in shape order first, p1's place in the list second.
                    // So within a class the first maximum is (first maximal p0, first maximal p1 of the list): two
                    // independent maxima.  One warp per chunk of 32 rows: each lane scores its row from the table
                    // (at most max_row_terms products) and the chunk's best key score << 16 | (65535 - tie-break word) is kept
                    // (the word is the run start for a first row, the place in the list for a second row: both grow in shape order).
                    const int n_chunks = (int)decs[0], stride = (int)decs[1];
                    for (int c = warp; c < n_chunks; c += n_warps) {
                        const uint32_t* ent = decs + decs[2] + (size_t)(c * 32 + lane) * stride;
                        uint64_t v = 0;
#pragma unroll 3
                        for (int t = 0; t < stride - 1; t++) {
                            const uint32_t tw = ent[t];
                            v += (uint64_t)tbl[tw & 0xffffu] * (tw >> 16);
                        }
                        const uint32_t meta = ent[stride - 1];
                        const uint64_t key = big_warp_max64(meta == 0xffffffffu ? 0ull : (v << 16 | (uint64_t)(65535u - (meta & 0xffffu))));
                        if (lane == 0) atomicMax((unsigned long long*)&red[decs[3 + 2 * dec_n + 1 + c]], (unsigned long long)key);
                    }
                } else {
                    uint32_t floor32 = 0;
                    if (last_s >= 0) {
                        best = score_key(last_s);                              // (the same in every thread)
                        floor32 = (uint32_t)(best >> 18);
                    }
#pragma unroll 1
                    for (int s = tid; s < dc.n_shapes; s += NT) {
                        if (bnd[s] < floor32) continue;
                        const uint64_t key = score_key(s);
                        bnd[s] = (uint32_t)(key >> 18);
                        best = max_v(best, key);
                    }
                    best = big_warp_max64(best);
                    if (lane == 0) red[warp] = (int64_t)best;
                }
                __syncthreads();
                uint64_t bkey;
                if (DEC) {                                     // the classes' candidates: largest score, lowest shape
                    uint64_t cand = 0;
                    if (lane < dec_n) {                          // (red[unit]: the best key of the unit's chunks)
                        const uint64_t k0 = (uint64_t)red[2 * lane], k1 = (uint64_t)red[2 * lane + 1];
                        const uint32_t shape = (65535u - (uint32_t)(k0 & 0xffffu)) + (65535u - (uint32_t)(k1 & 0xffffu));   // run start + place
                        cand = ((k0 >> 16) + (k1 >> 16)) << 16 | (uint64_t)(65535u - shape);
                    }
                    bkey = big_warp_max64(cand);
                } else {
                    bkey = big_warp_max64(lane < n_warps ? (uint64_t)red[lane] : 0ull);
                }
                if ((bkey >> 16) == 0) { st |= VP_ST_UNCOVERED; break; }
                const int best_s = 65535 - (int)(bkey & 0xffffu);
                last_s = best_s;
                const int f0 = (int)bucket[best_s], H = (int)bucket[best_s + 1] - f0;
                const int n_tasks = H * kp.n_start;
                VP_TICK(1);

                if (W == 2 && warp == FILL_WARP && s_job_next < s_job_total) fill_step(1);   // (this warp has no task as a rule)
                if (rows_async && warp >= copy_warp0 && copied < k) copy_row(copied++);      // the last activation's rows

                // (B) MultiStartAA: W warps per (family, start), one lane per rank group
                const int sub = W == 2 ? (warp & 1) : 0, wgroup = W == 2 ? (warp >> 1) : warp;
                const int a = sub * 32 + lane;                   // this lane's group: source group, then destination group
                const bool active = a < G;
                auto task_sync = [&]() {
                    if (W == 2) asm volatile("bar.sync %0, 64;" ::"r"(1 + wgroup) : "memory");
                    else __syncwarp();
                };
                if (tpw2) {
                    // Up to sixteen groups: two tasks share a warp, sixteen lanes each (half the warps then carry Step 2 and
                    // half the instructions are issued for it).  A task that ends is switched off lane by lane; votes and
                    // sums run over the task's half of the warp.
                    const int half = lane >> 4, a2 = lane & 15;
                    const unsigned hmask = half ? 0xffff0000u : 0x0000ffffu;
                    for (int task0 = warp * 2; task0 < n_tasks; task0 += n_warps * 2) {
                        const bool has = task0 + half < n_tasks && a2 < G;
                        const int task = min(task0 + half, n_tasks - 1);
                        const int h = ns_shift >= 0 ? task >> ns_shift : task / kp.n_start, f = f0 + h, t = task - h * kp.n_start;
                        uint8_t* srcb = bind_src + (size_t)task * N;
                        uint8_t* dstb = bind_dst + (size_t)task * N;
                        const int ag = a2 < G ? a2 : 0;
                        uint32_t cap_out[4], cap_in[4];
                        int rq[4], cls_in[4];
                        uint32_t my_dst = 0, my_src = 0;
                        uint32_t hot_in = 0xffffffffu;
                        if (hot_mode && has) hot_in = *((const uint32_t*)colmap + a2);
                        {
                            const uint32_t co = __ldg((const uint32_t*)(dc.fam_cls + (size_t)f * N) + ag);
                            const uint2 fi = __ldg((const uint2*)(dc.fam_in + (size_t)f * N) + ag);
                            if (t == 0 && has) {                  // the family's slot words, parked for step (D)
                                const uint4 sw = __ldg((const uint4*)(dc.fam_slot + (size_t)f * N) + a2);
                                *((uint4*)(slotw + h * N) + a2) = sw;
                            }
                            const uint32_t fw[4] = {fi.x & 0xffffu, fi.x >> 16, fi.y & 0xffffu, fi.y >> 16};
#pragma unroll
                            for (int q = 0; q < 4; q++) {
                                cap_out[q] = s_cap[(co >> (8 * q)) & 0xffu];
                                rq[q] = (int)(fw[q] & 0xffu);
                                cls_in[q] = (int)(fw[q] >> 8);
                                cap_in[q] = s_cap[cls_in[q]];
                                const uint32_t d = (uint32_t)(a2 * 4 + ((q + t) & 3));
                                if (has) dstb[rq[q]] = (uint8_t)d;
                                my_dst |= d << (8 * q);
                            }
                        }
                        __syncwarp();
                        int64_t F_old = -1, F_new = -1;
                        bool alive = has;
                        for (int sweep = 0; sweep < kp.i_aa && __any_sync(0xffffffffu, alive); sweep++) {
                            bool moved = false;
                            if (alive) {                          // source half
                                const uint32_t d4 = *((const uint32_t*)dstb + a2);
                                uint32_t v[4][4];
#pragma unroll
                                for (int q = 0; q < 4; q++) {
                                    const uint16_t* colp = Cs + (a2 * 4) * CS + ((d4 >> (8 * q)) & 0xffu);
#pragma unroll
                                    for (int i = 0; i < 4; i++) v[i][q] = min_v((uint32_t)colp[i * CS], cap_out[q]) * 256u + big_tag(i, q);
                                }
                                if (hot_mode) {
#pragma unroll
                                    for (int q = 0; q < 4; q++) {
                                        const int dq = (int)((d4 >> (8 * q)) & 0xffu), hc = colmap[dq];
                                        if (hc != 0xFF) {
#pragma unroll
                                            for (int i = 0; i < 4; i++) {
                                                const uint32_t val = (uint32_t)Cs[(a2 * 4 + i) * CS + dq] | (uint32_t)Hi[hc * N + a2 * 4 + i] << 16;
                                                v[i][q] = min_v(val, cap_out[q]) * 256u + big_tag(i, q);
                                            }
                                        }
                                    }
                                }
                                const uint32_t pb = ~big_best_key(v) & 255u;
                                const uint32_t word = (uint32_t)(a2 * 4) * 0x01010101u +
                                                      (((pb >> 6) & 3u) | (((pb >> 4) & 3u) << 8) | (((pb >> 2) & 3u) << 16) | ((pb & 3u) << 24));
                                moved = sweep == 0 || word != my_src;
                                my_src = word;
                                *((uint32_t*)srcb + a2) = word;
                            }
                            __syncwarp();
                            // no source binding of the task moved: the destination half would repeat itself (see below)
                            const bool any_moved = __any_sync(hmask, moved);
                            if (alive && !any_moved) {
                                if (a2 == 0) n_sweeps++;
                                F_new = F_old;
                                alive = false;
                            }
                            uint32_t part = 0;
                            moved = false;
                            if (alive) {                          // destination half
                                uint32_t v[4][4];
#pragma unroll
                                for (int q = 0; q < 4; q++) {
                                    const uint32_t* rowp = (const uint32_t*)(Cs + (int)srcb[rq[q]] * CS + a2 * 4);
                                    const uint32_t c2 = min_v(cap_in[q], 65535u) * 0x00010001u;
                                    const uint32_t lo = __vminu2(rowp[0], c2), hi = __vminu2(rowp[1], c2);
                                    v[0][q] = __byte_perm(lo, big_tag(0, q), 0x5104);
                                    v[1][q] = __byte_perm(lo, big_tag(1, q), 0x5324);
                                    v[2][q] = __byte_perm(hi, big_tag(2, q), 0x5104);
                                    v[3][q] = __byte_perm(hi, big_tag(3, q), 0x5324);
                                }
                                if (hot_in != 0xffffffffu) {
#pragma unroll
                                    for (int j = 0; j < 4; j++) {
                                        const int hc = (int)((hot_in >> (8 * j)) & 0xffu);
                                        if (hc != 0xFF) {
#pragma unroll
                                            for (int q = 0; q < 4; q++) {
                                                const int sq = srcb[rq[q]];
                                                const uint32_t val = (uint32_t)Cs[sq * CS + a2 * 4 + j] | (uint32_t)Hi[hc * N + sq] << 16;
                                                v[j][q] = min_v(val, cap_in[q]) * 256u + big_tag(j, q);
                                            }
                                        }
                                    }
                                }
                                const uint32_t key = big_best_key(v);
                                const uint32_t pb = ~key & 255u;
                                part = key >> 8;
                                uint32_t word = 0;
#pragma unroll
                                for (int q = 0; q < 4; q++) {
                                    const uint32_t d = (uint32_t)(a2 * 4) + ((pb >> (6 - 2 * q)) & 3u);
                                    dstb[rq[q]] = (uint8_t)d;
                                    word |= d << (8 * q);
                                }
                                moved = word != my_dst;
                                my_dst = word;
                            }
                            const uint32_t fm = __reduce_add_sync(hmask, part) << 1 | (uint32_t)__any_sync(hmask, moved);
                            __syncwarp();
                            if (alive) {
                                F_new = (int64_t)(fm >> 1);
                                if (a2 == 0) n_sweeps++;
                                if (F_new <= F_old) alive = false;
                                else {
                                    F_old = F_new;
                                    if (!(fm & 1u) && sweep + 1 < kp.i_aa) {   // no destination binding moved: the next sweep would repeat this one
                                        if (a2 == 0) n_sweeps++;
                                        alive = false;
                                    }
                                }
                            }
                        }
                        int64_t tmax = 0;
                        if (H > 1) {                              // Eq. (9), (10) over the task's sixteen lanes
                            if (has) {
#pragma unroll 1
                                for (int q = 0; q < 4; q++) {
                                    const int sq = srcb[rq[q]], dq = dstb[rq[q]];
                                    uint32_t val = Cs[sq * CS + dq];
                                    if (hot_mode && colmap[dq] != 0xFF) val |= (uint32_t)Hi[(int)colmap[dq] * N + sq] << 16;
                                    tmax = max_v(tmax, (int64_t)min_v(val, cap_in[q]) * s_tscale[cls_in[q]]);
                                }
                            }
#pragma unroll
                            for (int o = 8; o; o >>= 1) tmax = max_v(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
                        }
                        if (has && a2 == 0) {
                            n_tasks_done++;
                            task_f[task] = F_new;
                            task_den[task] = F_new > 0 ? kp.lambda_ns * dc.W + tmax : 1;
                        }
                    }
                } else
                for (int task = wgroup; task < n_tasks; task += n_warps / W) {
                    const int h = ns_shift >= 0 ? task >> ns_shift : task / kp.n_start, f = f0 + h, t = task - h * kp.n_start;
                    uint8_t* srcb = bind_src + (size_t)task * N;
                    uint8_t* dstb = bind_dst + (size_t)task * N;
                    int64_t* pair = pairs + wgroup * 8;
                    uint32_t cap_out[4], cap_in[4];
                    int rq[4], cls_in[4];
                    uint32_t my_dst = 0, my_src = 0;             // what this lane last wrote to the two bindings
                    uint32_t hot_in = 0xffffffffu;               // hot-column indices of this group's four ranks (0xFF = none)
                    if (hot_mode && active) hot_in = *((const uint32_t*)colmap + a);
                    if (active) {
                        uint32_t co;
                        uint2 fi;
                        const bool first = task == wgroup;
                        if (first && f == f_cached) {             // the same family as in the last iteration: tables still held
                            co = c_co; fi = c_fi;
                        } else {
                            co = __ldg((const uint32_t*)(dc.fam_cls + (size_t)f * N) + a);
                            fi = __ldg((const uint2*)(dc.fam_in + (size_t)f * N) + a);
                            if (t == 0) {                         // the family's slot words, parked for step (D)
                                const uint4 sw = __ldg((const uint4*)(dc.fam_slot + (size_t)f * N) + a);
                                *((uint4*)(slotw + h * N) + a) = sw;
                            }
                            if (first) { c_co = co; c_fi = fi; }
                        }
                        if (first) f_cached = f;
                        const uint32_t fw[4] = {fi.x & 0xffffu, fi.x >> 16, fi.y & 0xffffu, fi.y >> 16};
#pragma unroll
                        for (int q = 0; q < 4; q++) {
                            cap_out[q] = s_cap[(co >> (8 * q)) & 0xffu];
                            rq[q] = (int)(fw[q] & 0xffu);
                            cls_in[q] = (int)(fw[q] >> 8);
                            cap_in[q] = s_cap[cls_in[q]];
                            const uint32_t d = (uint32_t)(a * 4 + ((q + t) & 3));   // start t rotates the in-slots
                            dstb[rq[q]] = (uint8_t)d;
                            my_dst |= d << (8 * q);
                        }
                    }
                    task_sync();
                    int64_t F_old = -1, F_new = -1;
                    for (int sweep = 0; sweep < kp.i_aa; sweep++) {
                        bool moved = false;
                        if (active) {                             // source half: one exact assignment per source group
                            const uint32_t d4 = *((const uint32_t*)dstb + a);
                            uint32_t v[4][4];
#pragma unroll
                            for (int q = 0; q < 4; q++) {
                                const uint16_t* colp = Cs + (a * 4) * CS + ((d4 >> (8 * q)) & 0xffu);
#pragma unroll
                                for (int i = 0; i < 4; i++) v[i][q] = min_v((uint32_t)colp[i * CS], cap_out[q]) * 256u + big_tag(i, q);
                            }
                            if (hot_mode) {                       // out-slots bound to a hot column: exact 32-bit cells
#pragma unroll
                                for (int q = 0; q < 4; q++) {
                                    const int dq = (int)((d4 >> (8 * q)) & 0xffu), hc = colmap[dq];
                                    if (hc != 0xFF) {
#pragma unroll
                                        for (int i = 0; i < 4; i++) {
                                            const uint32_t val = (uint32_t)Cs[(a * 4 + i) * CS + dq] | (uint32_t)Hi[hc * N + a * 4 + i] << 16;
                                            v[i][q] = min_v(val, cap_out[q]) * 256u + big_tag(i, q);
                                        }
                                    }
                                }
                            }
                            const uint32_t pb = ~big_best_key(v) & 255u;
                            const uint32_t word = (uint32_t)(a * 4) * 0x01010101u +
                                                  (((pb >> 6) & 3u) | (((pb >> 4) & 3u) << 8) | (((pb >> 2) & 3u) << 16) | ((pb & 3u) << 24));
                            moved = sweep == 0 || word != my_src;
                            my_src = word;
                            *((uint32_t*)srcb + a) = word;
                        }
                        // If no source binding moved, the destination half would see what it saw last sweep and return the
                        // same binding and the same F: the run ends here exactly as it would after computing that.
                        bool any_moved = __any_sync(0xffffffffu, moved);
                        if (W == 2) {
                            if (lane == 0) ((int32_t*)(pair + 6))[sub] = any_moved;
                            task_sync();
                            any_moved = (((const int32_t*)(pair + 6))[0] | ((const int32_t*)(pair + 6))[1]) != 0;
                        } else {
                            __syncwarp();
                        }
                        if (!any_moved) {
                            if (sub == 0 && lane == 0) n_sweeps++;
                            F_new = F_old;
                            break;
                        }
                        uint32_t part = 0;
                        moved = false;
                        if (active) {                             // destination half
                            uint32_t v[4][4];
#pragma unroll
                            for (int q = 0; q < 4; q++) {
                                const uint32_t* rowp = (const uint32_t*)(Cs + (int)srcb[rq[q]] * CS + a * 4);
                                const uint32_t c2 = min_v(cap_in[q], 65535u) * 0x00010001u;   // the capacity in both halves
                                const uint32_t lo = __vminu2(rowp[0], c2), hi = __vminu2(rowp[1], c2);
                                v[0][q] = __byte_perm(lo, big_tag(0, q), 0x5104);  // (low half) << 8 | tag
                                v[1][q] = __byte_perm(lo, big_tag(1, q), 0x5324);  // (high half) << 8 | tag
                                v[2][q] = __byte_perm(hi, big_tag(2, q), 0x5104);
                                v[3][q] = __byte_perm(hi, big_tag(3, q), 0x5324);
                            }
                            if (hot_in != 0xffffffffu) {          // some rank of this group is a hot column: exact 32-bit cells
#pragma unroll
                                for (int j = 0; j < 4; j++) {
                                    const int hc = (int)((hot_in >> (8 * j)) & 0xffu);
                                    if (hc != 0xFF) {
#pragma unroll
                                        for (int q = 0; q < 4; q++) {
                                            const int sq = srcb[rq[q]];
                                            const uint32_t val = (uint32_t)Cs[sq * CS + a * 4 + j] | (uint32_t)Hi[hc * N + sq] << 16;
                                            v[j][q] = min_v(val, cap_in[q]) * 256u + big_tag(j, q);
                                        }
                                    }
                                }
                            }
                            const uint32_t key = big_best_key(v);
                            const uint32_t pb = ~key & 255u;
                            part = key >> 8;
                            uint32_t word = 0;
#pragma unroll
                            for (int q = 0; q < 4; q++) {
                                const uint32_t d = (uint32_t)(a * 4) + ((pb >> (6 - 2 * q)) & 3u);
                                dstb[rq[q]] = (uint8_t)d;
                                word |= d << (8 * q);
                            }
                            moved = word != my_dst;
                            my_dst = word;
                        }
                        // Eq. (8): at most 2^8 lanes of less than 2^18 granules.  The low bit carries "a destination
                        // binding moved": if none did, the next sweep would be a repetition of this one (same sources, same
                        // destinations, same F) and would end the run, so it is counted and skipped.
                        uint32_t fm = __reduce_add_sync(0xffffffffu, part) << 1 | (uint32_t)__any_sync(0xffffffffu, moved);
                        if (W == 2) {
                            if (lane == 0) ((uint32_t*)(pair + (sweep & 1) * 2))[sub] = fm;
                            task_sync();
                            const uint32_t f0w = ((const uint32_t*)(pair + (sweep & 1) * 2))[0], f1w = ((const uint32_t*)(pair + (sweep & 1) * 2))[1];
                            fm = ((f0w >> 1) + (f1w >> 1)) << 1 | ((f0w | f1w) & 1u);
                        } else {
                            __syncwarp();
                        }
                        F_new = (int64_t)(fm >> 1);
                        if (sub == 0 && lane == 0) n_sweeps++;
                        if (F_new <= F_old) break;
                        F_old = F_new;
                        if (!(fm & 1u) && sweep + 1 < kp.i_aa) {
                            if (sub == 0 && lane == 0) n_sweeps++;
                            break;
                        }
                    }
                    // Eq. (9) volumes of the binding as it stands (the credit of every in-slot) and the slowest lane of
                    // Eq. (10): only needed when several families compete on utility
                    int64_t tmax = 0;
                    if (H > 1) {
                        tmax = big_slowest_lane(Cs, CS, Hi, colmap, N, hot_mode, srcb, dstb, rq, cap_in, cls_in, s_tscale, dc.n_classes, active);
                        if (W == 2) {
                            if (lane == 0) pair[4 + sub] = tmax;
                            task_sync();
                            tmax = max_v(pair[4], pair[5]);
                        }
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
                if (H == 1 && kp.n_start == 4) {                 // one family, four starts: best start, no utilities to compare
                    const int64_t f0v = task_f[0], f1v = task_f[1], f2v = task_f[2], f3v = task_f[3];
                    const int64_t m01 = max_v(f0v, f1v), m23 = max_v(f2v, f3v);
                    wF = max_v(m01, m23);
                    wtask = m01 >= m23 ? (f0v >= f1v ? 0 : 1) : (f2v >= f3v ? 2 : 3);
                } else if (H == 1) {
                    wtask = 0; wF = task_f[0];
                    for (int t = 1; t < kp.n_start; t++)
                        if (task_f[t] > wF) { wF = task_f[t]; wtask = t; }
                } else {
                    big_select_family(task_f, task_den, H, kp.n_start, lane, wtask, wF);
                }
                if (wF <= 0) { st |= VP_ST_NO_PROGRESS; break; }
                VP_TICK(3);

                // (D) emit activation k: volumes off the residual and off the score table, next offset row
                if (warp * 32 < N) {
                    const int h = ns_shift >= 0 ? wtask >> ns_shift : wtask / kp.n_start;
                    const uint32_t* slot = slotw + h * N;
                    const uint8_t* srcb = bind_src + (size_t)wtask * N;
                    const uint8_t* dstb = bind_dst + (size_t)wtask * N;
                    const size_t row = (size_t)k * N, orow = (size_t)(k + 1) * N;
                    for (int r = tid; r < N; r += NT) {
                        uint32_t x = 0;
                        {
                            const uint32_t w = slot[r];
                            const int i = srcb[r], j = dstb[r];
                            uint16_t* cell = Cs + i * CS + j;
                            uint32_t c = *cell;
                            uint16_t* hcell = nullptr;
                            if (hot_mode && colmap[j] != 0xFF) {  // a hot column: the exact 32-bit cell
                                hcell = Hi + (int)colmap[j] * N + i;
                                c |= (uint32_t)*hcell << 16;
                            }
                            x = min_v(s_cap[(w >> 24) & 0xf], c);
                            const bool busy = x > 0;
                            const int64_t bytes = (int64_t)x * kp.granule;
                            const int64_t sa = send_acc[i] + bytes, ra = recv_acc[j] + bytes;
                            send_acc[i] = sa;
                            recv_acc[j] = ra;
                            // (src and dst are permutations: every rank of every row is written once)
                            if (rows_async) {
                                unsigned char* sb = smem_raw + L.emit;
                                ((int16_t*)sb)[i] = busy ? (int16_t)j : (int16_t)-1;
                                ((uint16_t*)(sb + 2 * N))[i] = busy ? (uint16_t)(w & 0xffffu) : (uint16_t)0xFFFF;
                                ((int64_t*)(sb + 4 * N))[i] = bytes;
                                ((int64_t*)(sb + 12 * N))[i] = sa;
                                ((int64_t*)(sb + 20 * N))[j] = ra;
                            } else {
                                lane_dst_b[row + i] = busy ? (int16_t)j : (int16_t)-1;
                                lane_inst_b[row + i] = busy ? (uint16_t)(w & 0xffffu) : (uint16_t)0xFFFF;
                                lane_bytes_b[row + i] = bytes;
                                send_off_b[orow + i] = sa;
                                if (recv_off_b) recv_off_b[orow + j] = ra;
                            }
                            if (busy) {
                                if (hcell) {
                                    *cell = (uint16_t)(c - x);
                                    *hcell = (uint16_t)((c - x) >> 16);
                                } else if (c >= (uint32_t)big_floor && !hot_mode) {   // a big cell: exact value in the side list
                                    const uint32_t now = side[c - big_floor] - x;
                                    if (now >= (uint32_t)big_floor) side[c - big_floor] = now;
                                    else *cell = (uint16_t)now;   // (an ordinary cell from here on)
                                } else {
                                    *cell = (uint16_t)(c - x);
                                }
                                // the volume leaves the table entry of its group pair
                                const int ga = i >> 2, gd = j >> 2;
                                int delta = (int)gnode[gd] - (int)gnode[ga];
                                if (delta < 0) delta += P;
                                atomicSub(&tbl[(delta * S + gnode[G + ga]) * S + gnode[G + gd]], x);
                            }
                        }
                    }
                    if (tid == 0) chan_id_b[k] = f0 + h;
                    if (DEC && tid < 2 * dec_n) red[tid] = 0;    // the units' best keys start the next iteration at zero
                }
                left -= wF;
                k++;
                __syncthreads();
                VP_TICK(4);
            }
            if (rows_async && warp >= copy_warp0 && copied < k) copy_row(copied++);       // the last activation of the matrix
        }
        __syncthreads();
        // ---- idle rows beyond n_steps; offset rows repeat the totals
        const bool off_aligned = (((uintptr_t)send_off_b | (uintptr_t)(recv_off_b ? recv_off_b : send_off_b)) & 15) == 0;
        const bool lane_aligned = (((uintptr_t)lane_dst_b | (uintptr_t)lane_inst_b | (uintptr_t)lane_bytes_b) & 15) == 0 && N % 8 == 0;
        if (W == 2 && L.fill_rows > 0 && off_aligned && lane_aligned) {
            // Bulk asynchronous copies out of the fill buffers, issued a batch at a time while the next matrices are
            // decomposed.  First the copies still pending from the last matrix: they read the totals that change now.
            if (warp == FILL_WARP) {
                fill_step(0x7fffffff);
                bulk_wait_read<0>();
            }
            __syncthreads();
            const unsigned chunk = (unsigned)(L.fill_rows * N * 8);
            unsigned char* buf = smem_raw + L.fill;
            for (unsigned e = tid; e < chunk / 16; e += NT) {
                const int i2 = (int)(e % (unsigned)(N / 2));
                ((longlong2*)(buf + 2 * chunk))[e] = ((const longlong2*)send_acc)[i2];
                ((longlong2*)(buf + 3 * chunk))[e] = ((const longlong2*)recv_acc)[i2];
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            if (tid == 0) {
                const int rows = kp.k_max - k, R = L.fill_rows;
                s_job_ptr[0] = (unsigned char*)(lane_dst_b + (size_t)k * N);
                s_job_ptr[1] = (unsigned char*)(lane_inst_b + (size_t)k * N);
                s_job_ptr[2] = (unsigned char*)(lane_bytes_b + (size_t)k * N);
                s_job_ptr[3] = (unsigned char*)(send_off_b + (size_t)(k + 1) * N);
                s_job_ptr[4] = recv_off_b ? (unsigned char*)(recv_off_b + (size_t)(k + 1) * N) : nullptr;
                s_job_rows = rows;
                s_job_next = 0;
                s_job_total = 2 * ((rows + 4 * R - 1) / (4 * R)) + 3 * ((rows + R - 1) / R);
            }
        } else {
            const size_t lo = (size_t)k * N, hi = (size_t)kp.k_max * N;
            big_fill_bytes((unsigned char*)lane_dst_b, lo * 2, hi * 2, 0xff, tid, NT);
            big_fill_bytes((unsigned char*)lane_inst_b, lo * 2, hi * 2, 0xff, tid, NT);
            big_fill_bytes((unsigned char*)lane_bytes_b, lo * 8, hi * 8, 0x00, tid, NT);
            if (off_aligned) {                               // N is a multiple of four: rows are whole 16-byte pairs
                const int half = N / 2;
                for (size_t e = lo / 2 + tid; e < hi / 2; e += NT) {
                    const int i2 = (int)(e % half);
                    ((longlong2*)(send_off_b + N))[e] = ((const longlong2*)send_acc)[i2];
                    if (recv_off_b) ((longlong2*)(recv_off_b + N))[e] = ((const longlong2*)recv_acc)[i2];
                }
            } else {
                for (size_t e = lo + tid; e < hi; e += NT) {
                    const int i = (int)(e % N);
                    send_off_b[N + e] = send_acc[i];
                    if (recv_off_b) recv_off_b[N + e] = recv_acc[i];
                }
            }
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
    if (W == 2 && warp == FILL_WARP) fill_step(0x7fffffff);     // what is left of the last fill
    bulk_wait_all();
    unsigned long long* stats = (unsigned long long*)(counter + 4);
    if (tid == 0 && n_act) atomicAdd(&stats[0], n_act);
    n_tasks_done = (unsigned long long)warp_sum_i64((int64_t)n_tasks_done);    // (counted by the first lane of every task)
    n_sweeps = (unsigned long long)warp_sum_i64((int64_t)n_sweeps);
    if (lane == 0 && n_tasks_done) { atomicAdd(&stats[1], n_tasks_done); atomicAdd(&stats[2], n_sweeps); }
#ifdef VP_PHASE_TIMING
    if (tid == 0) for (int i = 0; i < 6; i++) atomicAdd(&stats[3 + i], (unsigned long long)cnt.cyc[i]);
#endif
}

}  // namespace
