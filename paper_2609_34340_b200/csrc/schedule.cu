// vp_schedule_batch: Algorithm 2 (Section 4.2) for a batch of demand matrices.
//
// One CTA decomposes one matrix at a time (persistent CTAs pull matrix indices
// from a counter).  The residual demand D_rem lives in shared memory when
// N <= 64 and in an L2-resident workspace slot otherwise; the group sums D-hat
// are kept in shared memory and updated incrementally after every activation.
// The catalog (shape terms, per-family slot tables) is staged in shared memory
// once per CTA when it fits.
//
// Value type.  Every demand entry and every lane capacity is a multiple of the
// granule, so a matrix whose capacities are below 2^25 granules is decomposed
// in 32-bit granule units (credits, sums of four credits and a 5-bit
// permutation tag then fit one 32-bit key); other matrices run the same code
// on 64-bit byte values.  Both give the same plan.
//
// Per iteration, three block barriers:
//  (A) every thread scores shapes (Eq. 6) on fixed-stride term lists; a
//      (value, lowest index) arg-max by warp shuffles, then across warps through
//      shared memory, picks M*;
//  (B) every (family, start) pair of the bucket is one warp-level task that runs
//      the Alternating Algorithm (Eq. 7, 8).  For groups of four ranks a team
//      of 8 / 4 / 2 lanes shares one rank group: the 16 credits go to shared
//      memory, each lane evaluates its 3 / 6 / 12 of the 24 permutations, and a
//      shuffle reduction keeps the first maximum in lexicographic order.  With
//      more than 16 groups (or other group sizes) one lane owns a group and
//      enumerates all g! permutations in registers.  Then Evaluate (Eq. 9, 10);
//  (C) every warp redundantly picks the best start per family and the family of
//      largest utility (exact 128-bit cross-multiplication), no barrier;
//  (D) all threads emit the activation, subtract it from D_rem / D-hat and write
//      the next row of the running send / receive offsets.
#include <cuda_runtime.h>

#include <cstring>
#include <mutex>
#include <utility>

#include "bulk_copy.cuh"
#include "vp_internal.h"

namespace {

struct KParams {
    int64_t lambda_ns, granule;
    int k_target, n_start, i_aa, k_max;
    int max_tasks, stage_terms, stage_fam, stage_bucket, drem_in_smem;
    int incremental;          // keep the shape scores in shared memory and update them after every activation
};

struct Smem {                 // offsets (bytes) into dynamic shared memory
    int drem, dhat, tbl, send_acc, recv_acc, red, task_f, task_den, bind_src, bind_dst, cred, slotw, pair;
    int term, fam_in, fam_cls, bucket, score, inv, inv_ptr, delta, total;
};

__host__ __device__ inline int align16(int x) { return (x + 15) & ~15; }
__host__ __device__ inline int cred_bytes_per_warp(int lpg) { return lpg > 1 ? (32 / lpg) * 17 * 8 : 0; }

__host__ __device__ inline Smem smem_layout(const DevCat& dc, const KParams& kp, int n_warps, int lpg) {
    Smem L;
    int o = 0;
    L.drem = o;      o += kp.drem_in_smem ? dc.N * dc.N * 8 : 0;
    L.dhat = o;      o += dc.G * dc.G * 8;
    L.tbl = o;       o += dc.sym ? dc.tbl_size * 8 : 0;
    L.send_acc = o;  o += dc.N * 8;
    L.recv_acc = o;  o += dc.N * 8;
    L.red = o;       o += 64 * 8;
    L.pair = o;      o += 16 * 6 * 8;      // per warp pair: partial F (two sweeps in flight) and slowest-lane times
    L.task_f = o;    o += kp.max_tasks * 8;
    L.task_den = o;  o += kp.max_tasks * 8;
    L.cred = o;      o += n_warps * cred_bytes_per_warp(lpg);
    L.slotw = o;     o += dc.max_bucket * dc.N * 4;
    L.bind_src = o;  o += align16(kp.max_tasks * dc.N);
    L.bind_dst = o;  o += align16(kp.max_tasks * dc.N);
    o = align16(o);           // the staged arrays are filled by 16-byte bulk copies
    L.term = o;      o += kp.stage_terms ? ((dc.n_shapes + 31) & ~31) * dc.max_terms * 4 : 0;   // transposed, padded rows
    L.fam_in = o;    o += kp.stage_fam ? align16(dc.n_families * dc.N * 2) : 0;
    L.fam_cls = o;   o += kp.stage_fam ? align16(dc.n_families * dc.N) : 0;
    L.bucket = o;    o += kp.stage_bucket ? align16((dc.n_shapes + 1) * 4) : 0;
    L.score = o;     o += kp.incremental ? align16(dc.n_shapes * 8) : 0;
    L.inv = o;       o += kp.incremental ? align16(dc.n_terms * 4) : 0;
    L.inv_ptr = o;   o += kp.incremental ? align16((dc.tbl_size + 1) * 4) : 0;
    L.delta = o;     o += kp.incremental ? 32 * 8 + 32 * 4 : 0;
    L.total = o;
    return L;
}

template <typename T> __device__ __forceinline__ T min_v(T a, T b) { return a < b ? a : b; }
template <typename T> __device__ __forceinline__ T max_v(T a, T b) { return a > b ? a : b; }
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
__host__ __device__ constexpr unsigned long long perm4_word(int w) {  // packed permutations 8w .. 8w+7, one per byte
    unsigned long long x = 0;
    for (int k = 0; k < 8; k++) x |= (unsigned long long)perm_packed(4, w * 8 + k) << (8 * k);
    return x;
}
__device__ __forceinline__ unsigned perm4_packed_rt(int p) {
    constexpr unsigned long long W0 = perm4_word(0), W1 = perm4_word(1), W2 = perm4_word(2);
    const unsigned long long w = p < 8 ? W0 : (p < 16 ? W1 : W2);
    return (unsigned)(w >> (8 * (p & 7))) & 0xffu;
}

template <int GS, int P, int Q> struct PermAt { static constexpr int value = perm_entry(GS, P, Q); };
template <int GS, int P> struct PermPacked { static constexpr unsigned value = perm_packed(GS, P); };

template <int GS, typename V, int P, int... Q>
__device__ __forceinline__ V perm_value(const V (&c)[GS][GS], std::integer_sequence<int, Q...>) {
    return (c[PermAt<GS, P, Q>::value][Q] + ...);
}
template <int GS, typename V, int... P>
__device__ __forceinline__ V best_assignment_impl(const V (&c)[GS][GS], unsigned& bpk, std::integer_sequence<int, P...>) {
    V best = 0;
    bpk = PermPacked<GS, 0>::value;
    bool first = true;
    (([&] {
         const V v = perm_value<GS, V, P>(c, std::make_integer_sequence<int, GS>{});
         if (first || v > best) { best = v; bpk = PermPacked<GS, P>::value; first = false; }
     }()),
     ...);
    return best;
}
// Exact g x g assignment in registers: maximise sum_q c[phi(q)][q] over all g! permutations, enumerated
// in lexicographic order of (phi(0), ..., phi(g-1)); the first maximum wins.  Returns phi packed 2 bits each.
// Groups of four in 32-bit granule units take the subset dynamic programme instead (same winner, 28 operations).
template <int GS, typename V>
__device__ __forceinline__ V best_assignment(const V (&c)[GS][GS], unsigned& bpk) {
    if constexpr (GS == 4 && sizeof(V) == 4) {
        // credits below 2^22: (credit << 8 | tag) values, subset dynamic programme with add-max (see schedule_big.cuh)
        uint32_t v[4][4];
#pragma unroll
        for (int r = 0; r < 4; r++)
#pragma unroll
            for (int q = 0; q < 4; q++) v[r][q] = (uint32_t)c[r][q] * 256u + ((uint32_t)(3 - r) << (6 - 2 * q));
        auto am = [](uint32_t a, uint32_t b, uint32_t cc) { return __viaddmax_u32(a, b, cc); };
        const uint32_t b01 = am(v[0][0], v[1][1], v[1][0] + v[0][1]), b02 = am(v[0][0], v[2][1], v[2][0] + v[0][1]);
        const uint32_t b03 = am(v[0][0], v[3][1], v[3][0] + v[0][1]), b12 = am(v[1][0], v[2][1], v[2][0] + v[1][1]);
        const uint32_t b13 = am(v[1][0], v[3][1], v[3][0] + v[1][1]), b23 = am(v[2][0], v[3][1], v[3][0] + v[2][1]);
        const uint32_t c012 = am(b01, v[2][2], am(b02, v[1][2], b12 + v[0][2])), c013 = am(b01, v[3][2], am(b03, v[1][2], b13 + v[0][2]));
        const uint32_t c023 = am(b02, v[3][2], am(b03, v[2][2], b23 + v[0][2])), c123 = am(b12, v[3][2], am(b13, v[2][2], b23 + v[1][2]));
        const uint32_t key = am(c012, v[3][3], am(c013, v[2][3], am(c023, v[1][3], c123 + v[0][3])));
        const uint32_t pb = ~key & 255u;
        bpk = ((pb >> 6) & 3u) | ((pb >> 4) & 3u) << 2 | ((pb >> 2) & 3u) << 4 | (pb & 3u) << 6;
        return (V)(key >> 8);
    }
    return best_assignment_impl<GS, V>(c, bpk, std::make_integer_sequence<int, factorial(GS)>{});
}

__device__ __forceinline__ int64_t warp_sum_i64(int64_t v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int64_t warp_max_i64(int64_t v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = max_v(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// First maximum of (value, index) pairs over the warp by warp-reduce instructions: the maximum of the high
// words, then of the low words among the lanes that hold it, then the lowest index among those.
__device__ __forceinline__ void warp_argmax_first(int64_t& best, int& best_s) {
    const uint32_t hi = (uint32_t)((uint64_t)best >> 32), lo = (uint32_t)best;
    const uint32_t mhi = __reduce_max_sync(0xffffffffu, best < 0 ? 0u : hi);
    const bool in1 = best >= 0 && hi == mhi;
    const uint32_t mlo = __reduce_max_sync(0xffffffffu, in1 ? lo : 0u);
    const bool in2 = in1 && lo == mlo;
    const unsigned any = __ballot_sync(0xffffffffu, in2);
    const uint32_t ms = __reduce_min_sync(0xffffffffu, in2 ? (uint32_t)best_s : 0x7fffffffu);
    best = any ? (int64_t)(((uint64_t)mhi << 32) | mlo) : -1;
    best_s = (int)ms;
}

// f1/d1 > f2/d2, exactly, by 128-bit cross-multiplication (all four in [0, 2^63)).
__device__ __forceinline__ bool util_greater(int64_t f1, int64_t d1, int64_t f2, int64_t d2) {
    unsigned long long a = (unsigned long long)f1, b = (unsigned long long)d2;
    unsigned long long c = (unsigned long long)f2, d = (unsigned long long)d1;
    unsigned long long hi1 = __umul64hi(a, b), lo1 = a * b, hi2 = __umul64hi(c, d), lo2 = c * d;
    return hi1 > hi2 || (hi1 == hi2 && lo1 > lo2);
}

// Two lanes per group, 32-bit granule units: each lane copies the team's 4 x 4 credit tile into registers once
// (16 loads at fixed offsets instead of 48 indexed ones) and evaluates twelve permutations on pair sums
// (c[p0][0] + c[p1][1]) + (c[p2][2] + c[p3][3]), which the compiler shares between permutations: 30 additions
// instead of 36.  Both lanes run the same code on the permutations that start with row 0 or 1; lane 1 sees the
// rows rotated by two, so it covers the permutations that start with row 2 or 3, and tags each value with the
// real permutation (as a byte, see below) so that the first maximum still wins.
// A permutation as one byte with position 0 in the two highest bits: as a number this grows with the lexicographic
// order, so 255 - byte is a tag that makes "larger key" mean "larger sum, then earlier permutation", and the byte
// itself says which row goes to which position (no table needed to decode it).
__host__ __device__ constexpr unsigned perm_byte(int a, int b, int c2, int d) { return (unsigned)(a << 6 | b << 4 | c2 << 2 | d); }
template <int P, int ROT> struct RotByte {         // the permutation P with every row rotated by ROT
    static constexpr unsigned value = perm_byte((perm_entry(4, P, 0) + ROT) & 3, (perm_entry(4, P, 1) + ROT) & 3,
                                                (perm_entry(4, P, 2) + ROT) & 3, (perm_entry(4, P, 3) + ROT) & 3);
};
// row placed at position q by a permutation byte
__device__ __forceinline__ int perm_byte_at(unsigned b, int q) { return (int)((b >> (6 - 2 * q)) & 3u); }
template <int... P>
__device__ __forceinline__ uint32_t reg2_best_impl(const uint32_t (&c)[4][4], int tl, std::integer_sequence<int, P...>) {
    uint32_t key = 0;
    ((key = max_v(key, (((c[PermAt<4, P, 0>::value][0] + c[PermAt<4, P, 1>::value][1]) +
                         (c[PermAt<4, P, 2>::value][2] + c[PermAt<4, P, 3>::value][3])) << 8) +
                           (uint32_t)(tl ? 255 - RotByte<P, 2>::value : 255 - RotByte<P, 0>::value))),
     ...);
    return key;
}
__device__ __forceinline__ uint32_t team_best_reg2(const uint32_t* cred, int tl, unsigned& bpk) {
    uint32_t c[4][4];
#pragma unroll
    for (int r = 0; r < 4; r++) {
        const uint32_t* row = cred + ((r + 2 * tl) & 3) * 4;
#pragma unroll
        for (int q = 0; q < 4; q++) c[r][q] = row[q];
    }
    uint32_t key = reg2_best_impl(c, tl, std::make_integer_sequence<int, 12>{});
    key = max_v(key, __shfl_xor_sync(0xffffffffu, key, 1));
    bpk = ~key & 255u;
    return key >> 8;
}

// Eight lanes per group, 32-bit granule units.  Team lane tl evaluates the three permutations 3 tl .. 3 tl + 2.
// Seen through a relabelling of the rows that depends on the lane only -- row 0 -> tl / 2, the other three
// ascending for even lanes and descending for odd lanes -- these are always the permutations (0,1,2,3), (0,1,3,2)
// and (0,2,1,3): every lane runs the same straight-line code on eight credits at fixed offsets from four row
// pointers (instead of twelve indexed loads), shares the pair sums, and tags value P with the real permutation
// (255 - its byte, see perm_byte).
struct Reg8Lane {
    unsigned row[4];      // offset of relabelled row r in the tile, in credits
    uint32_t tag[3];      // 255 - byte of the real permutation behind P = 0, 1, 2
};
__device__ __forceinline__ Reg8Lane reg8_lane(int tl) {
    Reg8Lane L;
    const int a = tl >> 1, odd = tl & 1;
    const int rest0 = a == 0 ? 1 : 0, rest1 = a <= 1 ? 2 : 1, rest2 = a == 3 ? 2 : 3;    // the other rows, ascending
    L.row[0] = (unsigned)a * 4;
    L.row[1] = (unsigned)(odd ? rest2 : rest0) * 4;
    L.row[2] = (unsigned)rest1 * 4;
    L.row[3] = (unsigned)(odd ? rest0 : rest2) * 4;
    const int R0 = a, R1 = odd ? rest2 : rest0, R2 = rest1, R3 = odd ? rest0 : rest2;    // real rows behind 0, 1, 2, 3
    L.tag[0] = 255u - perm_byte(R0, R1, R2, R3);
    L.tag[1] = 255u - perm_byte(R0, R1, R3, R2);
    L.tag[2] = 255u - perm_byte(R0, R2, R1, R3);
    return L;
}
// key = max over the lane's three permutations of (sum << 8 | tag); cred points at the team's tile
__device__ __forceinline__ uint32_t reg8_key(const uint32_t* cred, const Reg8Lane& L) {
    const uint32_t *r0 = cred + L.row[0], *r1 = cred + L.row[1], *r2 = cred + L.row[2], *r3 = cred + L.row[3];
    const uint32_t c00 = r0[0], c11 = r1[1], c21 = r2[1], c12 = r1[2], c22 = r2[2], c32 = r3[2], c23 = r2[3], c33 = r3[3];
    const uint32_t a01 = c00 + c11;
    const uint32_t v0 = a01 + (c22 + c33), v1 = a01 + (c32 + c23), v2 = (c00 + c21) + (c12 + c33);
    return max_v(max_v((v0 << 8) + L.tag[0], (v1 << 8) + L.tag[1]), (v2 << 8) + L.tag[2]);
}

// Four lanes per group, 32-bit granule units.  Team lane tl evaluates the six permutations that start with row tl.
// With the rows rotated by tl these are the six permutations that start with row 0: every lane runs the same code on
// ten credits at fixed offsets and six pair sums, and tags value P with the real permutation (255 - its byte).
struct Reg4Lane {
    unsigned row[4];      // offset of rotated row r in the tile, in credits
    uint32_t tag[6];      // 255 - byte of the real permutation behind P = 0 .. 5
};
template <int... P>
__device__ __forceinline__ void reg4_tags(Reg4Lane& L, int tl, std::integer_sequence<int, P...>) {
    ((L.tag[P] = 255u - perm_byte(tl, (perm_entry(4, P, 1) + tl) & 3, (perm_entry(4, P, 2) + tl) & 3, (perm_entry(4, P, 3) + tl) & 3)),
     ...);
}
__device__ __forceinline__ Reg4Lane reg4_lane(int tl) {
    Reg4Lane L;
#pragma unroll
    for (int r = 0; r < 4; r++) L.row[r] = (unsigned)((r + tl) & 3) * 4;
    reg4_tags(L, tl, std::make_integer_sequence<int, 6>{});
    return L;
}
__device__ __forceinline__ uint32_t reg4_key(const uint32_t* cred, const Reg4Lane& L) {
    const uint32_t *r0 = cred + L.row[0], *r1 = cred + L.row[1], *r2 = cred + L.row[2], *r3 = cred + L.row[3];
    const uint32_t c00 = r0[0];
    const uint32_t a1 = c00 + r1[1], a2 = c00 + r2[1], a3 = c00 + r3[1];
    const uint32_t c12 = r1[2], c22 = r2[2], c32 = r3[2], c13 = r1[3], c23 = r2[3], c33 = r3[3];
    const uint32_t v0 = a1 + (c22 + c33), v1 = a1 + (c32 + c23), v2 = a2 + (c12 + c33), v3 = a2 + (c32 + c13),
                   v4 = a3 + (c12 + c23), v5 = a3 + (c22 + c13);
    uint32_t key = max_v((v0 << 8) + L.tag[0], (v1 << 8) + L.tag[1]);
    key = max_v(key, max_v((v2 << 8) + L.tag[2], (v3 << 8) + L.tag[3]));
    return max_v(key, max_v((v4 << 8) + L.tag[4], (v5 << 8) + L.tag[5]));
}

// ---- team path (groups of four ranks, LPG lanes per group) -----------------------------------------
//
// Team lane tl owns the credit elements (i, q) with q in qv[] and i in iv[]:
//   LPG 8: q = tl & 3, i in {tl >> 2, (tl >> 2) + 2};  LPG 4: q = tl, all i;  LPG 2: q in {tl, tl + 2}, all i
// and the permutations tl*PPL .. tl*PPL + PPL - 1 (PPL = 24 / LPG).
template <int LPG> struct TeamCfg {
    static constexpr int NQ = LPG >= 4 ? 1 : 4 / LPG;
    static constexpr int NI = LPG == 8 ? 2 : 4;
    static constexpr int PPL = 24 / LPG;
    static constexpr int NW = (PPL + 3) / 4;          // 32-bit words holding this lane's packed permutations
};

// Best permutation of the team's 4 x 4 credit tile (first maximum in lexicographic order); every team
// lane returns the value and receives the permutation packed 2 bits per position.
template <int LPG>
__device__ __forceinline__ int64_t team_best(const int64_t* cred, int tl, const unsigned (&mp)[TeamCfg<LPG>::NW],
                                             unsigned& bpk) {
    constexpr int PPL = TeamCfg<LPG>::PPL;
    int64_t best = -1;
    int bp = 0;
    bpk = 0;
#pragma unroll
    for (int pp = 0; pp < PPL; pp++) {
        const unsigned pk = (mp[pp >> 2] >> (8 * (pp & 3))) & 0xffu;
        const int64_t v = cred[(pk & 3) * 4] + cred[((pk >> 2) & 3) * 4 + 1] + cred[((pk >> 4) & 3) * 4 + 2] +
                          cred[((pk >> 6) & 3) * 4 + 3];
        if (v > best) { best = v; bp = tl * PPL + pp; bpk = pk; }
    }
#pragma unroll
    for (int o = LPG / 2; o; o >>= 1) {                // within the team: larger value, then lower permutation index
        const int64_t ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int op = __shfl_xor_sync(0xffffffffu, bp, o);
        const unsigned ok = __shfl_xor_sync(0xffffffffu, bpk, o);
        if (ov > best || (ov == best && op < bp)) { best = ov; bp = op; bpk = ok; }
    }
    return best;
}
// 32-bit granule units: value and permutation travel as one key (sum << 8 | 255 - permutation byte), so a plain
// maximum keeps the larger sum and, among equal sums, the earlier permutation.  Sums are below 2^24.  The
// permutation comes back as its byte (position 0 in the highest two bits, see perm_byte_at).
template <int LPG>
__device__ __forceinline__ uint32_t team_best(const uint32_t* cred, int tl, const unsigned (&mp)[TeamCfg<LPG>::NW],
                                              const uint8_t (&pidx)[TeamCfg<LPG>::PPL][4], const uint8_t* lut,
                                              unsigned& bpk) {
    static_assert(LPG == 2 || LPG == 4 || LPG == 8, "lane teams have two, four or eight lanes");
    if constexpr (LPG == 2) return team_best_reg2(cred, tl, bpk);
    uint32_t key;
    if constexpr (LPG == 4) {
        key = reg4_key(cred, reg4_lane(tl));
        key = max_v(key, __shfl_xor_sync(0xffffffffu, key, 2));
        key = max_v(key, __shfl_xor_sync(0xffffffffu, key, 1));
    } else {
        key = reg8_key(cred, reg8_lane(tl));
#pragma unroll
        for (int o = 4; o; o >>= 1) key = max_v(key, __shfl_xor_sync(0xffffffffu, key, o));
    }
    bpk = ~key & 255u;
    return key >> 8;
}
template <int LPG>
__device__ __forceinline__ int64_t team_best(const int64_t* cred, int tl, const unsigned (&mp)[TeamCfg<LPG>::NW],
                                             const uint8_t (&pidx)[TeamCfg<LPG>::PPL][4], const uint8_t* lut,
                                             unsigned& bpk) {
    return team_best<LPG>(cred, tl, mp, bpk);
}

// Row that the permutation returned by team_best puts at position q: a byte with position 0 on top for 32-bit granule
// units, two bits per position from the bottom for 64-bit byte values.
template <typename V> __device__ __forceinline__ int perm_pos(unsigned bpk, int q) {
    return sizeof(V) == 4 ? perm_byte_at(bpk, q) : (int)((bpk >> (2 * q)) & 3u);
}

// Per-CTA pointers and constants shared by the two value types.
struct Ctx {
    int N, G, tid, NT, lane, warp, n_warps;
    int term_ss, term_se;              // term e of shape s is at p_term[s * term_ss + e * term_se]
    int64_t *Dhat, *tbl, *send_acc, *recv_acc, *red, *task_f, *task_den, *pair;
    int64_t *score, *delta;            // incremental scoring: score of every shape; change of the chosen shape's table entries
    int32_t* dent;                     // ... and which entries those are (-1 = none)
    const uint32_t *p_inv, *p_inv_ptr;
    uint8_t *bind_src, *bind_dst;
    uint32_t* slotw;
    unsigned char* cred_warp;          // this warp's credit tiles
    const uint32_t* p_term;
    const uint16_t* p_fam_in;
    const uint8_t* p_fam_cls;
    const uint32_t* p_bucket_ptr;
    const uint8_t* perm_lut;           // tag (31 - p) -> packed permutation p of four items
    const int64_t* tscale;             // per rate class: (rate_lcm / bw) x bytes per value unit
    int32_t* chan_id_b;                // this matrix's outputs
    int16_t* lane_dst_b;
    uint16_t* lane_inst_b;
    int64_t *lane_bytes_b, *send_off_b, *recv_off_b;
};

struct Counters { unsigned long long tasks, sweeps; long long cyc[6], t_mark; };

#ifdef VP_PHASE_TIMING
// (the "memory" clobber keeps loads and stores on their side of the clock read)
#define VP_TICK(i) do { long long now_; asm volatile("mov.u64 %0, %%clock64;" : "=l"(now_) :: "memory"); cnt.cyc[i] += now_ - cnt.t_mark; cnt.t_mark = now_; } while (0)
#else
#define VP_TICK(i) do { } while (0)
#endif

// Algorithm 2 main loop for one matrix whose residual demand is held as values of type V
// (V = int64_t: bytes, unit = 1; V = uint32_t: granules, unit = granule_bytes).
template <int GS, int LPG, typename V>
__device__ __forceinline__ void decompose(const DevCat& dc, const KParams& kp, const Ctx& c, V* Drem, const V* cap,
                                          int64_t unit, int64_t left, int& k, int& st, Counters& cnt) {
    using TC = TeamCfg<LPG>;
    const int N = c.N, G = c.G, tid = c.tid, NT = c.NT, lane = c.lane, warp = c.warp, n_warps = c.n_warps;
    const int team = lane / LPG, tl = lane % LPG;
    int qv[TC::NQ], iv[TC::NI];
    unsigned mp[TC::NW];
    if constexpr (LPG > 1) {
#pragma unroll
        for (int kq = 0; kq < TC::NQ; kq++) qv[kq] = (tl & 3) + kq * LPG;
#pragma unroll
        for (int m = 0; m < TC::NI; m++) iv[m] = LPG == 8 ? (tl >> 2) + 2 * m : m;
#pragma unroll
        for (int w = 0; w < TC::NW; w++) mp[w] = 0;
#pragma unroll
        for (int pp = 0; pp < TC::PPL; pp++) mp[pp >> 2] |= perm4_packed_rt(tl * TC::PPL + pp) << (8 * (pp & 3));
    }
    uint8_t pidx[TC::PPL][4];
    if constexpr (LPG > 1) {
#pragma unroll
        for (int pp = 0; pp < TC::PPL; pp++) {
            const unsigned pk = (mp[pp >> 2] >> (8 * (pp & 3))) & 0xffu;
#pragma unroll
            for (int q = 0; q < 4; q++) pidx[pp][q] = (uint8_t)(((pk >> (2 * q)) & 3) * 4 + q);
        }
    }
    // Tile placement.  Two lanes per group: lane 1 reads the tile's rows rotated by two, i.e. eight credits away from lane 0,
    // so the sixteen tiles start in banks 0..7 and 16..23 (tile k at 33 (k mod 8) + 16 (k / 8)): every load of the warp then
    // touches 32 different banks.  Otherwise tiles are 17 credits apart.
    V* cred = (V*)c.cred_warp + (LPG == 2 && sizeof(V) == 4 ? 33 * (team & 7) + 16 * (team >> 3) : team * 17);
    const int n_score_warps = min(n_warps, (dc.n_shapes + 31) >> 5);
    const int ns_shift = (kp.n_start & (kp.n_start - 1)) == 0 ? 31 - __clz(kp.n_start) : -1;     // n_start a power of two: shifts for divisions

    const bool inc = kp.incremental != 0;
    // Small plain score tables (at most 16 D-hat cells, one shape per thread): the shape's lane counts are kept in a
    // register, four bits per cell, and scoring needs no term loads (see phase A).  Cells beyond G*G have count 0.
    const bool dense = LPG == 8 && !dc.sym && dc.tbl_size <= 16 && dc.n_shapes <= NT && ((uintptr_t)c.Dhat & 15) == 0;
    unsigned long long shape_mask = 0;
    if (LPG == 8 && dense && tid < dc.n_shapes)
        for (int e = 0; e < dc.max_terms; e++) {
            const uint32_t w = __ldg(&dc.term[(size_t)tid * dc.max_terms + e]);
            shape_mask |= (unsigned long long)(w >> 16) << (4 * ((w & 0xffffu) >> 3));
        }
    // a score is at most g x (what is left) and only shrinks: when that fits 32 bits the scores are kept as 32-bit
    // words, which shared memory can add to natively (64-bit adds are compare-and-swap loops)
    const bool s32 = inc && left * GS < ((int64_t)1 << 31);
    auto build_table = [&]() {
            // per-node-offset sums of D-hat; four threads share an entry when the CTA has that many
            const int S = dc.S, P = dc.P;
            const int parts = dc.tbl_size * 4 <= NT ? 4 : 1;
            const int total = dc.tbl_size * parts;
            for (int e0 = warp * 32; e0 < total; e0 += NT) {     // whole warps enter: the shuffles below need every lane
                const int e4 = e0 + lane;
                const bool live = e4 < total;
                const int e = e4 / parts, part = e4 % parts;
                const int q2 = e % S, q = (e / S) % S, delta = e / (S * S);
                int64_t s = 0;
                if (live)
                    for (int n = part; n < P; n += parts) {
                        int n2 = n + delta; if (n2 >= P) n2 -= P;
                        s += c.Dhat[(size_t)(n * S + q) * G + n2 * S + q2];
                    }
                if (parts == 4) {                       // the four threads of an entry are neighbours in a warp
                    s += __shfl_xor_sync(0xffffffffu, s, 1);
                    s += __shfl_xor_sync(0xffffffffu, s, 2);
                }
                if (live && part == 0) c.tbl[e] = s;
            }
            __syncthreads();
    };
    if (inc) {
        // incremental scoring: all scores once, then only what an activation changes (see the end of the loop)
        build_table();
        const char* tb = (const char*)c.tbl;
        for (int s = tid; s < dc.n_shapes; s += NT) {
            const uint32_t* tp = dc.term + (size_t)s * dc.max_terms;
            int64_t score = 0;
            for (int e = 0; e < dc.max_terms; e++) {
                const uint32_t w = __ldg(&tp[e]);
                score += *(const int64_t*)(tb + (w & 0xffffu)) * (int64_t)(w >> 16);
            }
            if (s32) ((uint32_t*)c.score)[s] = (uint32_t)score; else c.score[s] = score;
        }
        __syncthreads();
    }

    for (;;) {
        if (left == 0) break;
        if (k == kp.k_max) { st |= VP_ST_STEP_LIMIT; break; }
        // (A) Eq. (6): shape scores, first maximum
        if (dc.sym && !inc) build_table();
        // a score is at most g x (what is left): when that fits 32 bits the low words of the table suffice, and a cell of
        // D-hat can be decremented by a native 32-bit shared-memory add (a 64-bit one is a compare-and-swap loop)
        const bool narrow = left * GS < ((int64_t)1 << 31);
        if (warp < n_score_warps) {
            int64_t best = -1;
            int best_s = 0x7fffffff;
            const char* tb = (const char*)c.tbl;
            if (LPG == 8 && dense && narrow) {
                // one shape per thread, its lane counts in a register (a nibble per D-hat cell): sixteen multiply-adds
                // on the low words of D-hat, which eight 16-byte loads (the same for every thread) bring in
                const uint4* dh = (const uint4*)c.Dhat;
                uint32_t sc = 0;
#pragma unroll
                for (int v = 0; v < 8; v++) {
                    const uint4 x = dh[v];
                    sc += x.x * (uint32_t)((shape_mask >> (8 * v)) & 15u) + x.z * (uint32_t)((shape_mask >> (8 * v + 4)) & 15u);
                }
                if (tid < dc.n_shapes) { best = (int64_t)sc; best_s = tid; }
            } else
            for (int s = tid; s < dc.n_shapes; s += NT) {
                const uint32_t* tp = c.p_term + (size_t)s * c.term_ss;
                int64_t score = 0;
                if (inc) {
                    score = s32 ? (int64_t)((const uint32_t*)c.score)[s] : c.score[s];
                } else if (narrow) {
                    uint32_t score32 = 0;
#pragma unroll 4
                    for (int e = 0; e < dc.max_terms; e++) {
                        const uint32_t w = tp[(size_t)e * c.term_se];
                        score32 += *(const uint32_t*)(tb + (w & 0xffffu)) * (w >> 16);
                    }
                    score = (int64_t)score32;
                } else {
#pragma unroll 4
                    for (int e = 0; e < dc.max_terms; e++) {
                        const uint32_t w = tp[(size_t)e * c.term_se];
                        score += *(const int64_t*)(tb + (w & 0xffffu)) * (int64_t)(w >> 16);
                    }
                }
                if (score > best) { best = score; best_s = s; }     // ascending s: keeps the first maximum
            }
            warp_argmax_first(best, best_s);
            if (lane == 0) { c.red[warp] = best; c.red[32 + warp] = best_s; }
        }
        __syncthreads();
        int64_t best = -1;
        int best_s = 0x7fffffff;
        for (int w = 0; w < n_score_warps; w++) {
            const int64_t v = c.red[w];
            const int si = (int)c.red[32 + w];
            if (v > best || (v == best && si < best_s)) { best = v; best_s = si; }
        }
        if (best <= 0) { st |= VP_ST_UNCOVERED; break; }
        const int f0 = (int)c.p_bucket_ptr[best_s], H = (int)c.p_bucket_ptr[best_s + 1] - f0;
        const int n_tasks = H * kp.n_start;
        uint32_t my_term = 0;                              // incremental scoring: this warp's term of the chosen shape
        if (inc && warp < dc.max_terms) my_term = __ldg(&dc.term[(size_t)best_s * dc.max_terms + warp]);
        VP_TICK(1);

        // (B) MultiStartAA: one warp per (family, start)
        // With more than 32 groups and one lane per group, two warps share a task (each lane one group) and
        // meet at a named barrier of 64 threads where a single warp would use __syncwarp.
        const int W = (GS == 4 && LPG == 1 && G > 32 && n_warps >= 8) ? 2 : 1;
        const int sub = W == 2 ? (warp & 1) : 0, wgroup = W == 2 ? (warp >> 1) : warp;
        auto task_sync = [&]() {
            if constexpr (GS == 4 && LPG == 1) {
                if (W == 2) { asm volatile("bar.sync %0, 64;" ::"r"(1 + wgroup) : "memory"); return; }
            }
            __syncwarp();
        };
        for (int task = wgroup; task < n_tasks; task += n_warps / W) {
            const int h = ns_shift >= 0 ? task >> ns_shift : task / kp.n_start, f = f0 + h, t = task - h * kp.n_start;
            const uint16_t* fin = c.p_fam_in + (size_t)f * N;
            const uint8_t* fcls = c.p_fam_cls + (size_t)f * N;
            uint8_t* srcb = c.bind_src + (size_t)task * N;
            uint8_t* dstb = c.bind_dst + (size_t)task * N;
            // the family's slot words (instance ids) are fetched now and parked in shared memory for step (D)
            uint32_t slot_pre[(VP_MAX_N + 31) / 32];
            if (t == 0 && sub == 0) {
#pragma unroll
                for (int rr = 0; rr < (VP_MAX_N + 31) / 32; rr++) {
                    if (LPG > 1 && rr * 32 >= N) break;              // (lane teams: N <= 64, mostly one round)
                    if (rr * 32 + lane < N) slot_pre[rr] = __ldg(&dc.fam_slot[(size_t)f * N + rr * 32 + lane]);
                }
            }
            // initial destination binding: in-slot e = d * GS + q, start t rotates q by t
            if (LPG > 1 && N <= 32 && (N & (N - 1)) == 0) {
                const int e = lane & (N - 1), q = e % GS;            // (lanes beyond N repeat the first N: no branch)
                dstb[fin[e] & 0xff] = (uint8_t)(e - q + (q + t) % GS);
            } else if (LPG > 1) {
                for (int e = lane; e < N; e += 32) {
                    const int q = e % GS;
                    dstb[fin[e] & 0xff] = (uint8_t)(e - q + (q + t) % GS);
                }
            } else {
                for (int d = sub * 32 + lane; d < G; d += 32 * W)
#pragma unroll
                    for (int q = 0; q < GS; q++) dstb[fin[d * GS + q] & 0xff] = (uint8_t)(d * GS + (q + t) % GS);
            }
            int64_t F_old = -1, F_new = -1, tmax = 0;
            bool tmax_done = false;
            if constexpr (LPG > 1) {
                // team path: one rank group per team of LPG lanes (G <= 32 / LPG)
                // Teams beyond the last group repeat the last group's work on a tile of their own (same values to the same
                // binding entries), so the code below needs no per-team predicates; only the sum over teams leaves them out.
                const bool active = team < G;
                const int a = active ? team : G - 1;        // the team's group: source group, then destination group
                V cap_out[TC::NQ], cap_in[TC::NQ];
                int r_in[TC::NQ], cls_in[TC::NQ];
#pragma unroll
                for (int kq = 0; kq < TC::NQ; kq++) {
                    const unsigned w = fin[a * 4 + qv[kq]];
                    cap_out[kq] = cap[fcls[a * 4 + qv[kq]]];
                    cls_in[kq] = (int)(w >> 8);
                    cap_in[kq] = cap[cls_in[kq]];
                    r_in[kq] = (int)(w & 0xff);
                }
                __syncwarp();
                unsigned bpk = 0;
                for (int sweep = 0; sweep < kp.i_aa; sweep++) {
#pragma unroll
                    for (int kq = 0; kq < TC::NQ; kq++) {      // source half: credits of source group a
                        const int dq = dstb[a * 4 + qv[kq]];
#pragma unroll
                        for (int m = 0; m < TC::NI; m++)
                            cred[iv[m] * 4 + qv[kq]] = min_v(Drem[(size_t)(a * 4 + iv[m]) * N + dq], cap_out[kq]);
                    }
                    __syncwarp();
                    team_best<LPG>(cred, tl, mp, pidx, c.perm_lut, bpk);
#pragma unroll
                    for (int kq = 0; kq < TC::NQ; kq++)          // (with eight lanes, lanes tl and tl + 4 write the same entry)
                        srcb[a * 4 + qv[kq]] = (uint8_t)(a * 4 + perm_pos<V>(bpk, qv[kq]));
                    __syncwarp();
#pragma unroll
                    for (int kq = 0; kq < TC::NQ; kq++) {      // destination half: credits into group a
                        const int sq = srcb[r_in[kq]];
#pragma unroll
                        for (int m = 0; m < TC::NI; m++)
                            cred[iv[m] * 4 + qv[kq]] = min_v(Drem[(size_t)sq * N + a * 4 + iv[m]], cap_in[kq]);
                    }
                    __syncwarp();
                    const V v = team_best<LPG>(cred, tl, mp, pidx, c.perm_lut, bpk);
#pragma unroll
                    for (int kq = 0; kq < TC::NQ; kq++)
                        dstb[r_in[kq]] = (uint8_t)(a * 4 + perm_pos<V>(bpk, qv[kq]));
                    // Eq. (8): sum over the teams.  Every lane of a team holds the team's value and the
                    // exchanges connect equal team lanes only, so all 32 lanes end with the same total.
                    if constexpr (sizeof(V) == 4) {
                        // at most 64 lanes of less than 2^25 granules each: the total fits 32 bits, one warp-reduce
                        F_new = (int64_t)__reduce_add_sync(0xffffffffu, (active && tl == 0) ? (uint32_t)v : 0u);
                    } else {
                        int64_t part = active ? (int64_t)v : 0;
#pragma unroll
                        for (int o = 16; o >= LPG; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                        F_new = part;
                    }
                    cnt.sweeps++;
                    if (F_new <= F_old) break;
                    F_old = F_new;
                    __syncwarp();
                }
                // Eq. (9) volumes are the chosen credits of the last destination half; slowest lane of Eq. (10)
                V xmax = 0;
#pragma unroll
                for (int kq = 0; kq < TC::NQ; kq++) {
                    const V x = cred[perm_pos<V>(bpk, qv[kq]) * 4 + qv[kq]];
                    xmax = max_v(xmax, x);
                    tmax = max_v(tmax, (int64_t)x * c.tscale[cls_in[kq]]);
                }
                if constexpr (sizeof(V) == 4) {
                    if (dc.n_classes == 1) {          // one path rate: the slowest lane carries the largest volume
                        tmax = (int64_t)__reduce_max_sync(0xffffffffu, (uint32_t)xmax) * c.tscale[0];
                        tmax_done = true;
                    }
                }
                __syncwarp();
            } else {
                // register path: one lane per rank group
                task_sync();
                int64_t* pair = c.pair + wgroup * 6;
                for (int sweep = 0; sweep < kp.i_aa; sweep++) {
                    for (int a = sub * 32 + lane; a < G; a += 32 * W) {            // source half
                        V cr[GS][GS];
                        unsigned bpk;
#pragma unroll
                        for (int q = 0; q < GS; q++) {
                            const int r = a * GS + q;
                            const V cp = cap[fcls[r]];
                            const int dq = dstb[r];
#pragma unroll
                            for (int i = 0; i < GS; i++) cr[i][q] = min_v(Drem[(size_t)(a * GS + i) * N + dq], cp);
                        }
                        best_assignment<GS, V>(cr, bpk);
#pragma unroll
                        for (int q = 0; q < GS; q++) srcb[a * GS + q] = (uint8_t)(a * GS + ((bpk >> (2 * q)) & 3));
                    }
                    task_sync();
                    int64_t part = 0;
                    tmax = 0;
                    for (int d = sub * 32 + lane; d < G; d += 32 * W) {            // destination half
                        V cr[GS][GS];
                        int rq[GS], cls[GS];
                        unsigned bpk;
#pragma unroll
                        for (int q = 0; q < GS; q++) {
                            const unsigned w = fin[d * GS + q];
                            rq[q] = (int)(w & 0xff);
                            cls[q] = (int)(w >> 8);
                            const V cp = cap[cls[q]];
                            const int sq = srcb[rq[q]];
#pragma unroll
                            for (int j = 0; j < GS; j++) cr[j][q] = min_v(Drem[(size_t)sq * N + d * GS + j], cp);
                        }
                        part += (int64_t)best_assignment<GS, V>(cr, bpk);
#pragma unroll
                        for (int q = 0; q < GS; q++) {
                            const int j = (int)((bpk >> (2 * q)) & 3);
                            dstb[rq[q]] = (uint8_t)(d * GS + j);
                            V x = cr[0][q];                           // the chosen credit = the lane's volume, Eq. (9)
#pragma unroll
                            for (int jj = 1; jj < GS; jj++) if (j == jj) x = cr[jj][q];
                            tmax = max_v(tmax, (int64_t)x * c.tscale[cls[q]]);
                        }
                    }
                    F_new = warp_sum_i64(part);                      // Eq. (8)
                    if (W == 2) {                                    // add the partner warp's half (slots alternate by sweep)
                        if (lane == 0) pair[(sweep & 1) * 2 + sub] = F_new;
                        task_sync();
                        F_new = pair[(sweep & 1) * 2] + pair[(sweep & 1) * 2 + 1];
                    } else {
                        __syncwarp();
                    }
                    if (sub == 0) cnt.sweeps++;
                    if (F_new <= F_old) break;
                    F_old = F_new;
                }
                tmax = warp_max_i64(tmax);
                if (W == 2) {
                    if (lane == 0) pair[4 + sub] = tmax;
                    task_sync();
                    tmax = max_v(pair[4], pair[5]);
                }
                tmax_done = true;
            }
            if (!tmax_done) tmax = warp_max_i64(tmax);
            if (sub == 0) cnt.tasks++;
            if (t == 0 && sub == 0) {
#pragma unroll
                for (int rr = 0; rr < (VP_MAX_N + 31) / 32; rr++) {
                    if (LPG > 1 && rr * 32 >= N) break;
                    if (rr * 32 + lane < N) c.slotw[h * N + rr * 32 + lane] = slot_pre[rr];
                }
            }
            if (lane == 0 && sub == 0) {
                c.task_f[task] = F_new;
                c.task_den[task] = F_new > 0 ? kp.lambda_ns * dc.W + tmax : 1;
            }
        }
        __syncthreads();
        VP_TICK(2);

        // (C) best start per family (largest F, lowest t), then largest utility, lowest family;
        //     every warp computes it for itself, over the lanes 0 .. H-1 only
        int wtask;
        int64_t wF;
        if (H == 1 && kp.n_start <= 32) {
            // one family (the common case): its best start is one arg-max over the lanes, no utilities to compare
            int64_t ff = lane < kp.n_start ? c.task_f[lane] : -1;
            int tt = lane;
            warp_argmax_first(ff, tt);
            wtask = tt; wF = ff;
        } else {
            int64_t bf = -1, bd = 1;
            int bt = 0x7fffffff;
            for (int h = lane; h < H; h += 32) {
                int64_t ff = -1; int tt = 0;
                for (int t = 0; t < kp.n_start; t++)
                    if (c.task_f[h * kp.n_start + t] > ff) { ff = c.task_f[h * kp.n_start + t]; tt = h * kp.n_start + t; }
                if (bt == 0x7fffffff || util_greater(ff, c.task_den[tt], bf, bd)) { bf = ff; bd = c.task_den[tt]; bt = tt; }
            }
            int width = 1;
            while (width < H && width < 32) width <<= 1;
            for (int o = width >> 1; o; o >>= 1) {
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
            wtask = __shfl_sync(0xffffffffu, bt, 0);
            wF = __shfl_sync(0xffffffffu, bf, 0);
        }
        if (wF <= 0) { st |= VP_ST_NO_PROGRESS; break; }
        VP_TICK(3);

        // (D) emit activation k, D_rem -= X(E), update D-hat, write offset row k+1
        {
            const int h = ns_shift >= 0 ? wtask >> ns_shift : wtask / kp.n_start;
            const uint32_t* slot = c.slotw + h * N;
            const uint8_t* srcb = c.bind_src + (size_t)wtask * N;
            const uint8_t* dstb = c.bind_dst + (size_t)wtask * N;
            const size_t row = (size_t)k * N, orow = (size_t)(k + 1) * N;
            for (int r = tid; r < N; r += NT) {
                const uint32_t w = slot[r];
                const int i = srcb[r], j = dstb[r];
                const V x = min_v(cap[(w >> 24) & 0xf], Drem[(size_t)i * N + j]);
                // straight-line: an idle lane (x = 0) writes the idle values and adds zero; only the D-hat update is skipped
                const bool busy = x > 0;
                const int64_t bytes = (int64_t)x * unit;
                const int64_t sa = c.send_acc[i] + bytes, ra = c.recv_acc[j] + bytes;
                c.lane_dst_b[row + i] = busy ? (int16_t)j : (int16_t)-1;
                c.lane_inst_b[row + i] = busy ? (uint16_t)(w & 0xffffu) : (uint16_t)0xFFFF;
                c.lane_bytes_b[row + i] = bytes;
                c.send_acc[i] = sa;
                c.recv_acc[j] = ra;
                if (busy) {
                    Drem[(size_t)i * N + j] -= x;           // (for N = 256 this is a read-modify-write in L2: not for idle lanes)
                    int64_t* cell = &c.Dhat[(i / GS) * G + (j / GS)];
                    if (narrow) atomicSub((unsigned int*)cell, (unsigned int)x);        // high word is zero, low word >= x
                    else atomicAdd((unsigned long long*)cell, (unsigned long long)(-(int64_t)x));
                }
                c.send_off_b[orow + i] = sa;              // src and dst are permutations: every rank is written once
                if (c.recv_off_b) c.recv_off_b[orow + j] = ra;
            }
            if (tid == 0) c.chan_id_b[k] = f0 + h;
            left -= wF;
        }
        k++;
        __syncthreads();
        if (inc) {
            // The activation changed D-hat only on the cells of the chosen shape, i.e. only the table entries of its
            // terms: one warp re-sums an entry, then every shape that uses a changed entry gets count x change.
            const int S = dc.S, P = dc.P;
            for (int kk = warp; kk < dc.max_terms; kk += n_warps) {
                const uint32_t w = kk == warp ? my_term : __ldg(&dc.term[(size_t)best_s * dc.max_terms + kk]);
                int64_t dlt = 0;
                int e = -1;
                if (w >> 16) {                             // the same word in every lane of the warp
                    e = (int)(w & 0xffffu) >> 3;
                    const int q2 = e % S, q = (e / S) % S, delta = e / (S * S);
                    int64_t sum = 0;
                    for (int n = lane; n < P; n += 32) {
                        int n2 = n + delta; if (n2 >= P) n2 -= P;
                        sum += c.Dhat[(size_t)(n * S + q) * G + n2 * S + q2];
                    }
                    sum = warp_sum_i64(sum);
                    dlt = sum - c.tbl[e];
                    __syncwarp();
                    if (lane == 0) c.tbl[e] = sum;
                }
                if (lane == 0) { c.delta[kk] = dlt; c.dent[kk] = e; }
            }
            __syncthreads();
            for (int kk = 0; kk < dc.max_terms; kk++) {
                const int e = c.dent[kk];
                const int64_t dlt = c.delta[kk];
                if (e < 0 || dlt == 0) continue;
                for (uint32_t idx = c.p_inv_ptr[e] + tid; idx < c.p_inv_ptr[e + 1]; idx += NT) {
                    const uint32_t w = c.p_inv[idx];
                    if (s32) atomicAdd((uint32_t*)c.score + (w & 0xffffu), (uint32_t)(w >> 16) * (uint32_t)dlt);
                    else atomicAdd((unsigned long long*)&c.score[w & 0xffffu], (unsigned long long)((int64_t)(w >> 16) * dlt));
                }
            }
            __syncthreads();
        }
        VP_TICK(4);
    }
}

template <int GS, int LPG>
__global__ void __launch_bounds__(LPG > 1 ? 256 : 512, LPG > 1 ? 2 : 1)
vp_schedule_kernel(DevCat dc, KParams kp, const int64_t* __restrict__ demand, const int64_t* __restrict__ tau_in, int B,
                   int32_t* __restrict__ n_steps, int32_t* __restrict__ chan_id, int16_t* __restrict__ lane_dst,
                   uint16_t* __restrict__ lane_inst, int64_t* __restrict__ lane_bytes, int64_t* __restrict__ send_off,
                   int64_t* __restrict__ recv_off, int64_t* __restrict__ tau_out, int32_t* __restrict__ status,
                   int64_t* ws_drem, unsigned int* counter, const int* __restrict__ todo) {
    // With a to-do list (left by the kernel for large node-symmetric catalogs) the CTAs work through the matrices
    // todo[0 .. counter[1]) and pull positions from counter[2]; without one, through 0 .. B-1 from counter[0].
    static_assert(LPG == 1 || GS == 4, "lane teams are defined for groups of four ranks");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int N = dc.N, G = dc.G, tid = threadIdx.x, NT = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, n_warps = NT >> 5;
    const Smem L = smem_layout(dc, kp, n_warps, LPG);
    // lane teams are only used up to 16 groups (N <= 64), where D_rem is always in shared memory: saying so at
    // compile time lets every access to it be a shared-memory instruction with 32-bit addressing
    int64_t* Drem;
    if constexpr (LPG > 1) Drem = (int64_t*)(smem_raw + L.drem);
    else Drem = kp.drem_in_smem ? (int64_t*)(smem_raw + L.drem) : ws_drem + (size_t)blockIdx.x * N * N;
    Ctx c;
    c.N = N; c.G = G; c.tid = tid; c.NT = NT; c.lane = lane; c.warp = warp; c.n_warps = n_warps;
    c.Dhat = (int64_t*)(smem_raw + L.dhat);
    c.tbl = dc.sym ? (int64_t*)(smem_raw + L.tbl) : c.Dhat;
    c.send_acc = (int64_t*)(smem_raw + L.send_acc);
    c.recv_acc = (int64_t*)(smem_raw + L.recv_acc);
    c.red = (int64_t*)(smem_raw + L.red);
    c.pair = (int64_t*)(smem_raw + L.pair);
    c.score = (int64_t*)(smem_raw + L.score);
    c.delta = (int64_t*)(smem_raw + L.delta);
    c.dent = (int32_t*)(smem_raw + L.delta + 32 * 8);
    c.p_inv = dc.inv; c.p_inv_ptr = dc.inv_ptr;
    c.task_f = (int64_t*)(smem_raw + L.task_f);
    c.task_den = (int64_t*)(smem_raw + L.task_den);
    c.bind_src = smem_raw + L.bind_src;
    c.bind_dst = smem_raw + L.bind_dst;
    c.slotw = (uint32_t*)(smem_raw + L.slotw);
    c.cred_warp = smem_raw + L.cred + warp * cred_bytes_per_warp(LPG);
    __shared__ int s_b, s_flags, s_units;
    __shared__ int64_t s_tau, s_left;
    __shared__ int64_t s_cap[VP_MAX_CLASSES], s_tscale[VP_MAX_CLASSES];
    __shared__ uint32_t s_cap32[VP_MAX_CLASSES];
    __shared__ uint8_t s_perm_lut[32];
    c.tscale = s_tscale;
    c.perm_lut = s_perm_lut;
    if (tid < 32) s_perm_lut[tid] = (uint8_t)(31 - tid < 24 ? perm4_packed_rt(31 - tid) : 0);
    unsigned long long n_act = 0;                          // work counters (thread 0 / lane 0 of each warp)
    Counters cnt;
    cnt.tasks = 0; cnt.sweeps = 0; cnt.t_mark = 0;
    for (int i = 0; i < 6; i++) cnt.cyc[i] = 0;

    // ---- stage the catalog: whole arrays by bulk asynchronous copies (TMA) that complete on one mbarrier; should the
    // bounded wait give up, the same arrays are copied with plain loads
    c.p_term = dc.term;
    c.term_ss = dc.max_terms; c.term_se = 1;
    c.p_fam_in = dc.fam_in;
    c.p_fam_cls = dc.fam_cls;
    c.p_bucket_ptr = dc.bucket_ptr;
    {
        const int ns_pad = (dc.n_shapes + 31) & ~31;
        const unsigned b_term = kp.stage_terms ? (unsigned)(ns_pad * dc.max_terms * 4) : 0u;
        const unsigned b_bucket = kp.stage_bucket ? (unsigned)align16((dc.n_shapes + 1) * 4) : 0u;
        const unsigned b_inv = kp.incremental ? (unsigned)align16(dc.n_terms * 4) : 0u;
        const unsigned b_invp = kp.incremental ? (unsigned)align16((dc.tbl_size + 1) * 4) : 0u;
        const unsigned b_fin = kp.stage_fam ? (unsigned)align16(dc.n_families * N * 2) : 0u;
        const unsigned b_fcls = kp.stage_fam ? (unsigned)align16(dc.n_families * N) : 0u;
        const unsigned total = b_term + b_bucket + b_inv + b_invp + b_fin + b_fcls;
        __shared__ __align__(8) unsigned long long s_stage_bar;
        bool landed = false;
        if (total > 0 && total < (1u << 20)) {
            const unsigned bar = smem_u32(&s_stage_bar);
            if (tid == 0) {
                mbar_init(bar, 1);
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                mbar_expect_tx(bar, total);
                if (b_term) bulk_load(smem_u32(smem_raw + L.term), dc.term_t, b_term, bar);
                if (b_bucket) bulk_load(smem_u32(smem_raw + L.bucket), dc.bucket_ptr, b_bucket, bar);
                if (b_inv) bulk_load(smem_u32(smem_raw + L.inv), dc.inv, b_inv, bar);
                if (b_invp) bulk_load(smem_u32(smem_raw + L.inv_ptr), dc.inv_ptr, b_invp, bar);
                if (b_fin) bulk_load(smem_u32(smem_raw + L.fam_in), dc.fam_in, b_fin, bar);
                if (b_fcls) bulk_load(smem_u32(smem_raw + L.fam_cls), dc.fam_cls, b_fcls, bar);
            }
            __syncthreads();                                     // the barrier is initialised before anyone polls it
            landed = __syncthreads_and(mbar_wait_bounded(bar, 0, 1u << 20)) != 0;
        }
        if (kp.stage_terms) {
            uint32_t* st = (uint32_t*)(smem_raw + L.term);
            // transposed ([term][shape], rows padded to 32 shapes): consecutive threads score consecutive shapes, so
            // every load of a term is conflict-free
            if (!landed) for (int e = tid; e < ns_pad * dc.max_terms; e += NT) st[e] = dc.term_t[e];
            c.p_term = st;
            c.term_ss = 1; c.term_se = ns_pad;
        }
        if (kp.stage_bucket) {
            uint32_t* bp = (uint32_t*)(smem_raw + L.bucket);
            if (!landed) for (int e = tid; e <= dc.n_shapes; e += NT) bp[e] = dc.bucket_ptr[e];
            c.p_bucket_ptr = bp;
        }
        if (kp.incremental) {
            uint32_t* iv = (uint32_t*)(smem_raw + L.inv);
            uint32_t* ip = (uint32_t*)(smem_raw + L.inv_ptr);
            if (!landed) {
                for (int e = tid; e < dc.n_terms; e += NT) iv[e] = dc.inv[e];
                for (int e = tid; e <= dc.tbl_size; e += NT) ip[e] = dc.inv_ptr[e];
            }
            c.p_inv = iv; c.p_inv_ptr = ip;
        }
        if (kp.stage_fam) {
            uint16_t* fi = (uint16_t*)(smem_raw + L.fam_in);
            uint8_t* fc = smem_raw + L.fam_cls;
            if (!landed) for (int e = tid; e < dc.n_families * N; e += NT) { fi[e] = dc.fam_in[e]; fc[e] = dc.fam_cls[e]; }
            c.p_fam_in = fi; c.p_fam_cls = fc;
        }
    }

    for (;;) {
        if (tid == 0) {
            if (todo) {
                const unsigned at = atomicAdd(counter + 2, 1u);
                s_b = at < counter[1] ? todo[at] : B;
            } else {
                s_b = (int)atomicAdd(counter, 1u);
            }
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
        c.chan_id_b = chan_id + (size_t)b * kp.k_max;
        c.lane_dst_b = lane_dst + lane_base;
        c.lane_inst_b = lane_inst + lane_base;
        c.lane_bytes_b = lane_bytes + lane_base;
        c.send_off_b = send_off + off_base;
        c.recv_off_b = recv_off ? recv_off + off_base : nullptr;

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
            c.send_acc[i] = 0; c.recv_acc[i] = 0;
            c.send_off_b[i] = 0;
            if (c.recv_off_b) c.recv_off_b[i] = 0;
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
                est = max_v(est, max_v(ceil_div_i64(row, dc.bw_max), ceil_div_i64(col, dc.bw_max)));
            }
            for (int cell = tid; cell < G * G; cell += NT) {
                int a = cell / G, d = cell % G;
                int64_t s = 0;
#pragma unroll
                for (int i = 0; i < GS; i++)
#pragma unroll
                    for (int j = 0; j < GS; j++) s += Drem[(size_t)(a * GS + i) * N + d * GS + j];
                c.Dhat[cell] = s;
            }
            __syncthreads();
            for (int l = tid; l < dc.n_res; l += NT) {
                uint32_t bwl = dc.forced_bw[l];
                if (!bwl) continue;
                int64_t f = 0;
                for (uint32_t e = dc.forced_ptr[l]; e < dc.forced_ptr[l + 1]; e++) f += c.Dhat[dc.forced_cell[e]];
                est = max_v(est, ceil_div_i64(f, (int64_t)bwl));
            }
            est = warp_max_i64(est);
            tot = warp_sum_i64(tot);
            if (lane == 0) { c.red[warp] = est; c.red[32 + warp] = tot; }
            __syncthreads();
            if (tid == 0) {
                int64_t e = 0, t = 0;
                for (int w = 0; w < n_warps; w++) { e = max_v(e, c.red[w]); t += c.red[32 + w]; }
                int64_t tq = tau_given > 0 ? tau_given : max_v((int64_t)1, ceil_div_i64(e, (int64_t)kp.k_target));
                int64_t cap_max = 0;
                for (int cl = 0; cl < dc.n_classes; cl++) {
                    int64_t cp = (tq * dc.class_bw[cl]) / kp.granule * kp.granule;
                    s_cap[cl] = cp < kp.granule ? kp.granule : cp;
                    cap_max = max_v(cap_max, s_cap[cl]);
                }
                // granule units: capacities below 2^22 granules (four credits and a permutation byte share 32 bits)
                const int units = cap_max / kp.granule < ((int64_t)1 << 22) && kp.granule >= 256;
                for (int cl = 0; cl < dc.n_classes; cl++) {
                    s_cap32[cl] = (uint32_t)(units ? s_cap[cl] / kp.granule : 0);
                    s_tscale[cl] = dc.class_wdiv[cl] * (units ? kp.granule : 1);
                }
                s_tau = tq; s_left = t; s_units = units;
            }
            __syncthreads();
            tau = s_tau;
            const bool units = s_units != 0;
            VP_TICK(0);
            if (units) {
                // the byte copy is no longer needed: overwrite it with the demand in granules
                uint32_t* Drem32 = (uint32_t*)Drem;
                for (int e = tid; e < N * N; e += NT) Drem32[e] = (uint32_t)(D[e] / kp.granule);
                for (int cell = tid; cell < G * G; cell += NT) c.Dhat[cell] /= kp.granule;
                __syncthreads();
                decompose<GS, LPG, uint32_t>(dc, kp, c, Drem32, s_cap32, kp.granule, s_left / kp.granule, k, st, cnt);
            } else {
                decompose<GS, LPG, int64_t>(dc, kp, c, Drem, s_cap, 1, s_left, k, st, cnt);
            }
        }
        __syncthreads();
        // ---- idle rows beyond n_steps; offset rows repeat the totals
        for (size_t e = (size_t)k * N + tid; e < (size_t)kp.k_max * N; e += NT) {
            c.lane_dst_b[e] = -1;
            c.lane_inst_b[e] = 0xFFFF;
            c.lane_bytes_b[e] = 0;
            const int i = (int)(e % N);
            c.send_off_b[N + e] = c.send_acc[i];
            if (c.recv_off_b) c.recv_off_b[N + e] = c.recv_acc[i];
        }
        for (int kk = k + tid; kk < kp.k_max; kk += NT) c.chan_id_b[kk] = -1;
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
    if (lane == 0 && cnt.tasks) { atomicAdd(&stats[1], cnt.tasks); atomicAdd(&stats[2], cnt.sweeps); }
#ifdef VP_PHASE_TIMING
    if (tid == 0) for (int i = 0; i < 6; i++) atomicAdd(&stats[3 + i], (unsigned long long)cnt.cyc[i]);
#endif
}

}  // namespace

#include "schedule_big.cuh"
#include "schedule_warp.cuh"

#ifndef VP_BIG_MIN_GROUPS
#define VP_BIG_MIN_GROUPS 16      // node-symmetric catalogs with at least this many groups of four take vp_schedule_big_kernel
#endif

namespace {

struct Launch {
    int threads, grid, lpg;
    int kernel;               // 0: one CTA per matrix (vp_schedule_kernel), 1: one warp per matrix (vp_schedule_warp_kernel),
                              // 2: vp_schedule_big_kernel, followed by vp_schedule_kernel on the matrices it left
    size_t smem;
    KParams kp;
    int big_w, big_threads, big_grid;     // kernel 2: warps per task, threads and CTAs of the first launch
    size_t big_smem;
    int wave;                 // CTAs of the chosen kernel that are resident at once (the grid is min(B, wave) or less)
};
static_assert(sizeof(Launch) <= sizeof(((vp_launch_memo*)0)->launch), "the launch memo is too small");

typedef void (*KernelFn)(DevCat, KParams, const int64_t*, const int64_t*, int, int32_t*, int32_t*, int16_t*, uint16_t*,
                         int64_t*, int64_t*, int64_t*, int64_t*, int32_t*, int64_t*, unsigned int*, const int*);
typedef void (*BigKernelFn)(DevCat, KParams, const int64_t*, const int64_t*, int, int32_t*, int32_t*, int16_t*, uint16_t*,
                            int64_t*, int64_t*, int64_t*, int64_t*, int32_t*, unsigned int*, int*, const int*);

KernelFn pick_kernel(int g, int lpg) {
    switch (g) {
        case 1: return vp_schedule_kernel<1, 1>;
        case 2: return vp_schedule_kernel<2, 1>;
        case 3: return vp_schedule_kernel<3, 1>;
        case 4:
            switch (lpg) {
                case 8: return vp_schedule_kernel<4, 8>;
                case 4: return vp_schedule_kernel<4, 4>;
                case 2: return vp_schedule_kernel<4, 2>;
                default: return vp_schedule_kernel<4, 1>;
            }
    }
    return nullptr;
}
BigKernelFn pick_big_kernel(int w, bool dec) {
    if (dec) return w == 2 ? vp_schedule_big_kernel<2, true> : vp_schedule_big_kernel<1, true>;
    return w == 2 ? vp_schedule_big_kernel<2, false> : vp_schedule_big_kernel<1, false>;
}

// Raises a kernel's limit of dynamic shared memory on the current device to `bytes` if it is lower.  The limit belongs
// to the function, not to a launch: launches are planned once and replayed from a memo, several catalogs share the
// kernels, and one kernel is launched with different sizes, so the limit must never be lowered by a later plan.
int raise_dynamic_smem(const void* fn, size_t bytes) {
    struct Mark { int device; const void* fn; size_t bytes; };
    static Mark marks[64];
    static int n_marks = 0;
    static std::mutex lock;
    std::lock_guard<std::mutex> hold(lock);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return VP_E_CUDA;
    Mark* m = nullptr;
    for (int i = 0; i < n_marks; i++)
        if (marks[i].device == dev && marks[i].fn == fn) m = &marks[i];
    if (m && m->bytes >= bytes) return VP_OK;
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return VP_E_CUDA;
    if (m) m->bytes = bytes;
    else if (n_marks < 64) marks[n_marks++] = Mark{dev, fn, bytes};
    return VP_OK;
}

int resolve_params(const vp_catalog* c, const vp_sched_params* p, KParams* kp) {
    if (!c || !p || c->device < 0) return VP_E_BAD_ARG;         // (a host-only handle launches nothing)
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

// Works out kernel, launch shape and shared-memory layout for a batch of B matrices.  This sets function attributes
// and asks the runtime for occupancies, so vp_catalog keeps the last few results (see plan_launch).
int plan_launch_uncached(const vp_catalog* c, int B, const vp_sched_params* p, Launch* out) {
    const DevCat& dc = c->dc;
    Launch L;
    memset(&L, 0, sizeof(L));
    int rc = resolve_params(c, p, &L.kp);
    if (rc) return rc;
    L.kernel = 0;
    L.lpg = 1;
    if (dc.g == 4) L.lpg = dc.G <= 4 ? 8 : (dc.G <= 8 ? 4 : (dc.G <= 16 ? 2 : 1));
    L.threads = dc.N <= 64 ? 128 : 512;
    L.kp.drem_in_smem = dc.N <= 64;
    // terms go to shared memory when small, or when the CTA is alone on its SM anyway (512 threads)
    L.kp.stage_terms = (size_t)dc.n_shapes * dc.max_terms * 4 <= (L.threads >= 512 ? 128 * 1024 : 32 * 1024);
    // family tables go to shared memory only when small: beyond that, CTAs per SM matter more than their latency
    L.kp.stage_fam = (size_t)dc.n_families * dc.N * 3 <= 16 * 1024;
    L.kp.stage_bucket = ((size_t)dc.n_shapes + 1) * 4 <= 32 * 1024;
    // many shapes over a small node-symmetric score table: keep the scores and update them (the inverted terms
    // take the place of the staged terms in shared memory)
    L.kp.incremental = dc.sym && dc.inv && dc.n_shapes >= 512 && dc.max_terms <= 32 && dc.max_terms <= L.threads / 32;
    if (L.kp.incremental) {
        const int staged = L.kp.stage_terms;
        L.kp.stage_terms = 0;
        if ((size_t)smem_layout(dc, L.kp, L.threads / 32, L.lpg).total + 2048 > (size_t)c->max_smem_optin) {
            L.kp.incremental = 0;
            L.kp.stage_terms = staged;
        }
    }
    L.smem = (size_t)smem_layout(dc, L.kp, L.threads / 32, L.lpg).total;
    if (L.smem + 2048 > (size_t)c->max_smem_optin) return VP_E_UNSUPPORTED;
    KernelFn fn = pick_kernel(dc.g, L.lpg);
    if (!fn) return VP_E_UNSUPPORTED;
    if (raise_dynamic_smem((const void*)fn, L.smem) != VP_OK) return VP_E_CUDA;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, L.threads, L.smem) != cudaSuccess || per_sm < 1)
        return VP_E_CUDA;
    long long cap = (long long)per_sm * c->sm_count;
    L.wave = (int)cap;
    L.grid = (int)(B < cap ? B : cap);
#ifndef VP_NO_BIG_KERNEL
    // Large node-symmetric catalogs (groups of four, more than sixteen groups): 16-bit credits in shared memory and
    // scores on the per-node-offset table; the general kernel then takes whatever matrices that kernel left.
    const int big_min_groups = VP_BIG_MIN_GROUPS;
    if (dc.g == 4 && dc.G >= big_min_groups && dc.G <= 64 && dc.sym && dc.shape_pat && dc.n_patterns < 1024 && dc.n_classes <= 15) {
        const size_t smem = (size_t)big_smem_layout(dc, L.kp).total;
        if (smem + 2048 <= (size_t)c->max_smem_optin) {
            // one lane per group: two warps per task beyond 32 groups, and then sixteen warps for shape scoring and the
            // emit step; up to 32 groups a task is one warp and four to eight warps per CTA leave room for several CTAs per SM
            const int w = dc.G > 32 ? 2 : 1;
            // sixteen groups: two warps, two tasks each (eight CTAs per SM: config 3's 1,024 matrices are one wave)
            // up to 32 groups: four warps, a task each (256 threads, with four warps idle in Step 2, halve the CTAs per SM:
            // 6.9 -> 4.6 ms for 1,024 matrices at N = 96)
            const int threads = w == 2 ? BIG_W2_THREADS : (dc.G > 16 ? 128 : 64);
            BigKernelFn bf = pick_big_kernel(w, big_use_dec(dc));
            if (raise_dynamic_smem((const void*)bf, smem) != VP_OK) return VP_E_CUDA;
            int bper_sm = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bper_sm, bf, threads, smem) != cudaSuccess || bper_sm < 1) return VP_E_CUDA;
            const long long bcap = (long long)bper_sm * c->sm_count;
            L.kernel = 2; L.big_w = w; L.big_threads = threads; L.big_smem = smem;
            L.big_grid = (int)(B < bcap ? B : bcap);
            L.wave = (int)bcap;
        }
    }
#endif
#ifndef VP_NO_WARP_KERNEL
    // Small topologies (groups of four, at most four groups, plain D-hat scores): one warp per matrix.  It has no block
    // barriers and less work per activation than a CTA per matrix, and wins at every batch size once the matrices run
    // in 32-bit granule units (granule >= 256 bytes; the choice between units and bytes is made per matrix, so the
    // granule decides here); with smaller granules only when the batch exceeds the CTAs of one wave.  Up to four
    // matrices per SM get a CTA of one warp each (a scheduler to themselves), larger batches two or four warps per CTA.
    if (dc.g == 4 && dc.G <= 4 && !dc.sym && (B > cap || p->granule_bytes >= 256)) {
        const int warps = B <= 4 * c->sm_count ? 1 : (B <= 8 * c->sm_count ? 2 : 4);
        const size_t smem = (size_t)warp_smem_layout(dc, L.kp, warps).total;
        if (smem + 2048 <= (size_t)c->max_smem_optin) {
            if (raise_dynamic_smem((const void*)vp_schedule_warp_kernel, smem) != VP_OK) return VP_E_CUDA;
            int wper_sm = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&wper_sm, vp_schedule_warp_kernel, warps * 32, smem) != cudaSuccess || wper_sm < 1)
                return VP_E_CUDA;
            const long long wcap = (long long)wper_sm * c->sm_count, want = ((long long)B + warps - 1) / warps;
            L.kernel = 1; L.lpg = 8; L.threads = warps * 32; L.smem = smem;
            L.kp.drem_in_smem = 1; L.kp.stage_terms = L.kp.stage_fam = L.kp.stage_bucket = 1;
            L.grid = (int)(want < wcap ? want : wcap);
            L.wave = (int)wcap * warps;
        }
    }
#endif
    *out = L;
    return VP_OK;
}

// plan_launch_uncached through the catalog's memo.  A launch depends on B only through min(B, one wave) -- except for
// the switch to the warp kernel, which happens exactly when B exceeds the general kernel's wave -- so batches are
// keyed by min(B, 65536) and a cached launch is reused when its own grid rule gives the same answer.  The memo is not
// locked: calls that share a catalog handle from several host threads must be serialised by the caller (as must
// anything else that shares a workspace).
int plan_launch(const vp_catalog* cc, int B, const vp_sched_params* p, Launch* out) {
    vp_catalog* c = const_cast<vp_catalog*>(cc);
    if (!c || !p) return VP_E_BAD_ARG;
    for (vp_launch_memo& m : c->memo) {
        if (!m.valid || m.B_class != B || m.k_target != p->k_target || m.n_start != p->n_start || m.i_aa != p->i_aa ||
            m.k_max != p->k_max || m.lambda_ns != p->lambda_ns || m.granule != p->granule_bytes)
            continue;
        memcpy(out, m.launch, sizeof(Launch));
        return VP_OK;
    }
    Launch L;
    const int rc = plan_launch_uncached(c, B, p, &L);
    if (rc) return rc;
    vp_launch_memo& m = c->memo[c->memo_next];
    c->memo_next = (c->memo_next + 1) % (int)(sizeof(c->memo) / sizeof(c->memo[0]));
    m.valid = 1; m.B_class = B;
    m.k_target = p->k_target; m.n_start = p->n_start; m.i_aa = p->i_aa; m.k_max = p->k_max;
    m.lambda_ns = p->lambda_ns; m.granule = p->granule_bytes;
    memcpy(m.launch, &L, sizeof(Launch));
    *out = L;
    return VP_OK;
}

// Workspace: 256 bytes of counters; one residual slot per CTA of the general kernel when it keeps the residual outside
// shared memory; with the kernel for large node-symmetric catalogs also the list of matrices left to the general
// kernel, the work order and its keys.
struct WsLayout { size_t drem, todo, order, key, total; };
WsLayout ws_layout(const vp_catalog* c, const Launch& L, int B) {
    WsLayout w;
    const size_t slot_bytes = !L.kp.drem_in_smem ? (size_t)L.grid * c->dc.N * c->dc.N * 8 : 0;
    w.drem = 256;
    w.todo = vp_align256(256 + slot_bytes);
    const size_t list = L.kernel == 2 ? vp_align256((size_t)B * 4) : 0;
    w.order = w.todo + list;
    w.key = w.order + list;
    w.total = w.key + list;
    return w;
}
size_t workspace_bytes(const vp_catalog* c, const Launch& L, int B) { return ws_layout(c, L, B).total; }

}  // namespace

extern "C" size_t vp_schedule_workspace_bytes(const vp_catalog* c, int B, const vp_sched_params* p) {
    Launch L;
    if (B <= 0 || !c || !p) return 0;
    int prev = -1;
    cudaGetDevice(&prev);
    if (prev != c->device) cudaSetDevice(c->device);
    int rc = plan_launch(c, B, p, &L);
    if (prev >= 0 && prev != c->device) cudaSetDevice(prev);
    return rc == VP_OK ? workspace_bytes(c, L, B) : 0;
}

extern "C" int vp_schedule_batch(const vp_catalog* c, const vp_sched_params* p, const int64_t* demand,
                                 const int64_t* tau_ns_in, int B, int32_t* n_steps, int32_t* chan_id,
                                 int16_t* lane_dst, uint16_t* lane_inst, int64_t* lane_bytes, int64_t* send_off,
                                 int64_t* recv_off, int64_t* tau_ns_out, int32_t* status, void* workspace,
                                 size_t workspace_bytes_given, void* cuda_stream) {
    if (!c || !p) return VP_E_BAD_ARG;
    if (B <= 0 || !demand || !n_steps || !chan_id || !lane_dst || !lane_inst || !lane_bytes || !send_off || !status)
        return VP_E_BAD_ARG;
    int prev = -1;
    cudaGetDevice(&prev);
    if (prev != c->device && cudaSetDevice(c->device) != cudaSuccess) return VP_E_CUDA;
    Launch L;
    int rc = plan_launch(c, B, p, &L);
    if (!rc && (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes_given < workspace_bytes(c, L, B))) rc = VP_E_WORKSPACE;
    if (!rc) {
        cudaStream_t stream = (cudaStream_t)cuda_stream;
        unsigned int* counter = (unsigned int*)workspace;
        int64_t* ws_drem = (int64_t*)((char*)workspace + 256);
        if (cudaMemsetAsync(counter, 0, 256, stream) != cudaSuccess) rc = VP_E_CUDA;
        if (!rc) {
            vp_prof_mark(0, 0, stream);
            if (L.kernel == 1) {
                vp_schedule_warp_kernel<<<L.grid, L.threads, L.smem, stream>>>(
                    c->dc, L.kp, demand, tau_ns_in, B, n_steps, chan_id, lane_dst, lane_inst, lane_bytes, send_off, recv_off,
                    tau_ns_out, status, counter);
            } else if (L.kernel == 2) {
                const WsLayout w = ws_layout(c, L, B);
                int* todo = (int*)((char*)workspace + w.todo);
                int* order = nullptr;
                if (B > L.big_grid && B <= 16384) {          // more matrices than CTAs: longest first (see big_rank_kernel)
                    order = (int*)((char*)workspace + w.order);
                    int* key = (int*)((char*)workspace + w.key);
                    big_count_nonzero_kernel<<<(B + 7) / 8, 256, 0, stream>>>(demand, B, c->dc.N * c->dc.N, key);
                    big_rank_kernel<<<(B + 255) / 256, 256, 0, stream>>>(key, B, order);
                    g_vp_launches += 2;
                }
                pick_big_kernel(L.big_w, big_use_dec(c->dc))<<<L.big_grid, L.big_threads, L.big_smem, stream>>>(
                    c->dc, L.kp, demand, tau_ns_in, B, n_steps, chan_id, lane_dst, lane_inst, lane_bytes, send_off, recv_off,
                    tau_ns_out, status, counter, todo, order);
                g_vp_launches++;
                pick_kernel(c->dc.g, L.lpg)<<<L.grid, L.threads, L.smem, stream>>>(
                    c->dc, L.kp, demand, tau_ns_in, B, n_steps, chan_id, lane_dst, lane_inst, lane_bytes, send_off, recv_off,
                    tau_ns_out, status, ws_drem, counter, todo);
            } else {
                pick_kernel(c->dc.g, L.lpg)<<<L.grid, L.threads, L.smem, stream>>>(
                    c->dc, L.kp, demand, tau_ns_in, B, n_steps, chan_id, lane_dst, lane_inst, lane_bytes, send_off, recv_off,
                    tau_ns_out, status, ws_drem, counter, nullptr);
            }
            g_vp_launches++;
            if (cudaGetLastError() != cudaSuccess) rc = VP_E_CUDA;
            vp_prof_mark(0, 1, stream);
        }
    }
    if (prev >= 0 && prev != c->device) cudaSetDevice(prev);
    return rc;
}

extern "C" int vp_schedule_launch_info(const vp_catalog* c, int B, const vp_sched_params* p, int32_t* out4) {
    if (B <= 0 || !c || !p || !out4) return VP_E_BAD_ARG;
    Launch L;
    int prev = -1;
    cudaGetDevice(&prev);
    if (prev != c->device && cudaSetDevice(c->device) != cudaSuccess) return VP_E_CUDA;
    const int rc = plan_launch(c, B, p, &L);
    if (prev >= 0 && prev != c->device) cudaSetDevice(prev);
    if (rc) return rc;
    out4[0] = L.kernel;
    out4[1] = L.kernel == 2 ? L.big_grid : L.grid;
    out4[2] = L.kernel == 2 ? L.big_threads : L.threads;
    out4[3] = (int32_t)(L.kernel == 2 ? L.big_smem : L.smem);
    return VP_OK;
}

extern "C" int vp_schedule_read_stats(const void* workspace, void* cuda_stream, uint64_t* out3) {
    if (!workspace || !out3) return VP_E_BAD_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(out3, (const char*)workspace + 16, 24, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return VP_E_CUDA;
    return cudaStreamSynchronize(stream) == cudaSuccess ? VP_OK : VP_E_CUDA;
}
