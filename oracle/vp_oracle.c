/*
 * CPU oracle for the VarioPath online scheduler and send-buffer pack.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, single-threaded
 * statement of what the hot path computes, written from the paper.  It is used
 * by the tests, by the smoke check and by the benchmark's CPU-baseline leg and
 * by nothing else; the CUDA library shares no code with it.
 *
 * What follows which passage:
 *   channel model, Eq. (1) feasibility, schedule validity ... Section 3
 *   shapes Eq. (3), families Eq. (4), endpoint binding ...... Section 4.1
 *   Algorithm 2 (outer loop), Step 1 Eq. (5)(6), Step 2 Eq. (7)(8) with the
 *   Alternating Algorithm and MultiStartAA, Step 3 Eq. (9)(10) ... Section 4.2
 *   modeled completion time Eq. (2) ........................... Section 3
 *   time quantum from K_target ................................ Section 5
 *   send-buffer layout / pack ................................. Section 5
 *
 * Parity unpinned (conventions of this build that no value printed in the
 * paper fixes; only agreement between the two implementations is testable):
 * the tau rule, lambda, N_start, I_AA, catalog order and all tie-breaks.
 * Everything else is pinned by the tests under tests/ marked "not gpu".
 *
 * All arithmetic is integer.  Credits are kept in bytes, i.e. Eq. (7) scaled by
 * tau: tau*h = min(D_rem, tau*bw); the scaling does not change any arg-max.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

#define VPO_MAX_G 8          /* largest group size the permutation search supports */
#define VPO_MAX_RES 4
#define VPO_ENTRY_LIMIT ((int64_t)1 << 40)

/* per-matrix status bits */
enum {
    VPO_ST_NEGATIVE = 1, VPO_ST_OVERFLOW = 2, VPO_ST_DIAG = 4, VPO_ST_GRANULE = 8,
    VPO_ST_BAD_TAU = 16, VPO_ST_UNCOVERED = 32, VPO_ST_NO_PROGRESS = 64, VPO_ST_STEP_LIMIT = 128,
    VPO_ST_PACK_MISMATCH = 256, VPO_ST_PACK_CAPACITY = 512
};

typedef struct {
    int a, d, kind, n_res, mult;
    int64_t bw;
    int res[VPO_MAX_RES];
} vpo_inst;

typedef struct vpo_catalog {
    int N, G, g, groups_per_node, n_res, n_inst;
    vpo_inst *inst;
    int n_shapes, n_families, total_nnz;
    uint32_t *shape_ptr;
    uint16_t *nnz;            /* total_nnz x (a, d, count, pad) */
    uint32_t *bucket_ptr;
    uint16_t *fam_inst;       /* n_families x N */
    int64_t W;                /* lcm of all instance rates */
    int64_t bw_max;
} vpo_catalog;

/* ------------------------------------------------------------------ blobs */

static uint32_t rd32(const uint8_t *p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24); }
static uint16_t rd16(const uint8_t *p) { return (uint16_t)(p[0] | (p[1] << 8)); }

static int64_t gcd64(int64_t a, int64_t b) { while (b) { int64_t t = a % b; a = b; b = t; } return a; }

void vpo_free(vpo_catalog *c)
{
    if (!c) return;
    free(c->inst); free(c->shape_ptr); free(c->nnz); free(c->bucket_ptr); free(c->fam_inst); free(c);
}

/* Parse the two blobs.  Returns NULL and sets *err (1 truncated/bad magic, 2 bad field). */
vpo_catalog *vpo_load(const void *topo, size_t topo_bytes, const void *chan, size_t chan_bytes, int *err)
{
    const uint8_t *t = (const uint8_t *)topo, *h = (const uint8_t *)chan;
    *err = 1;
    if (topo_bytes < 32 || rd32(t) != 0x50545056u || rd32(t + 4) != 1) return NULL;
    if (chan_bytes < 24 || rd32(h) != 0x48435056u || rd32(h + 4) != 1) return NULL;
    vpo_catalog *c = (vpo_catalog *)calloc(1, sizeof(*c));
    c->N = (int)rd32(t + 8); c->G = (int)rd32(t + 12); c->g = (int)rd32(t + 16);
    c->groups_per_node = (int)rd32(t + 20); c->n_res = (int)rd32(t + 24); c->n_inst = (int)rd32(t + 28);
    if (topo_bytes < 32 + (size_t)c->n_inst * 20) { vpo_free(c); return NULL; }
    *err = 2;
    if (c->N <= 0 || c->G <= 0 || c->g <= 0 || c->N != c->G * c->g || c->g > VPO_MAX_G || c->n_inst <= 0) { vpo_free(c); return NULL; }
    c->inst = (vpo_inst *)calloc((size_t)c->n_inst, sizeof(vpo_inst));
    c->W = 1; c->bw_max = 0;
    for (int r = 0; r < c->n_inst; r++) {
        const uint8_t *p = t + 32 + (size_t)r * 20;
        vpo_inst *q = &c->inst[r];
        q->a = rd16(p); q->d = rd16(p + 2); q->kind = p[4]; q->n_res = p[5]; q->mult = rd16(p + 6);
        q->bw = rd32(p + 8);
        if (q->a >= c->G || q->d >= c->G || q->n_res > VPO_MAX_RES || q->bw <= 0 || q->mult < 1) { vpo_free(c); return NULL; }
        for (int k = 0; k < q->n_res; k++) {
            q->res[k] = rd16(p + 12 + 2 * k);
            if (q->res[k] >= c->n_res) { vpo_free(c); return NULL; }
        }
        c->W = c->W / gcd64(c->W, q->bw) * q->bw;
        if (c->W >= ((int64_t)1 << 20)) { vpo_free(c); return NULL; }
        if (q->bw > c->bw_max) c->bw_max = q->bw;
    }
    if ((int)rd32(h + 8) != c->N) { vpo_free(c); return NULL; }
    c->n_shapes = (int)rd32(h + 12); c->n_families = (int)rd32(h + 16); c->total_nnz = (int)rd32(h + 20);
    size_t need = 24 + 4 * ((size_t)c->n_shapes + 1) * 2 + 8 * (size_t)c->total_nnz + 2 * (size_t)c->n_families * c->N;
    *err = 1;
    if (chan_bytes < need) { vpo_free(c); return NULL; }
    const uint8_t *p = h + 24;
    c->shape_ptr = (uint32_t *)malloc(4 * ((size_t)c->n_shapes + 1));
    for (int s = 0; s <= c->n_shapes; s++, p += 4) c->shape_ptr[s] = rd32(p);
    c->nnz = (uint16_t *)malloc(8 * (size_t)c->total_nnz + 8);
    for (int k = 0; k < c->total_nnz * 4; k++, p += 2) c->nnz[k] = rd16(p);
    c->bucket_ptr = (uint32_t *)malloc(4 * ((size_t)c->n_shapes + 1));
    for (int s = 0; s <= c->n_shapes; s++, p += 4) c->bucket_ptr[s] = rd32(p);
    c->fam_inst = (uint16_t *)malloc(2 * (size_t)c->n_families * c->N + 2);
    for (size_t k = 0; k < (size_t)c->n_families * c->N; k++, p += 2) c->fam_inst[k] = rd16(p);
    *err = 0;
    return c;
}

void vpo_info(const vpo_catalog *c, int32_t *out /* N,G,g,n_inst,n_shapes,n_families,max_nnz,n_res */)
{
    int mx = 0;
    for (int s = 0; s < c->n_shapes; s++) {
        int n = (int)(c->shape_ptr[s + 1] - c->shape_ptr[s]);
        if (n > mx) mx = n;
    }
    out[0] = c->N; out[1] = c->G; out[2] = c->g; out[3] = c->n_inst; out[4] = c->n_shapes;
    out[5] = c->n_families; out[6] = mx; out[7] = c->n_res;
}

/*
 * Catalog validity.  Eq. (3): every shape has row and column sums g.  Eq. (4):
 * every family selects exactly M_ad instances of R_ad, no instance more often
 * than its lane multiplicity, and no directed resource twice.  Returns 0 when
 * all hold; 3 for a shape that breaks Eq. (3), 4 for a family that breaks
 * Eq. (4), 5 for malformed index arrays.
 */
int vpo_check_catalog(const vpo_catalog *c)
{
    int G = c->G, N = c->N;
    if (c->shape_ptr[0] != 0 || (int)c->shape_ptr[c->n_shapes] != c->total_nnz) return 5;
    if (c->bucket_ptr[0] != 0 || (int)c->bucket_ptr[c->n_shapes] != c->n_families) return 5;
    int64_t *M = (int64_t *)malloc(sizeof(int64_t) * G * G);
    int64_t *cnt = (int64_t *)malloc(sizeof(int64_t) * G * G);
    int *used = (int *)malloc(sizeof(int) * (c->n_res + 1));
    int *times = (int *)malloc(sizeof(int) * c->n_inst);
    int rc = 0;
    for (int s = 0; s < c->n_shapes && !rc; s++) {
        if (c->shape_ptr[s + 1] < c->shape_ptr[s] || c->bucket_ptr[s + 1] < c->bucket_ptr[s]) { rc = 5; break; }
        memset(M, 0, sizeof(int64_t) * G * G);
        for (uint32_t k = c->shape_ptr[s]; k < c->shape_ptr[s + 1]; k++) {
            int a = c->nnz[4 * k], d = c->nnz[4 * k + 1], m = c->nnz[4 * k + 2];
            if (a >= G || d >= G || m == 0 || M[a * G + d] != 0) { rc = 5; break; }
            M[a * G + d] = m;
        }
        if (rc) break;
        for (int a = 0; a < G; a++) {               /* Eq. (3) */
            int64_t row = 0, col = 0;
            for (int d = 0; d < G; d++) { row += M[a * G + d]; col += M[d * G + a]; }
            if (row != c->g || col != c->g) { rc = 3; break; }
        }
        if (rc) break;
        for (uint32_t f = c->bucket_ptr[s]; f < c->bucket_ptr[s + 1] && !rc; f++) {   /* Eq. (4) */
            memset(cnt, 0, sizeof(int64_t) * G * G);
            memset(used, 0, sizeof(int) * (c->n_res + 1));
            memset(times, 0, sizeof(int) * c->n_inst);
            int prev = -1;
            for (int r = 0; r < N; r++) {
                int id = c->fam_inst[(size_t)f * N + r];
                if (id >= c->n_inst || id < prev) { rc = 5; break; }
                prev = id;
                const vpo_inst *q = &c->inst[id];
                cnt[q->a * G + q->d]++;
                if (++times[id] > q->mult) { rc = 4; break; }
                for (int k = 0; k < q->n_res; k++)
                    if (used[q->res[k]]++) { rc = 4; break; }
                if (rc) break;
            }
            if (!rc && memcmp(cnt, M, sizeof(int64_t) * G * G) != 0) rc = 4;
        }
    }
    free(M); free(cnt); free(used); free(times);
    return rc;
}

/* 1 when every ordered group pair that can carry demand has a shape with M_ad > 0. */
int vpo_catalog_covers(const vpo_catalog *c)
{
    int G = c->G;
    char *seen = (char *)calloc((size_t)G * G, 1);
    for (int k = 0; k < c->total_nnz; k++) seen[c->nnz[4 * k] * G + c->nnz[4 * k + 1]] = 1;
    int ok = 1;
    for (int a = 0; a < G; a++)
        for (int d = 0; d < G; d++)
            if ((a != d || c->g >= 2) && !seen[a * G + d]) ok = 0;
    free(seen);
    return ok;
}

/* ------------------------------------------------- concrete-channel model */

/*
 * Eq. (1) on concrete lanes.  Lane i (source rank i) goes to dst[i] over path
 * instance inst[i]; dst[i] < 0 marks an idle lane.  Checks: the instance
 * connects the two ranks' groups, i != dst, no destination receives twice, no
 * instance carries more lanes than its multiplicity, no directed resource is
 * used by two lanes.  Returns 0 when feasible, else 1..5 naming the failed test.
 */
int vpo_lanes_feasible(const vpo_catalog *c, const int16_t *dst, const uint16_t *inst)
{
    int N = c->N, g = c->g, rc = 0;
    int *used = (int *)calloc((size_t)c->n_res + 1, sizeof(int));
    int *recv = (int *)calloc((size_t)N, sizeof(int));
    int *times = (int *)calloc((size_t)c->n_inst, sizeof(int));
    for (int i = 0; i < N && !rc; i++) {
        if (dst[i] < 0) continue;
        int j = dst[i];
        if (j >= N || j == i) { rc = 1; break; }
        if (inst[i] >= c->n_inst) { rc = 2; break; }
        const vpo_inst *q = &c->inst[inst[i]];
        if (q->a != i / g || q->d != j / g) { rc = 2; break; }
        if (recv[j]++) { rc = 3; break; }
        if (++times[inst[i]] > q->mult) { rc = 4; break; }
        for (int k = 0; k < q->n_res; k++)
            if (used[q->res[k]]++) { rc = 5; break; }
    }
    free(used); free(recv); free(times);
    return rc;
}

/*
 * Modeled aggregate bandwidth of one stage when lanes MAY share resources
 * (Figure 1): a directed resource used by m lanes gives each of them 1/m of
 * its path rate; a lane runs at its most contended resource's share.
 * Returned as numerator over the common denominator 5040 = lcm(1..10).
 */
int64_t vpo_aggregate_bw_x5040(const vpo_catalog *c, const int16_t *dst, const uint16_t *inst)
{
    int N = c->N;
    int *used = (int *)calloc((size_t)c->n_res + 1, sizeof(int));
    for (int i = 0; i < N; i++) {
        if (dst[i] < 0) continue;
        const vpo_inst *q = &c->inst[inst[i]];
        for (int k = 0; k < q->n_res; k++) used[q->res[k]]++;
    }
    int64_t total = 0;
    for (int i = 0; i < N; i++) {
        if (dst[i] < 0) continue;
        const vpo_inst *q = &c->inst[inst[i]];
        int share = 1;
        for (int k = 0; k < q->n_res; k++) if (used[q->res[k]] > share) share = used[q->res[k]];
        total += q->bw * 5040 / share;
    }
    free(used);
    return total;
}

/* --------------------------------------------------------- tau and caps */

static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

/*
 * Time quantum from K_target (Section 5, "Global execution granularity"; the
 * formula is this build's reading).  est = the largest of: every rank's send
 * and receive volume over the fastest path rate, and for every directed
 * resource l the demand of all group pairs whose EVERY path instance crosses l,
 * over the fastest such instance.  tau = max(1, ceil(est / K_target)).
 */
static int64_t derive_tau(const vpo_catalog *c, const int64_t *D, int k_target)
{
    int N = c->N, G = c->G, g = c->g;
    int64_t est = 0;
    for (int i = 0; i < N; i++) {
        int64_t row = 0, col = 0;
        for (int j = 0; j < N; j++) { row += D[(size_t)i * N + j]; col += D[(size_t)j * N + i]; }
        int64_t t = ceil_div(row, c->bw_max); if (t > est) est = t;
        t = ceil_div(col, c->bw_max); if (t > est) est = t;
    }
    int64_t *forced = (int64_t *)calloc((size_t)c->n_res + 1, sizeof(int64_t));
    int64_t *fbw = (int64_t *)calloc((size_t)c->n_res + 1, sizeof(int64_t));
    int *common = (int *)malloc(sizeof(int) * (c->n_res + 1));
    for (int a = 0; a < G; a++)
        for (int d = 0; d < G; d++) {
            int n_paths = 0;
            int64_t best_bw = 0;
            memset(common, 0, sizeof(int) * (c->n_res + 1));
            for (int r = 0; r < c->n_inst; r++) {
                const vpo_inst *q = &c->inst[r];
                if (q->a != a || q->d != d) continue;
                n_paths++;
                if (q->bw > best_bw) best_bw = q->bw;
                for (int k = 0; k < q->n_res; k++) common[q->res[k]]++;
            }
            if (!n_paths) continue;
            int64_t dhat = 0;
            for (int i = a * g; i < a * g + g; i++)
                for (int j = d * g; j < d * g + g; j++) dhat += D[(size_t)i * N + j];
            for (int l = 0; l < c->n_res; l++)
                if (common[l] == n_paths) {
                    forced[l] += dhat;
                    if (best_bw > fbw[l]) fbw[l] = best_bw;
                }
        }
    for (int l = 0; l < c->n_res; l++)
        if (fbw[l] > 0) {
            int64_t t = ceil_div(forced[l], fbw[l]);
            if (t > est) est = t;
        }
    free(forced); free(fbw); free(common);
    int64_t tau = ceil_div(est, k_target);
    return tau < 1 ? 1 : tau;
}

/* Capacity of instance r within one quantum, in whole granules (at least one). */
static int64_t inst_cap(const vpo_inst *q, int64_t tau, int64_t u)
{
    int64_t cap = (tau * q->bw) / u * u;
    return cap < u ? u : cap;
}

static int64_t min64(int64_t a, int64_t b) { return a < b ? a : b; }

/* ----------------------------------------------- permutations, in order */

/* Lexicographic successor of p[0..n-1]; returns 0 after the last permutation. */
static int next_perm(int *p, int n)
{
    int i = n - 2;
    while (i >= 0 && p[i] > p[i + 1]) i--;
    if (i < 0) return 0;
    int j = n - 1;
    while (p[j] < p[i]) j--;
    int t = p[i]; p[i] = p[j]; p[j] = t;
    for (int l = i + 1, r = n - 1; l < r; l++, r--) { t = p[l]; p[l] = p[r]; p[r] = t; }
    return 1;
}

/*
 * Exact g x g assignment by enumeration: maximise sum_q credit[phi(q)][q]
 * (row phi(q) is given to column q); first maximum in lexicographic order of
 * (phi(0), ..., phi(g-1)) wins.  Returns the value.
 */
static int64_t best_assignment(const int64_t credit[VPO_MAX_G][VPO_MAX_G], int g, int *phi_out)
{
    int p[VPO_MAX_G];
    for (int q = 0; q < g; q++) p[q] = q;
    int64_t best = -1;
    do {
        int64_t v = 0;
        for (int q = 0; q < g; q++) v += credit[p[q]][q];
        if (v > best) { best = v; memcpy(phi_out, p, sizeof(int) * g); }
    } while (next_perm(p, g));
    return best;
}

/* ------------------------------------------------------- MultiStartAA */

typedef struct {
    int64_t *trace; int cap; int len;   /* optional records: (step, family, start, sweep, F) per AA sweep,
                                           (step, family, -2 - start, slot, src * 65536 + dst) for the binding a run
                                           ends with, and (step, family, -1, sum of volumes, W * duration) per
                                           candidate */
} vpo_trace;

/*
 * Step 2 for one family.  Slots r = 0..N-1 are the family's instances in
 * ascending id; slots a*g..a*g+g-1 leave group a (out-slots), and the slots
 * entering group d, in ascending position, are its in-slots.  Start t binds
 * in-slot q of group d to rank d*g + (q+t) mod g.  A sweep is the source half
 * (one exact assignment per source group, destinations fixed) followed by the
 * destination half (sources fixed).  A run ends after i_aa sweeps or after the
 * first sweep that does not raise F; its binding is kept as it then stands.
 * The start with the largest F wins, lowest t on ties.
 */
static int64_t multistart_aa(const vpo_catalog *c, int fam, const int64_t *Drem, const int64_t *cap_inst,
                             int n_start, int i_aa, int *src_best, int *dst_best,
                             vpo_trace *tr, int step)
{
    int N = c->N, G = c->G, g = c->g;
    const uint16_t *fi = &c->fam_inst[(size_t)fam * N];
    int *in_slot = (int *)malloc(sizeof(int) * N);     /* in_slot[d*g+q] = slot */
    int *fill = (int *)calloc((size_t)G, sizeof(int));
    int *src = (int *)malloc(sizeof(int) * N), *dst = (int *)malloc(sizeof(int) * N);
    for (int r = 0; r < N; r++) {
        int d = c->inst[fi[r]].d;
        in_slot[d * g + fill[d]++] = r;
    }
    int64_t F_best = -1;
    int64_t credit[VPO_MAX_G][VPO_MAX_G];
    int phi[VPO_MAX_G];
    for (int t = 0; t < n_start; t++) {
        for (int d = 0; d < G; d++)
            for (int q = 0; q < g; q++) dst[in_slot[d * g + q]] = d * g + (q + t) % g;
        for (int r = 0; r < N; r++) src[r] = r;          /* overwritten by the first source half */
        int64_t F_old = -1, F_new = -1;
        for (int sweep = 0; sweep < i_aa; sweep++) {
            for (int a = 0; a < G; a++) {                /* source half */
                for (int i = 0; i < g; i++)
                    for (int q = 0; q < g; q++) {
                        int r = a * g + q;
                        credit[i][q] = min64(Drem[(size_t)(a * g + i) * N + dst[r]], cap_inst[fi[r]]);
                    }
                best_assignment(credit, g, phi);
                for (int q = 0; q < g; q++) src[a * g + q] = a * g + phi[q];
            }
            for (int d = 0; d < G; d++) {                /* destination half */
                for (int j = 0; j < g; j++)
                    for (int q = 0; q < g; q++) {
                        int r = in_slot[d * g + q];
                        credit[j][q] = min64(Drem[(size_t)src[r] * N + d * g + j], cap_inst[fi[r]]);
                    }
                best_assignment(credit, g, phi);
                for (int q = 0; q < g; q++) dst[in_slot[d * g + q]] = d * g + phi[q];
            }
            F_new = 0;                                   /* Eq. (8), in bytes */
            for (int r = 0; r < N; r++)
                F_new += min64(Drem[(size_t)src[r] * N + dst[r]], cap_inst[fi[r]]);
            if (tr && tr->trace && tr->len < tr->cap) {
                int64_t *o = &tr->trace[5 * (size_t)tr->len++];
                o[0] = step; o[1] = fam; o[2] = t; o[3] = sweep; o[4] = F_new;
            }
            if (F_new <= F_old) break;
            F_old = F_new;
        }
        if (tr && tr->trace)                             /* tracing only: the binding this run ends with */
            for (int r = 0; r < N && tr->len < tr->cap; r++) {
                int64_t *o = &tr->trace[5 * (size_t)tr->len++];
                o[0] = step; o[1] = fam; o[2] = -2 - t; o[3] = r; o[4] = (int64_t)src[r] * 65536 + dst[r];
            }
        if (F_new > F_best) {
            F_best = F_new;
            memcpy(src_best, src, sizeof(int) * N);
            memcpy(dst_best, dst, sizeof(int) * N);
        }
    }
    free(in_slot); free(fill); free(src); free(dst);
    return F_best;
}

/* ------------------------------------------------------- Algorithm 2 */

/*
 * Decompose one demand matrix.  Outputs are for one matrix:
 *   chan_id[k_max], lane_dst/lane_inst/lane_bytes[k_max][N] indexed by source
 *   rank, send_off/recv_off[k_max+1][N] (recv_off may be NULL).  Steps at or
 *   beyond n_steps are filled with chan_id -1, lane_dst -1, lane_inst 0xFFFF,
 *   bytes 0; offset rows past n_steps repeat the totals.
 * tau_in > 0 overrides the derived quantum.  k_target, n_start, i_aa = 0 select
 * the defaults 2N, g, 3.
 */
int vpo_schedule(const vpo_catalog *c, const int64_t *D, int64_t tau_in,
                 int64_t lambda_ns, int k_target, int n_start, int i_aa, int64_t granule, int k_max,
                 int32_t *n_steps, int32_t *chan_id, int16_t *lane_dst, uint16_t *lane_inst,
                 int64_t *lane_bytes, int64_t *send_off, int64_t *recv_off, int64_t *tau_out,
                 int32_t *status, int64_t *trace, int trace_cap, int32_t *trace_len)
{
    int N = c->N, G = c->G, g = c->g;
    if (k_max <= 0 || granule <= 0 || lambda_ns < 0 || lambda_ns >= VPO_ENTRY_LIMIT) return -1;
    if (k_target == 0) k_target = 2 * N;
    if (n_start == 0) n_start = g;
    if (i_aa == 0) i_aa = 3;
    if (k_target < 0 || n_start < 0 || i_aa < 0) return -1;
    vpo_trace tr = { trace, trace_cap, 0 };

    for (int k = 0; k < k_max; k++) {
        chan_id[k] = -1;
        for (int i = 0; i < N; i++) {
            lane_dst[(size_t)k * N + i] = -1;
            lane_inst[(size_t)k * N + i] = 0xFFFF;
            lane_bytes[(size_t)k * N + i] = 0;
        }
    }
    memset(send_off, 0, sizeof(int64_t) * (size_t)(k_max + 1) * N);
    if (recv_off) memset(recv_off, 0, sizeof(int64_t) * (size_t)(k_max + 1) * N);
    *n_steps = 0;
    if (tau_out) *tau_out = 0;

    int st = 0;
    for (int i = 0; i < N; i++)
        for (int j = 0; j < N; j++) {
            int64_t v = D[(size_t)i * N + j];
            if (v < 0) st |= VPO_ST_NEGATIVE;
            else if (v >= VPO_ENTRY_LIMIT) st |= VPO_ST_OVERFLOW;
            else {
                if (i == j && v != 0) st |= VPO_ST_DIAG;
                if (v % granule) st |= VPO_ST_GRANULE;
            }
        }
    if (tau_in < 0 || tau_in > VPO_ENTRY_LIMIT) st |= VPO_ST_BAD_TAU;
    if (st) { *status = st; if (trace_len) *trace_len = 0; return 0; }

    int64_t tau = tau_in > 0 ? tau_in : derive_tau(c, D, k_target);
    if (tau_out) *tau_out = tau;
    int64_t *cap = (int64_t *)malloc(sizeof(int64_t) * c->n_inst);
    for (int r = 0; r < c->n_inst; r++) cap[r] = inst_cap(&c->inst[r], tau, granule);

    int64_t *Drem = (int64_t *)malloc(sizeof(int64_t) * (size_t)N * N);
    int64_t *Dhat = (int64_t *)malloc(sizeof(int64_t) * (size_t)G * G);
    memcpy(Drem, D, sizeof(int64_t) * (size_t)N * N);
    int *src = (int *)malloc(sizeof(int) * N), *dst = (int *)malloc(sizeof(int) * N);
    int *src_b = (int *)malloc(sizeof(int) * N), *dst_b = (int *)malloc(sizeof(int) * N);
    int k = 0;
    for (;;) {
        int64_t left = 0;                                   /* ||D_rem||_1 */
        for (size_t e = 0; e < (size_t)N * N; e++) left += Drem[e];
        if (left == 0) break;
        if (k == k_max) { st |= VPO_ST_STEP_LIMIT; break; }
        for (int a = 0; a < G; a++)                         /* Eq. (5) */
            for (int d = 0; d < G; d++) {
                int64_t s = 0;
                for (int i = a * g; i < a * g + g; i++)
                    for (int j = d * g; j < d * g + g; j++) s += Drem[(size_t)i * N + j];
                Dhat[a * G + d] = s;
            }
        int best_shape = -1;                                /* Eq. (6), first maximum */
        int64_t best_score = -1;
        for (int s = 0; s < c->n_shapes; s++) {
            int64_t score = 0;
            for (uint32_t e = c->shape_ptr[s]; e < c->shape_ptr[s + 1]; e++)
                score += Dhat[c->nnz[4 * e] * G + c->nnz[4 * e + 1]] * (int64_t)c->nnz[4 * e + 2];
            if (score > best_score) { best_score = score; best_shape = s; }
        }
        if (best_score <= 0) { st |= VPO_ST_UNCOVERED; break; }
        int fam_best = -1;
        int64_t F_b = 0, den_b = 1;
        for (uint32_t f = c->bucket_ptr[best_shape]; f < c->bucket_ptr[best_shape + 1]; f++) {
            int64_t F = multistart_aa(c, (int)f, Drem, cap, n_start, i_aa, src, dst, &tr, k);
            const uint16_t *fi = &c->fam_inst[(size_t)f * N];
            int64_t sum = 0, tmax = 0;                      /* Eq. (9), Eq. (10) */
            for (int r = 0; r < N; r++) {
                int64_t x = min64(cap[fi[r]], Drem[(size_t)src[r] * N + dst[r]]);
                int64_t t = x * (c->W / c->inst[fi[r]].bw);
                sum += x;
                if (t > tmax) tmax = t;
            }
            (void)F;                                        /* equals sum: credit and volume coincide */
            int64_t den = lambda_ns * c->W + tmax;
            if (sum == 0) den = 1;                          /* U = 0 */
            if (tr.trace && tr.len < tr.cap) {              /* (step, family, -1, sum x, W * duration) */
                int64_t *o = &tr.trace[5 * (size_t)tr.len++];
                o[0] = k; o[1] = (int64_t)f; o[2] = -1; o[3] = sum; o[4] = den;
            }
            int better = fam_best < 0 || (u128)sum * (u128)den_b > (u128)F_b * (u128)den;
            if (better) {
                fam_best = (int)f; F_b = sum; den_b = den;
                memcpy(src_b, src, sizeof(int) * N); memcpy(dst_b, dst, sizeof(int) * N);
            }
        }
        if (fam_best < 0 || F_b == 0) { st |= VPO_ST_NO_PROGRESS; break; }
        const uint16_t *fi = &c->fam_inst[(size_t)fam_best * N];
        chan_id[k] = fam_best;
        for (int r = 0; r < N; r++) {
            int i = src_b[r], j = dst_b[r];
            int64_t x = min64(cap[fi[r]], Drem[(size_t)i * N + j]);
            if (x > 0) {
                lane_dst[(size_t)k * N + i] = (int16_t)j;
                lane_inst[(size_t)k * N + i] = fi[r];
                lane_bytes[(size_t)k * N + i] = x;
                Drem[(size_t)i * N + j] -= x;
            }
        }
        k++;
    }
    *n_steps = k;
    *status = st;
    for (int s = 0; s < k_max; s++) {                       /* exclusive prefix sums over steps */
        for (int i = 0; i < N; i++)
            send_off[(size_t)(s + 1) * N + i] = send_off[(size_t)s * N + i] + lane_bytes[(size_t)s * N + i];
        if (!recv_off) continue;
        for (int j = 0; j < N; j++) recv_off[(size_t)(s + 1) * N + j] = recv_off[(size_t)s * N + j];
        for (int i = 0; i < N; i++) {
            int j = lane_dst[(size_t)s * N + i];
            if (j >= 0) recv_off[(size_t)(s + 1) * N + j] += lane_bytes[(size_t)s * N + i];
        }
    }
    if (trace_len) *trace_len = tr.len;
    free(cap); free(Drem); free(Dhat); free(src); free(dst); free(src_b); free(dst_b);
    return 0;
}

/* Batch driver: matrices b0 .. b1-1 of dense [B,...] arrays.  tau_in may be NULL. */
int vpo_schedule_batch(const vpo_catalog *c, const int64_t *D, const int64_t *tau_in, int b0, int b1,
                       int64_t lambda_ns, int k_target, int n_start, int i_aa, int64_t granule, int k_max,
                       int32_t *n_steps, int32_t *chan_id, int16_t *lane_dst, uint16_t *lane_inst,
                       int64_t *lane_bytes, int64_t *send_off, int64_t *recv_off, int64_t *tau_out,
                       int32_t *status)
{
    size_t N = (size_t)c->N, K = (size_t)k_max;
    for (int b = b0; b < b1; b++) {
        int rc = vpo_schedule(c, D + (size_t)b * N * N, tau_in ? tau_in[b] : 0, lambda_ns, k_target, n_start,
                              i_aa, granule, k_max, n_steps + b, chan_id + (size_t)b * K,
                              lane_dst + (size_t)b * K * N, lane_inst + (size_t)b * K * N,
                              lane_bytes + (size_t)b * K * N, send_off + (size_t)b * (K + 1) * N,
                              recv_off ? recv_off + (size_t)b * (K + 1) * N : NULL,
                              tau_out ? tau_out + b : NULL, status + b, NULL, 0, NULL);
        if (rc) return rc;
    }
    return 0;
}

/* ------------------------------------------------ plan-level quantities */

/*
 * Eq. (2) for a plan with per-activation overhead lambda_ns: returns
 * W * T_hat in nanoseconds (W = lcm of the path rates, so the value is an
 * integer): sum_k ( lambda*W + max_i x_ki * W / bw(p_ki) ).
 */
int64_t vpo_modeled_time_xW(const vpo_catalog *c, int n_steps, const int16_t *lane_dst,
                            const uint16_t *lane_inst, const int64_t *lane_bytes, int64_t lambda_ns)
{
    int N = c->N;
    int64_t total = 0;
    for (int k = 0; k < n_steps; k++) {
        int64_t tmax = 0;
        for (int i = 0; i < N; i++) {
            if (lane_dst[(size_t)k * N + i] < 0) continue;
            int64_t t = lane_bytes[(size_t)k * N + i] * (c->W / c->inst[lane_inst[(size_t)k * N + i]].bw);
            if (t > tmax) tmax = t;
        }
        total += lambda_ns * c->W + tmax;
    }
    return total;
}

int64_t vpo_rate_lcm(const vpo_catalog *c) { return c->W; }

/*
 * Validity of a plan against its demand (Section 3): every step feasible by
 * Eq. (1), every lane volume positive and at most cap (when cap_check),
 * and the steps summing to D exactly for every pair.  0 = valid, else
 * 100*step+reason for a bad step or -1 for a conservation failure.
 */
int vpo_check_plan(const vpo_catalog *c, const int64_t *D, int n_steps, const int16_t *lane_dst,
                   const uint16_t *lane_inst, const int64_t *lane_bytes, int64_t tau, int64_t granule)
{
    int N = c->N;
    int64_t *acc = (int64_t *)calloc((size_t)N * N, sizeof(int64_t));
    int rc = 0;
    for (int k = 0; k < n_steps && !rc; k++) {
        int f = vpo_lanes_feasible(c, lane_dst + (size_t)k * N, lane_inst + (size_t)k * N);
        if (f) { rc = 100 * k + f; break; }
        int active = 0;
        for (int i = 0; i < N; i++) {
            int j = lane_dst[(size_t)k * N + i];
            int64_t x = lane_bytes[(size_t)k * N + i];
            if (j < 0) { if (x != 0) rc = 100 * k + 6; continue; }
            if (x <= 0) { rc = 100 * k + 7; break; }
            if (tau > 0 && x > inst_cap(&c->inst[lane_inst[(size_t)k * N + i]], tau, granule)) { rc = 100 * k + 8; break; }
            acc[(size_t)i * N + j] += x;
            active++;
        }
        if (!rc && !active) rc = 100 * k + 9;
    }
    if (!rc && memcmp(acc, D, sizeof(int64_t) * (size_t)N * N) != 0) rc = -1;
    free(acc);
    return rc;
}

/* ------------------------------------------------------------- pack */

/*
 * Send-buffer pack for one rank (Section 5, "Device-resident buffer layout").
 * Copies routed to destination j != rank form stream_j in ascending
 * (token, slot).  Step k of the plan sends lane_bytes[k][rank] bytes to
 * lane_dst[k][rank]; its rows are the next rows of that destination's stream and
 * land at staged row send_off[k][rank] / row_bytes onwards.  src_map (optional)
 * receives token*topk+slot per staged row.  The plan arrays are one matrix's,
 * with row stride N.  Returns the status bits.
 */
int vpo_pack(const int32_t *n_steps, const int16_t *lane_dst, const int64_t *lane_bytes,
             const int64_t *send_off, int N, int rank, int k_max,
             const int32_t *expert_idx, int T, int topk, int experts_per_rank,
             const void *rows, int64_t row_bytes, void *staged, int64_t staged_capacity_bytes,
             int32_t *src_map)
{
    (void)k_max;
    int K = *n_steps, st = 0;
    if (send_off[(size_t)K * N + rank] > staged_capacity_bytes) return VPO_ST_PACK_CAPACITY;
    int64_t *len = (int64_t *)calloc((size_t)N, sizeof(int64_t));
    for (int64_t e = 0; e < (int64_t)T * topk; e++) {
        int x = expert_idx[e];
        if (x < 0) continue;
        int j = x / experts_per_rank;
        if (j >= N) { st |= VPO_ST_PACK_MISMATCH; continue; }
        if (j != rank) len[j]++;
    }
    int32_t **stream = (int32_t **)calloc((size_t)N, sizeof(int32_t *));
    int64_t *fill = (int64_t *)calloc((size_t)N, sizeof(int64_t));
    for (int j = 0; j < N; j++) stream[j] = (int32_t *)malloc(sizeof(int32_t) * (size_t)(len[j] + 1));
    for (int64_t e = 0; e < (int64_t)T * topk; e++) {
        int x = expert_idx[e];
        if (x < 0) continue;
        int j = x / experts_per_rank;
        if (j >= N || j == rank) continue;
        stream[j][fill[j]++] = (int32_t)e;
    }
    int64_t *cursor = (int64_t *)calloc((size_t)N, sizeof(int64_t));
    for (int k = 0; k < K; k++) {
        int j = lane_dst[(size_t)k * N + rank];
        if (j < 0) continue;
        int64_t bytes = lane_bytes[(size_t)k * N + rank];
        if (bytes % row_bytes) { st |= VPO_ST_PACK_MISMATCH; continue; }
        int64_t n = bytes / row_bytes, base = send_off[(size_t)k * N + rank] / row_bytes;
        for (int64_t p = 0; p < n; p++) {
            if (cursor[j] >= len[j]) { st |= VPO_ST_PACK_MISMATCH; break; }
            int32_t e = stream[j][cursor[j]++];
            memcpy((char *)staged + (size_t)(base + p) * row_bytes,
                   (const char *)rows + (size_t)(e / topk) * row_bytes, (size_t)row_bytes);
            if (src_map) src_map[base + p] = e;
        }
    }
    for (int j = 0; j < N; j++) {
        if (cursor[j] != len[j]) st |= VPO_ST_PACK_MISMATCH;
        free(stream[j]);
    }
    free(stream); free(fill); free(cursor); free(len);
    return st;
}

/* ------------------------------------------------- demand from routing */

/*
 * Demand rows from top-k routing (Section 6, "Workloads": demand matrices derived from top-k MoE
 * routing).  Source rank src0+s routes T tokens; copy (t, slot) goes to expert idx[s][t][slot], which lives
 * on rank idx / experts_per_rank; D[src][dst] = row_bytes x number of such copies, D[src][src] = 0
 * (Section 3).  Negative indices are dropped copies.  Returns 1 if an index addresses a rank >= N.
 */
int vpo_demand_from_routing(const int32_t *idx, int n_src, int T, int topk, int experts_per_rank, int N, int src0,
                            int64_t row_bytes, int64_t *rows)
{
    int bad = 0;
    memset(rows, 0, sizeof(int64_t) * (size_t)n_src * N);
    for (int s = 0; s < n_src; s++)
        for (int t = 0; t < T; t++)
            for (int k = 0; k < topk; k++) {
                int x = idx[((size_t)s * T + t) * topk + k];
                if (x < 0) continue;
                int j = x / experts_per_rank;
                if (j >= N) { bad = 1; continue; }
                if (j != src0 + s) rows[(size_t)s * N + j] += row_bytes;
            }
    return bad;
}

/* ---------------------------------------------------------- exchange */

/*
 * What the transport does between pack and unpack (Section 5, "Device-resident buffer layout": one contiguous
 * chunk per peer and activation).  Sender side for one rank: in step k the lane_bytes[k][rank] bytes at offset
 * send_off[k][rank] of its staged buffer go to rank j = lane_dst[k][rank], where they land at offset recv_off[k][j]
 * of j's receive buffer (recv_bufs[j]); arrived[j] (optional) counts the bytes delivered to j.  A chunk that would
 * overrun recv_capacity[j] is not copied and the function returns VPO_ST_PACK_CAPACITY.
 */
int vpo_exchange_put(const int32_t *n_steps, const int16_t *lane_dst, const int64_t *lane_bytes, const int64_t *send_off,
                     const int64_t *recv_off, int N, int rank, int k_max, const uint8_t *staged,
                     uint8_t *const *recv_bufs, const int64_t *recv_capacity, uint64_t *arrived)
{
    int K = *n_steps < 0 ? 0 : (*n_steps > k_max ? k_max : *n_steps);
    int st = 0;
    for (int k = 0; k < K; k++) {
        int j = lane_dst[(size_t)k * N + rank];
        int64_t n = lane_bytes[(size_t)k * N + rank];
        if (j < 0 || n <= 0) continue;
        int64_t from = send_off[(size_t)k * N + rank], to = recv_off[(size_t)k * N + j];
        if (to + n > recv_capacity[j]) { st |= VPO_ST_PACK_CAPACITY; continue; }
        memcpy(recv_bufs[j] + to, staged + from, (size_t)n);
        if (arrived) arrived[j] += (uint64_t)n;
    }
    return st;
}

/* ------------------------------------------------------------ unpack */

/*
 * Receive side of the buffer layout (Section 5: "the receive kernel unpacks them directly into the
 * output layout").  Rank `rank` has received, for every step k in which some source i sends to it
 * (lane_dst[k][i] == rank; at most one such i), that step's rows at byte offset recv_off[k][rank] of the
 * receive buffer; recv_expert[r] is the local expert (0 .. experts_per_rank-1) of received row r.  The
 * output is expert-major: all rows of local expert 0, then 1, ...; inside an expert by source rank, inside a
 * source in arrival order (which is the source's (token, slot) order).  expert_off[e] is the first output row of
 * expert e (expert_off[experts_per_rank] = total), out_src / out_map (optional) give each output row's source
 * rank and the received row it came from.  Returns status bits.
 */
int vpo_unpack(const int32_t *n_steps, const int16_t *lane_dst, const int64_t *recv_off, int N, int rank, int k_max,
               const void *recv, int64_t row_bytes, int64_t capacity_rows, const int32_t *recv_expert,
               int experts_per_rank, void *out, int32_t *expert_off, int32_t *out_src, int32_t *out_map)
{
    (void)k_max;
    int K = *n_steps, st = 0;
    int64_t total = recv_off[(size_t)K * N + rank];
    for (int e = 0; e <= experts_per_rank; e++) expert_off[e] = 0;
    if (total % row_bytes) st |= VPO_ST_PACK_MISMATCH;
    int64_t R = total / row_bytes;
    if (R > capacity_rows) return st | VPO_ST_PACK_CAPACITY;
    int *src_of = (int *)malloc(sizeof(int) * (size_t)(R + 1));
    for (int64_t r = 0; r < R; r++) src_of[r] = -1;
    for (int k = 0; k < K; k++) {
        int64_t lo = recv_off[(size_t)k * N + rank], hi = recv_off[(size_t)(k + 1) * N + rank];
        if (hi == lo) continue;
        if (lo % row_bytes || hi % row_bytes) { st |= VPO_ST_PACK_MISMATCH; continue; }
        int src = -1;
        for (int i = 0; i < N; i++) if (lane_dst[(size_t)k * N + i] == rank) src = i;
        for (int64_t r = lo / row_bytes; r < hi / row_bytes; r++) src_of[r] = src;
    }
    int64_t o = 0;
    for (int e = 0; e < experts_per_rank; e++) {
        expert_off[e] = (int32_t)o;
        for (int i = 0; i < N; i++)
            for (int64_t r = 0; r < R; r++) {
                if (src_of[r] != i || recv_expert[r] != e) continue;
                memcpy((char *)out + (size_t)o * row_bytes, (const char *)recv + (size_t)r * row_bytes, (size_t)row_bytes);
                if (out_src) out_src[o] = i;
                if (out_map) out_map[o] = (int32_t)r;
                o++;
            }
    }
    expert_off[experts_per_rank] = (int32_t)o;
    if (o != R) st |= VPO_ST_PACK_MISMATCH;      /* a row with an expert id out of range or without a source */
    free(src_of);
    return st;
}

/* ------------------------------------------------------------ return direction */

/*
 * Receive side of the RETURN AlltoAllv (Section 1: expert parallelism "dispatches activations to experts and
 * returns their outputs"; Section 5: "the receive kernel unpacks them directly into the output layout").
 * The return call carries demand D^T and has a plan of its own (n_steps, lane_dst, lane_bytes, recv_off below
 * are that plan's).  Rank `rank` routed copies (t, slot) to experts expert_idx[t][slot]; the rank j that hosts
 * an expert sends the outputs back in its expert-major order, i.e. for source `rank`: by expert id, then by
 * (t, slot).  In step k of the return plan the one sender j with lane_dst[k][j] == rank delivers the next
 * lane_bytes[k][j] / row_bytes rows of that stream at byte offset recv_off[k][rank] of the receive buffer.
 * The output layout is the token layout: out row t*topk+slot receives the output of copy (t, slot); rows of
 * local or dropped copies are left alone.  out_map (optional, [T*topk]) receives the receive-buffer row of each
 * copy, -1 for copies that do not travel.  Returns status bits.
 */
int vpo_unpack_tokens(const int32_t *n_steps, const int16_t *lane_dst, const int64_t *lane_bytes, const int64_t *recv_off,
                      int N, int rank, int k_max, const int32_t *expert_idx, int T, int topk, int experts_per_rank,
                      const void *recv, int64_t row_bytes, int64_t capacity_rows, void *out, int32_t *out_map)
{
    (void)k_max;
    int K = *n_steps, st = 0;
    int64_t copies = (int64_t)T * topk;
    if (out_map) for (int64_t c = 0; c < copies; c++) out_map[c] = -1;
    if (recv_off[(size_t)K * N + rank] > capacity_rows * row_bytes) return VPO_ST_PACK_CAPACITY;
    int64_t *order = (int64_t *)malloc(sizeof(int64_t) * (size_t)(copies + 1));
    for (int j = 0; j < N; j++) {
        if (j == rank) continue;
        /* stream of sender j: this rank's copies to j by (expert id, t, slot) */
        int64_t n = 0;
        for (int e = j * experts_per_rank; e < (j + 1) * experts_per_rank; e++)
            for (int64_t c = 0; c < copies; c++)
                if (expert_idx[c] == e) order[n++] = c;
        int64_t pos = 0;
        for (int k = 0; k < K; k++) {
            if (lane_dst[(size_t)k * N + j] != rank) continue;
            int64_t bytes = lane_bytes[(size_t)k * N + j], at = recv_off[(size_t)k * N + rank];
            if (bytes % row_bytes || at % row_bytes) { st |= VPO_ST_PACK_MISMATCH; continue; }
            for (int64_t r = 0; r < bytes / row_bytes; r++, pos++) {
                if (pos >= n) { st |= VPO_ST_PACK_MISMATCH; continue; }
                int64_t row = at / row_bytes + r;
                memcpy((char *)out + (size_t)order[pos] * row_bytes, (const char *)recv + (size_t)row * row_bytes, (size_t)row_bytes);
                if (out_map) out_map[order[pos]] = (int32_t)row;
            }
        }
        if (pos != n) st |= VPO_ST_PACK_MISMATCH;
    }
    free(order);
    return st;
}
