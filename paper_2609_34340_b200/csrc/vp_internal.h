// Internal declarations shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "variopath.h"

#define VP_MAX_CLASSES 8          // distinct path rates in one catalog
#define VP_MAX_GROUP 4            // ranks per group handled by the permutation search
#define VP_MAX_N 256
#define VP_ENTRY_LIMIT ((int64_t)1 << 40)

// Device-side view of a catalog; every pointer is device memory owned by vp_catalog.
struct DevCat {
    int N, G, g, S, P;            // ranks, groups, group size, groups per node, nodes
    int n_inst, n_shapes, n_families, n_res, n_classes;
    int sym;                      // 1: shape terms index per-node-offset sums, 0: D-hat cells
    int tbl_size;                 // entries of the score table (G*G or P*S*S)
    int max_bucket;
    // Eq. (6): shape s has terms term[s*max_terms .. s*max_terms + max_terms) = 8 * table index | count << 16
    // (shapes with fewer terms are padded with zero counts)
    const uint32_t* term;
    const uint32_t* term_t;       // the same, transposed: term e of shape s at term_t[e * ((n_shapes + 31) & ~31) + s]
    int max_terms;
    // Row patterns (node-symmetric catalogs): the terms of a shape whose source group is rail q of node 0 form the
    // shape's row q; Eq. (6) is the sum of its S row scores, and distinct rows are few (127 per rail for 4,095 shapes on
    // 32 nodes).  pat_term[p * max_row_terms + t] = table index | count << 16 (zero padded) lists the terms of row
    // pattern p; shape_pat[w * ((n_shapes + 31) & ~31) + s] holds the pattern ids of rows 2w and 2w + 1 of shape s
    // (16 bits each).  Null unless there are fewer than 65,536 patterns.
    const uint32_t* pat_term;
    const uint32_t* shape_pat;
    int n_patterns, max_row_terms;
    // Class decomposition of the arg-max (two rails): the shapes with first row p0 are consecutive, starting at shape
    // run_start(p0), and first rows of one class share the list of second rows that complete them, in shape order, so
    // shape(p0, p1) = run_start(p0) + place of p1 in the list of p0's class.  Unit 2 cl holds the first rows of class cl,
    // unit 2 cl + 1 its second rows, each padded to whole chunks of 32 entries.  dec[0] = chunks, dec[1] = words per
    // entry, dec[2] = offset of the entries, dec[3 .. 3 + 2 n] = first chunk of every unit, then the unit of every chunk; an entry is the row's terms
    // (table index | count << 16, zero padded) followed by its tie-break word: run_start for a first row, place for a second row (all ones marks padding).  Null
    // when the catalog has no such structure.
    const uint32_t* dec;
    int dec_classes, dec_words;
    const uint32_t* bucket_ptr;
    // family f, slot r: instance id | destination group << 16 | rate class << 24
    const uint32_t* fam_slot;
    // family f, slot r: rate class (the out-slots of group a are slots a*g .. a*g+g-1)
    const uint8_t* fam_cls;
    // family f, in-slot d*g+q of destination group d: slot index (N <= 256) | rate class << 8
    const uint16_t* fam_in;
    int n_terms;
    // inverted terms, for keeping the scores up to date instead of recomputing them: the shapes that use table
    // entry e are inv[inv_ptr[e] .. inv_ptr[e+1]) = shape | count << 16 (built when n_shapes < 65536)
    const uint32_t* inv_ptr;
    const uint32_t* inv;
    // quantum rule: resource l is forced for the D-hat cells forced_cell[forced_ptr[l] .. forced_ptr[l+1])
    const uint32_t* forced_ptr;
    const uint16_t* forced_cell;
    const uint32_t* forced_bw;
    // per path instance: rate_lcm / bw (Eq. 2 lane times are bytes x this, in 1/rate_lcm ns)
    const uint32_t* inst_wdiv;
    int64_t class_bw[VP_MAX_CLASSES];
    int64_t class_wdiv[VP_MAX_CLASSES];   // rate_lcm / bw
    int64_t bw_max, W;
};

// A launch shape worked out once per (catalog, batch class, parameters) and reused by later calls.
struct vp_launch_memo {
    int valid;
    int B_class;                  // min(B, CTAs of one wave + 1): batches of one class launch alike up to the grid size
    int32_t k_target, n_start, i_aa, k_max;
    int64_t lambda_ns, granule;
    unsigned char launch[160];    // the scheduler's Launch record
};

struct vp_catalog {
    int device;
    vp_info info;
    DevCat dc;
    std::vector<void*> allocs;
    int sm_count;
    int max_smem_optin;
    vp_launch_memo memo[4];
    int memo_next;
    // the host-buffer scheduler call's own copy stream and events (created on first use, see host_api.cu)
    std::vector<uint32_t> dec_host;   // host copy of DevCat::dec (vp_catalog_argmax_classes)
    cudaStream_t copy_stream;
    cudaEvent_t host_ev[4];
    int host_pipe_ready;
};

extern std::atomic<long long> g_vp_launches;

// Profiling hook: when enabled, records a CUDA event on `stream` before (edge 0) / after (edge 1)
// the kernels of one kind (0 schedule kernel, 1 pack index kernels, 2 pack copy kernel).
void vp_prof_mark(int kind, int edge, cudaStream_t stream);

static inline size_t vp_align256(size_t x) { return (x + 255) & ~(size_t)255; }
