/*
 * variopath.h - C ABI of the B200 (sm_100a) VarioPath online scheduler and
 * send-buffer pack.
 *
 * The library implements the demand-dependent half of the method: for every
 * AlltoAllv invocation, decompose the N x N integer demand matrix over an
 * offline catalog of contention-free channel families into a sequence of
 * channel activations (Algorithm 2, Section 4.2), and lay one rank's token rows
 * out in the send buffer in activation x destination order (Section 5,
 * "Device-resident buffer layout").  Everything runs in CUDA kernels on one
 * GPU; there is no CPU fallback.
 *
 * Conventions
 *  - Every call returns 0 (VP_OK) or a negative VP_E_* code; nothing throws,
 *    traps or aborts.  Per-matrix problems are reported as bit flags in
 *    status[b] (VP_ST_*), never by faulting.
 *  - "device" pointers are plain CUDA global-memory addresses on the
 *    catalog's device, owned by the caller; "host" pointers are ordinary host
 *    memory.  The library allocates device memory only in vp_load_catalog; all
 *    scratch is passed in by the caller (see the *_workspace_bytes calls).
 *  - Kernels are enqueued on the caller's stream (a cudaStream_t passed as
 *    void*; NULL = the default stream) and the device-pointer calls return
 *    without synchronising.
 *  - Ranks of group a are a*g .. a*g+g-1 (Section 4.1: N = G*g switch-local
 *    groups).  All volumes are bytes held in int64.
 *  - Results are deterministic: the same inputs give the same bytes whatever
 *    the batch size or launch geometry.
 */
#ifndef VARIOPATH_H
#define VARIOPATH_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- return codes ------------------------------------------------------ */
#define VP_OK               0
#define VP_E_BAD_ARG      (-1)  /* NULL pointer, non-positive size, parameter out of range      */
#define VP_E_BAD_CATALOG  (-2)  /* blob truncated / malformed, or violates Eq. (3) / Eq. (4)      */
#define VP_E_NOMEM        (-3)  /* host or device allocation failed in vp_load_catalog            */
#define VP_E_CUDA         (-4)  /* a CUDA runtime call failed; the extension may be unusable      */
#define VP_E_WORKSPACE    (-5)  /* workspace NULL, misaligned (256 B) or smaller than required    */
#define VP_E_UNSUPPORTED  (-6)  /* group size > 4, N > 256, more than 8 distinct path rates ...   */

/* ---- per-matrix status bits (status[b]); 0 = a complete valid schedule ---- */
#define VP_ST_NEGATIVE        1   /* some D_ij < 0                                               */
#define VP_ST_OVERFLOW_RISK   2   /* some D_ij >= 2^40                                           */
#define VP_ST_DIAG_NONZERO    4   /* some D_ii != 0 (Section 3: self traffic is omitted)          */
#define VP_ST_NOT_GRANULE     8   /* some D_ij not a multiple of granule_bytes                    */
#define VP_ST_BAD_TAU        16   /* tau_ns_in[b] < 0 or > 2^40                                   */
#define VP_ST_UNCOVERED      32   /* residual demand left but every shape scores 0 (Eq. 6)        */
#define VP_ST_NO_PROGRESS    64   /* best candidate carries 0 bytes (only if n_start < g)         */
#define VP_ST_STEP_LIMIT    128   /* k_max activations emitted, residual demand left              */
#define VP_ST_PACK_MISMATCH 256   /* vp_pack: routed copies disagree with the plan's byte counts  */
#define VP_ST_PACK_CAPACITY 512   /* vp_pack: staged buffer smaller than the plan's send volume   */
#define VP_ST_EXCHANGE_TIMEOUT 2048 /* vp_exchange_wait: the arrival counter did not reach the plan's byte count in max_polls polls */
/* Row-copy kernels (vp_pack, vp_pack_static, vp_unpack, vp_unpack_tokens): a bounded wait for an asynchronous
 * copy into shared memory gave up (2^22 polls; never seen in practice).  The kernel then issues no further
 * loads, lets the stores it already issued finish and returns; the output buffer is INCOMPLETE and the call
 * must be repeated.  Nothing faults and the context stays usable. */
#define VP_ST_INTERNAL_TIMEOUT (1 << 30)
/* Bits 1..16 reject the matrix before scheduling: n_steps[b] = 0 and an empty plan. */

typedef struct vp_catalog vp_catalog;   /* opaque, owned by the library */

typedef struct vp_info {
    int32_t N, G, g;              /* ranks, groups, ranks per group                              */
    int32_t groups_per_node;
    int32_t n_resources;          /* directed shared resources (the set U of Section 3)           */
    int32_t n_instances;          /* group-level path instances                                   */
    int32_t n_shapes, n_families; /* catalog size (Table 3 columns)                               */
    int32_t max_nnz;              /* largest number of non-zero group pairs of a shape            */
    int32_t max_bucket;           /* largest number of families realising one shape               */
    int32_t covered;              /* 1 if every group pair that can carry demand is in some shape */
    int32_t node_symmetric;       /* 1 if every shape is invariant under a shift of the node index:
                                     Eq. (6) is then evaluated on per-node-offset sums of D-hat   */
    int64_t rate_lcm;             /* lcm of all path rates (utilities are compared exactly)       */
    int32_t row_patterns;         /* node-symmetric catalogs: distinct rows (terms of a shape that leave
                                     one rail of node 0); 0 otherwise                              */
    int32_t argmax_classes;       /* two-rail node-symmetric catalogs whose shapes decompose into classes
                                     of first rows with a common list of second rows (see
                                     vp_catalog_argmax_classes): the number of classes; 0 otherwise */
} vp_info;

/*
 * Scheduler parameters (Algorithm 2 "Require": tau, lambda, N_start, I_AA;
 * Section 5 "Global execution granularity": K_target).
 */
typedef struct vp_sched_params {
    int64_t lambda_ns;      /* per-activation overhead of Eq. (2)/(10), 0 <= lambda < 2^40        */
    int64_t granule_bytes;  /* every D_ij must be a multiple; lane capacities are rounded down to
                               it (at least one granule).  Use the row size when packing.  >= 1   */
    int32_t k_target;       /* target round count, 0 -> 2N                                        */
    int32_t n_start;        /* AA starts, 0 -> g; start t rotates every group's in-slots by t      */
    int32_t i_aa;           /* AA sweep limit, 0 -> 3                                             */
    int32_t k_max;          /* capacity of the plan arrays in activations, > 0                    */
} vp_sched_params;

/*
 * vp_load_catalog - parse, validate and upload a topology + channel catalog
 * (Section 4.1: rank groups, path instances, shapes, families, buckets).
 *
 * topology, channels: host, little-endian blobs.
 *   topology: u32 magic 'VPTP', u32 version(1), u32 N, u32 G, u32 g,
 *     u32 groups_per_node, u32 n_resources, u32 n_instances; then per instance
 *     20 bytes: u16 src_group, u16 dst_group, u8 kind, u8 n_res (<=4), u16 mult
 *     (lanes of one family that may share it), u32 bw (bytes/ns), u16 res[4].
 *     Instance id = position; ids must be sorted by (src_group, dst_group).
 *   channels: u32 magic 'VPCH', u32 version(1), u32 N, u32 n_shapes,
 *     u32 n_families, u32 total_nnz; u32 shape_ptr[n_shapes+1]; total_nnz x
 *     {u16 a, u16 d, u16 count, u16 pad}; u32 bucket_ptr[n_shapes+1] (families
 *     of shape s are ids bucket_ptr[s]..bucket_ptr[s+1]-1, in tie-break order);
 *     u16 fam_inst[n_families][N] ascending instance ids.
 * Rejected with VP_E_BAD_CATALOG: a shape whose row or column sums differ from
 * g (Eq. 3); a family that does not select exactly M_ad instances per group
 * pair, repeats an instance beyond mult, or uses a directed resource twice
 * (Eq. 4).  A catalog that leaves a group pair uncovered loads (info.covered
 * = 0); demand on that pair ends with VP_ST_UNCOVERED.
 * device: CUDA device ordinal that will hold the image, or -1 for a host-only
 * handle: the blobs are parsed, validated and analysed as usual, nothing is
 * uploaded, vp_catalog_info and vp_catalog_argmax_classes work, and every call
 * that would launch a kernel returns VP_E_BAD_ARG.  *out receives the handle,
 * to be released with vp_free_catalog.  Synchronous.
 */
int vp_load_catalog(const void* topology, size_t topology_bytes,
                    const void* channels, size_t channels_bytes,
                    int device, vp_catalog** out);
void vp_free_catalog(vp_catalog* catalog);
int vp_catalog_info(const vp_catalog* catalog, vp_info* out);

/*
 * The catalog's class decomposition of Eq. (6)'s arg-max, as the scheduler kernel for large catalogs uses it (host
 * call; for tests and tools).  In a two-rail node-symmetric catalog a shape is a pair (first row, second row).  When
 * the shapes that share a first row are consecutive and first rows fall into few classes with one common list of
 * second rows, the shape of (first row p0, second row at place j of the list of p0's class) is run_start(p0) + j, and
 * the first maximum over all shapes is the best of the classes' (first maximal p0, first maximal second row).
 * out (host, capacity_words 32-bit words; may be NULL to query) receives: [0] chunks, [1] words per entry, [2] offset
 * of the entries, [3 .. 3 + 2n] the first chunk of every unit (unit 2c = the first rows of class c, unit 2c + 1 its
 * second rows; a chunk is 32 entries), then the unit of every chunk; an entry is the row's terms (table index |
 * lane count << 16, zero padded; table index of (node offset delta, rail q, rail q') = (delta S + q) S + q') followed
 * by its tie-break word: run_start for a first row, the place for a second row, all ones for padding.
 * *words_needed receives the length; 0 when the catalog has no such structure.  VP_E_WORKSPACE if out is too small.
 */
int vp_catalog_argmax_classes(const vp_catalog* catalog, uint32_t* out, size_t capacity_words, size_t* words_needed);

/*
 * vp_build_template_catalog - a node-symmetric catalog for many nodes (host code, no GPU work; no counterpart in the
 * paper, whose Algorithm 1 enumerates every family and grows exponentially with the node count).  One per-node
 * template is applied to every node: each of the two switch-local groups q of a node gets a network target "none" or
 * (delta, q2) = group q2 of node (n + delta) mod P (delta = 0 needs q2 != q; the two groups use different q2) and one
 * flag per direction of the path between the two sibling groups; a group sends as many such lanes as it receives and
 * switch-local lanes fill the rest of its g slots.  Every family satisfies Eq. (3) / Eq. (4) and is invariant under a
 * shift of the node index (vp_info.node_symmetric = 1).  Arguments and results as for vp_build_catalog; the topology
 * must have two groups per node with instance kinds 0 (switch-local), 1 (sibling) and 2 (network), else
 * VP_E_UNSUPPORTED.  8 nodes: 255 shapes / 272 families; 32 nodes: 4095 / 4160.
 */
int vp_build_template_catalog(const void* topology, size_t topology_bytes, void* channels_out, size_t capacity_bytes,
                              size_t* bytes_needed, int32_t* n_shapes_out, int32_t* n_families_out);

/*
 * vp_prune_paths - the path filter that precedes the search, PrunePaths of Section 4.1 ("Pruning and search cost";
 * host code): a path instance is dropped when another instance of the same group pair uses a subset of its directed
 * resources at a rate that is not lower, one of the two strictly.  topology: a topology blob (layout under
 * vp_load_catalog) holding the candidate instances; topology_out receives the same blob with the surviving
 * instances in their original order.  *bytes_needed is always set; with topology_out == NULL only the size and
 * *n_kept_out are computed; VP_E_WORKSPACE if capacity_bytes is too small.
 */
int vp_prune_paths(const void* topology, size_t topology_bytes, void* topology_out, size_t capacity_bytes,
                   size_t* bytes_needed, int32_t* n_kept_out);

/*
 * vp_build_catalog - offline catalog construction, Algorithm 1 of Section 4.1 (host code, no GPU work).
 *
 * Enumerates, by the pruned binary depth-first search of Algorithm 1 (CanAdd: resource disjointness and the
 * per-group degree limit g; SuffixOK; Complete), every multiset of the topology's path instances that gives
 * each group exactly g outgoing and g incoming lanes without using a directed resource twice, groups the
 * families by shape, applies PruneFamilies (duplicates; same footprints with no lower and somewhere higher
 * rates) and serialises the result as a channels blob (layout under vp_load_catalog; shapes ordered by their
 * sorted (a, d, count) lists, families by instance-id list).  The search is exponential in the number of
 * instances (Section 4.1): it is meant for one or two nodes; more than 2^22 families gives VP_E_UNSUPPORTED.
 *
 * topology: host blob (layout under vp_load_catalog; apply PrunePaths before serialising it).
 * channels_out: host buffer of capacity_bytes, or NULL to query the size.  *bytes_needed always receives the
 * blob size; n_shapes_out / n_families_out (may be NULL) the catalog size (the columns of Table 3).
 * Returns VP_E_WORKSPACE if the buffer is too small, VP_E_BAD_CATALOG for a malformed topology or one that
 * admits no family at all.
 */
int vp_build_catalog(const void* topology, size_t topology_bytes, void* channels_out, size_t capacity_bytes,
                     size_t* bytes_needed, int32_t* n_shapes_out, int32_t* n_families_out);

/* Bytes of device scratch vp_schedule_batch needs for a batch of B (multiple of 256). */
size_t vp_schedule_workspace_bytes(const vp_catalog* catalog, int B, const vp_sched_params* params);

/*
 * vp_schedule_batch - Algorithm 2 for B independent demand matrices.
 *
 * Per matrix: tau from K_target unless given; D_rem <- D; repeat { group sums
 * (Eq. 5); first shape of maximal score (Eq. 6); for every family of its bucket
 * MultiStartAA endpoint binding (Eq. 7, 8) and Evaluate (Eq. 9, 10); emit the
 * first family of maximal utility; D_rem -= X(E) } until D_rem = 0; then
 * exclusive prefix sums of the per-rank send / receive bytes over the steps.
 *
 * All array arguments are device pointers, row-major, caller-owned:
 *   demand      [B][N][N] int64 bytes from rank i to rank j, zero diagonal
 *   tau_ns_in   [B] or NULL; entries > 0 override the derived time quantum
 *   n_steps     [B]            activations emitted
 *   chan_id     [B][k_max]     global family index of step k, -1 beyond n_steps
 *   lane_dst    [B][k_max][N]  destination of source rank i in step k, -1 = idle
 *   lane_inst   [B][k_max][N]  path-instance id of that lane, 0xFFFF = idle
 *   lane_bytes  [B][k_max][N]  bytes for the pair (i, lane_dst), 0 = idle
 *   send_off    [B][k_max+1][N] bytes rank i has sent before step k
 *   recv_off    [B][k_max+1][N] bytes rank j has received before step k; may be NULL
 *   tau_ns_out  [B] quantum used; may be NULL
 *   status      [B] VP_ST_* bits
 * Every element of every output array is written (rows beyond n_steps hold the
 * idle values; offset rows beyond n_steps repeat the totals).
 * workspace: device, 256-byte aligned, >= vp_schedule_workspace_bytes; contents
 * are scratch (see vp_schedule_read_stats for the counters it keeps).  Calls
 * sharing a workspace must be stream-ordered.
 */
int vp_schedule_batch(const vp_catalog* catalog, const vp_sched_params* params,
                      const int64_t* demand, const int64_t* tau_ns_in, int B,
                      int32_t* n_steps, int32_t* chan_id, int16_t* lane_dst, uint16_t* lane_inst,
                      int64_t* lane_bytes, int64_t* send_off, int64_t* recv_off,
                      int64_t* tau_ns_out, int32_t* status,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Bytes of device scratch vp_pack needs (multiple of 256). */
size_t vp_pack_workspace_bytes(int N, int T, int topk, int k_max);

/*
 * vp_pack - stage one rank's routed token rows in activation x destination
 * order (Section 5: "groups elements by destination rank and packs each peer's
 * ... payload contiguously into the ... send buffer").
 *
 * Copies (t, slot) with expert_idx >= 0 whose destination rank
 * j = expert_idx / experts_per_rank differs from `rank` form stream_j in
 * ascending (t, slot).  Step k of the plan sends lane_bytes[k][rank] bytes to
 * j = lane_dst[k][rank]: the next lane_bytes/row_bytes rows of stream_j, stored
 * at staged row send_off[k][rank]/row_bytes onwards.  One row per (token, slot);
 * copies to the rank itself are not staged (D_ii = 0).
 *
 * n_steps_b, lane_dst_b, lane_bytes_b, send_off_b: device pointers to ONE
 *   matrix's plan as written by vp_schedule_batch (row stride N).
 * expert_idx [T][topk] int32 device; < 0 = dropped copy.
 * rows       [T][row_bytes] device.  staged: device, staged_capacity_bytes long.
 *   When rows, staged and row_bytes are multiples of 16 the copy uses bulk
 *   asynchronous (TMA) transfers; otherwise a plain-load path.
 * src_map    [staged_capacity_bytes/row_bytes] int32 device or NULL: receives
 *   t*topk+slot for each staged row; rows not written keep their content.
 * status     device int32[1]: VP_ST_PACK_MISMATCH if the routed copies per
 *   destination differ from the plan (copies beyond the plan are not staged),
 *   VP_ST_PACK_CAPACITY if send_off[n_steps][rank] > capacity (nothing copied).
 * workspace: device, 256-byte aligned, >= vp_pack_workspace_bytes.
 */
int vp_pack(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* lane_bytes_b,
            const int64_t* send_off_b, int N, int rank, int k_max,
            const int32_t* expert_idx, int T, int topk, int experts_per_rank,
            const void* rows, int64_t row_bytes,
            void* staged, int64_t staged_capacity_bytes, int32_t* src_map,
            int32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * vp_pack_static - vp_pack without a workspace argument.  (The paper has no counterpart: this entry
 * point exists for callers that cannot provide scratch memory.)
 *
 * Who needs it: code that runs the pack from inside a serving engine's steady-state step.  Such code is
 * given the input and output buffers and nothing else; it owns no allocator, and calling cudaMalloc there
 * is off the table (the call synchronises the whole device, may fail under the engine's memory cap, and
 * bypasses the engine's own accounting).  For these callers the library carries its own scratch: one
 * block of VP_PACK_STATIC_SCRATCH_BYTES of device memory per GPU, which the CUDA runtime sets aside when the
 * library's pack code is first used on that GPU (with lazy module loading that can be inside the first
 * vp_pack_static call itself) and keeps until the process exits.  Calls after the first one on a device
 * allocate nothing, on host or device.
 *
 * Arguments, results and status bits are those of vp_pack; inputs and outputs are still the caller's.
 * Limits and rules:
 *  - vp_pack_workspace_bytes(N, T, topk, k_max) must not exceed VP_PACK_STATIC_SCRATCH_BYTES (4 MiB; about
 *    0.9 million routed copies at N = 16); a larger problem is refused with VP_E_WORKSPACE before anything
 *    is launched.  Use vp_pack with your own workspace for those.
 *  - The first call on each device looks up the block's device address (a cudaGetSymbolAddress query made
 *    with that device current).  Make that first call outside any stream capture.
 *  - All calls on one device share the one block, and the block keeps whatever the last call left in it.
 *    The call itself resets what has to start from zero, so stale contents are harmless, but two calls
 *    whose kernels can overlap on the GPU (different streams without ordering between them) race on the
 *    block: order them, or give one of them vp_pack and a workspace of its own.
 */
#define VP_PACK_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
int vp_pack_static(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* lane_bytes_b,
                   const int64_t* send_off_b, int N, int rank, int k_max,
                   const int32_t* expert_idx, int T, int topk, int experts_per_rank,
                   const void* rows, int64_t row_bytes,
                   void* staged, int64_t staged_capacity_bytes, int32_t* src_map,
                   int32_t* status, void* cuda_stream);

/*
 * Host-buffer variants: the same operations with every array in HOST memory
 * (pinned memory makes the copies asynchronous).  The calls copy inputs to
 * device scratch, run the kernels above, copy the results back and return
 * after synchronising the stream.  device_scratch must hold
 * vp_schedule_host_scratch_bytes / vp_pack_host_scratch_bytes bytes.
 *
 * A scheduler batch of 64 matrices or more is worked through in chunks of about one matrix per SM (at least three
 * chunks), two chunks in flight inside the same scratch: one is decomposed on cuda_stream while the results of the
 * chunk before it are copied to the host on a second stream that the catalog handle owns (created on first use, freed
 * with the handle).  The results are the same as for one chunk; the call still returns only when everything is in
 * host memory.  Host-buffer calls that share a catalog handle must not run concurrently.
 */
size_t vp_schedule_host_scratch_bytes(const vp_catalog* catalog, int B, const vp_sched_params* params);
int vp_schedule_batch_host(const vp_catalog* catalog, const vp_sched_params* params,
                           const int64_t* demand, const int64_t* tau_ns_in, int B,
                           int32_t* n_steps, int32_t* chan_id, int16_t* lane_dst, uint16_t* lane_inst,
                           int64_t* lane_bytes, int64_t* send_off, int64_t* recv_off,
                           int64_t* tau_ns_out, int32_t* status,
                           void* device_scratch, size_t device_scratch_bytes, void* cuda_stream);
/*
 * vp_schedule_batch_host_used - vp_schedule_batch_host that brings back only what a plan uses: of every matrix b the
 * rows k < n_steps[b] of chan_id, lane_dst, lane_inst and lane_bytes and the rows k <= n_steps[b] of send_off / recv_off
 * (row n_steps[b] holds the totals).  Rows beyond keep whatever the host buffers held.  With k_max sized for the
 * longest plan this is a small part of the arrays (config 4: 26 GB instead of 122 GB per 4096 matrices).  Same
 * arguments, scratch and errors as vp_schedule_batch_host; it synchronises the stream once more (to read n_steps).
 */
int vp_schedule_batch_host_used(const vp_catalog* catalog, const vp_sched_params* params,
                                const int64_t* demand, const int64_t* tau_ns_in, int B,
                                int32_t* n_steps, int32_t* chan_id, int16_t* lane_dst, uint16_t* lane_inst,
                                int64_t* lane_bytes, int64_t* send_off, int64_t* recv_off,
                                int64_t* tau_ns_out, int32_t* status,
                                void* device_scratch, size_t device_scratch_bytes, void* cuda_stream);
size_t vp_pack_host_scratch_bytes(int N, int T, int topk, int k_max, int64_t row_bytes,
                                  int64_t staged_capacity_bytes);
int vp_pack_host(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* lane_bytes_b,
                 const int64_t* send_off_b, int N, int rank, int k_max,
                 const int32_t* expert_idx, int T, int topk, int experts_per_rank,
                 const void* rows, int64_t row_bytes,
                 void* staged, int64_t staged_capacity_bytes, int32_t* src_map,
                 int32_t* status, void* device_scratch, size_t device_scratch_bytes, void* cuda_stream);

/*
 * vp_plan_time - modeled completion time of each plan of a batch, Eq. (2) of Section 3:
 *   T(S) = sum_k ( lambda + max_i x_ki / bw(p_ki) ).
 * To stay in integers the result is scaled by rate_lcm (vp_info): time_xw[b] = rate_lcm * T(S_b) in
 * nanoseconds.  Inputs are the device arrays vp_schedule_batch wrote (same B, k_max); time_xw is device
 * int64[B].  Only steps below n_steps[b] count.
 */
int vp_plan_time(const vp_catalog* catalog, int B, int k_max, const int32_t* n_steps, const uint16_t* lane_inst,
                 const int64_t* lane_bytes, int64_t lambda_ns, int64_t* time_xw, void* cuda_stream);

/*
 * vp_exchange_put / vp_exchange_wait - executing a plan over peer memory (Section 5, "Device-resident buffer layout":
 * one contiguous chunk per peer and activation in the send buffer; arrival signalled through device-resident counters
 * instead of a global barrier; two buffer slots alternate between invocations).  This is the step between vp_pack and
 * vp_unpack.
 *
 * vp_exchange_put, the sender side of rank `rank`: for every step k < n_steps with j = lane_dst[k][rank] >= 0 the bytes
 * [send_off[k][rank], send_off[k+1][rank]) of `staged` (device; what vp_pack wrote) are stored into
 * recv_bufs[j] + recv_off[k][j].  The plan pointers are one matrix's device arrays (row stride N), as for vp_pack.
 *   recv_bufs            device array [N] of device pointers: the receive buffer of every rank for the current slot.
 *                        Ordinary device memory when ranks share a GPU; peer-mapped memory of the other GPUs otherwise
 *                        (the kernel only issues ordinary loads and stores, never multicast or cluster-scope copies)
 *   recv_capacity_bytes  device int64 [N]: size of each receive buffer; a chunk that would overrun it is not copied and
 *                        VP_ST_PACK_CAPACITY is set in status
 *   arrived              device array [N] of pointers to uint64 counters (NULL array or NULL entries: no signalling):
 *                        after a part of a chunk has been stored and fenced system-wide its byte count is added to
 *                        *arrived[j] with a system-scope atomic.  A rank's counter ends at base + recv_off[n_steps][rank]
 *   status               device int32[1], bits are OR-ed in (not cleared)
 * The call only enqueues one kernel on cuda_stream of the current device; it never waits.
 *
 * vp_exchange_wait, the receiver side: one thread polls *arrived_counter (acquire, system scope) until it is at least
 * counter_base + recv_off[n_steps][rank], at most max_polls times 200 ns apart; if it is not, VP_ST_EXCHANGE_TIMEOUT is
 * OR-ed into status and the kernel returns -- it never spins unbounded, and the context stays usable.  Kernels enqueued
 * after it on the same stream (vp_unpack) then see the delivered bytes.  counter_base is the counter's value before this
 * invocation's puts (0 after a reset; counters may also be left to grow from invocation to invocation).
 *
 * Several ranks on ONE GPU: enqueue every rank's put before any wait (or puts and waits on one stream in that order);
 * kernels of one GPU must not wait for kernels that have not been enqueued before them.
 */
int vp_exchange_put(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* send_off_b, const int64_t* recv_off_b,
                    int N, int rank, int k_max, const void* staged, void* const* recv_bufs,
                    const int64_t* recv_capacity_bytes, uint64_t* const* arrived, int32_t* status, void* cuda_stream);
int vp_exchange_wait(const int32_t* n_steps_b, const int64_t* recv_off_b, int N, int rank, int k_max,
                     const uint64_t* arrived_counter, uint64_t counter_base, uint32_t max_polls, int32_t* status,
                     void* cuda_stream);

/*
 * vp_sweep_plan_time - plan quality over a grid of parameters: for every pair (lambda_ns[i], k_target[j]) the batch
 * is decomposed with those two parameters in place of params' (Algorithm 2; Section 5 "Global execution
 * granularity": K_target sets the time quantum) and Eq. (2) is evaluated with that lambda.  Results, device arrays
 * indexed [(i * n_k + j) * B + b]: time_xw = rate_lcm x T(S_b) in nanoseconds, n_steps_out (may be NULL) the
 * activation counts, status_out (may be NULL) the per-matrix status bits.  lambda_ns and k_target are HOST arrays
 * (k_target 0 = 2N).  The plans themselves live in `workspace` (device, 256-byte aligned,
 * vp_sweep_workspace_bytes(catalog, B, params) bytes) and are overwritten from pair to pair.  Everything is
 * enqueued on cuda_stream; nothing is synchronised.
 */
size_t vp_sweep_workspace_bytes(const vp_catalog* catalog, int B, const vp_sched_params* params);
int vp_sweep_plan_time(const vp_catalog* catalog, const vp_sched_params* params, const int64_t* demand, int B,
                       const int64_t* lambda_ns, int n_lambda, const int32_t* k_target, int n_k, int64_t* time_xw,
                       int32_t* n_steps_out, int32_t* status_out, void* workspace, size_t workspace_bytes,
                       void* cuda_stream);

/*
 * vp_demand_from_routing - the demand rows of n_src source ranks from their top-k routing indices
 * (Section 6 "Workloads": demand matrices derived from top-k MoE routing; Section 3: D_ii = 0).
 *   expert_idx  device int32 [n_src][T][topk]; < 0 = dropped copy; expert e lives on rank e / experts_per_rank
 *   demand_rows device int64 [n_src][N]: row s is D[src0 + s][.] = row_bytes x copies to each destination,
 *               the entry for the source rank itself is 0.  Point it at &D[src0][0] of an N x N matrix.
 *   status      device int32[1]: 1 if some index addresses a rank >= N (that copy is ignored), else 0.
 */
int vp_demand_from_routing(const int32_t* expert_idx, int n_src, int T, int topk, int experts_per_rank, int N,
                           int src0, int64_t row_bytes, int64_t* demand_rows, int32_t* status, void* cuda_stream);

/* Bytes of device scratch vp_unpack needs (multiple of 256); 0 if the sizes are not supported. */
size_t vp_unpack_workspace_bytes(int N, int64_t capacity_rows, int experts_per_rank, int k_max);

/*
 * vp_unpack - the receive side of the buffer layout (Section 5: "the receive kernel unpacks them
 * directly into the output layout").
 *
 * In step k of the plan rank j receives, from its one sender i of that step (lane_dst[k][i] == j), the
 * rows stored at receive-buffer byte offset recv_off[k][j] onwards.  The output is expert-major: the rows
 * for local expert 0, then 1, ...; inside an expert by source rank; inside a source in arrival order
 * (which, with vp_pack on the sending side, is the sender's ascending (token, slot) order).
 *
 * n_steps_b, lane_dst_b, recv_off_b: device pointers to ONE matrix's plan (row stride N).
 * recv        [capacity_rows][row_bytes] device: the receive buffer; rows beyond
 *             recv_off[n_steps][rank] / row_bytes are ignored.
 * recv_expert [capacity_rows] int32 device: local expert id (0 .. experts_per_rank-1) of each received
 *             row (the metadata that travels beside the payload).
 * out         [capacity_rows][row_bytes] device; rows beyond the received count keep their content.
 * expert_off  [experts_per_rank + 1] int32 device: first output row of each local expert, then the total.
 * out_src, out_map [capacity_rows] int32 device or NULL: source rank and receive-buffer row of each
 *             output row.
 * status      device int32[1]: VP_ST_PACK_CAPACITY if more rows were received than capacity_rows
 *             (nothing is copied); VP_ST_PACK_MISMATCH if an offset is not a multiple of row_bytes, a
 *             received segment has no sender in the plan, or an expert id is out of range (that row is
 *             left out).
 * Limits: N * experts_per_rank <= 1024 and capacity_rows < 2^31, else VP_E_UNSUPPORTED.
 * workspace: device, 256-byte aligned, >= vp_unpack_workspace_bytes.
 */
int vp_unpack(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* recv_off_b,
              int N, int rank, int k_max,
              const void* recv, int64_t row_bytes, int64_t capacity_rows,
              const int32_t* recv_expert, int experts_per_rank,
              void* out, int32_t* expert_off, int32_t* out_src, int32_t* out_map,
              int32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Bytes of device scratch vp_unpack_tokens needs (multiple of 256); 0 if the sizes are not supported. */
size_t vp_unpack_tokens_workspace_bytes(int N, int T, int topk, int experts_per_rank, int64_t capacity_rows, int k_max);

/*
 * vp_unpack_tokens - receive side of the RETURN AlltoAllv (Section 1: expert parallelism "dispatches
 * activations to experts and returns their outputs"; Section 5: "the receive kernel unpacks them directly
 * into the output layout").
 *
 * The return call carries the transposed demand and has a plan of its own (vp_schedule_batch on D^T); the
 * plan arguments below are that plan's.  On the sending side each expert rank j stages its expert-major
 * rows (the output order of vp_unpack) with vp_pack, using topk = 1, experts_per_rank = 1 and the row's
 * source rank as its "expert index": the stream for destination i is then ordered by expert id, then by
 * i's own (token, slot).  Here rank i maps that stream back: in step k the one sender j with
 * lane_dst[k][j] == rank delivers the next lane_bytes[k][j] / row_bytes rows of its stream at byte offset
 * recv_off[k][rank]; the n-th row of j's stream belongs to the n-th of this rank's copies routed to j in
 * (expert id, token, slot) order, and is written to out row token*topk + slot.
 *
 * expert_idx  [T][topk] int32 device: this rank's routing (the one vp_pack dispatched with).
 * recv        [capacity_rows][row_bytes] device: the return receive buffer.
 * out         [T*topk][row_bytes] device: rows of copies that do not travel (dropped, or routed to this
 *             rank itself) keep their content.
 * out_map     [T*topk] int32 device or NULL: receive-buffer row of each copy, -1 if it does not travel.
 * status      device int32[1]: VP_ST_PACK_CAPACITY if recv_off[n_steps][rank] exceeds the buffer (nothing is
 *             unpacked); VP_ST_PACK_MISMATCH if a sender's rows differ in number from the copies routed to it
 *             or an offset is not a multiple of row_bytes.
 * Limits: N * experts_per_rank <= 1024, T*topk and capacity_rows < 2^31, else VP_E_UNSUPPORTED.
 */
int vp_unpack_tokens(const int32_t* n_steps_b, const int16_t* lane_dst_b, const int64_t* lane_bytes_b,
                     const int64_t* recv_off_b, int N, int rank, int k_max,
                     const int32_t* expert_idx, int T, int topk, int experts_per_rank,
                     const void* recv, int64_t row_bytes, int64_t capacity_rows,
                     void* out, int32_t* out_map,
                     int32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * How vp_schedule_batch would launch for a batch of B matrices (for benchmarks and tests): out4 (host) receives
 * {kernel, CTAs, threads per CTA, dynamic shared memory bytes}.  kernel 0 = one CTA per matrix; kernel 1 = one
 * warp per matrix (one, two or four warps per CTA as B grows), chosen for topologies of at most four groups of four
 * ranks when granule_bytes >= 256, and with smaller granules once B exceeds the number of CTAs that fit the GPU at
 * once; kernel 2 = one CTA per matrix with 16-bit saturating credits in shared memory, chosen
 * for node-symmetric catalogs of more than sixteen groups of four ranks (a second launch of kernel 0 then takes the
 * matrices whose capacities or totals do not fit that representation).  All kernels produce identical plans.
 * CTAs is also the number of matrices in flight at once: a caller that splits a large batch into sub-batches
 * wastes least when each sub-batch is several times this number (the CTAs pull matrices from a shared counter, so
 * only the last matrix of each CTA can leave the others waiting).
 */
int vp_schedule_launch_info(const vp_catalog* catalog, int B, const vp_sched_params* params, int32_t* out4);

/*
 * Peak-rate probes (no counterpart in the paper; measurement support for Section 4.2's operation counts).  Launches
 * one kernel on `cuda_stream` of the current device that keeps every warp slot of every SM busy with
 *   kind 0: 32-bit integer add + min on eight independent chains per thread (units = integer operations),
 *   kind 1: the same on 64-bit integers (units = 64-bit operations),
 *   kind 2 / 3: conflict-free 32-bit / 64-bit shared-memory loads (units = bytes loaded),
 * for `iters` loop iterations, and stores the number of units one launch performs in *units_per_launch (host).
 * The caller times the launch (CUDA events on the same stream) and divides.  `sink_device` is 8 bytes of device
 * memory that the kernel never writes in practice.  Returns VP_E_BAD_ARG for an unknown kind or iters <= 0.
 */
int vp_microbench(int kind, int iters, void* sink_device, int64_t* units_per_launch, void* cuda_stream);

/*
 * Write-only bandwidth probe (no counterpart in the paper): enqueues one cudaMemsetAsync of `bytes` zero bytes over
 * the caller's device buffer on `cuda_stream`; the caller times it.
 */
int vp_memset_probe(void* device_buffer, size_t bytes, void* cuda_stream);

/*
 * Work counters of the last vp_schedule_batch that used `workspace` (device): copies three
 * uint64 to host `out3` after synchronising the stream: activations emitted, (family, start)
 * binding tasks run, AA sweeps run over all tasks.  Used to count the algorithmic operations
 * of Section 4.2 "Planning complexity" for a measured batch.
 */
int vp_schedule_read_stats(const void* workspace, void* cuda_stream, uint64_t* out3);

/*
 * Per-kernel timing for benchmarks (off by default).  While enabled, every call records CUDA
 * events on the caller's stream around its own launches; vp_profile_read synchronises those
 * events, returns the summed device time and the number of timed launches of one kind since
 * the last read (kind 0: schedule kernel, 1: the three pack index kernels as a group, 2: the
 * pack copy kernel, 3: the unpack copy kernel) and discards them.  Creating events allocates driver resources.
 */
int vp_profile_enable(int on);
int vp_profile_read(int kind, double* total_ms, int64_t* launches);

/* Number of kernels the library has launched in this process (for launch accounting). */
int64_t vp_kernel_launch_count(void);

/* Static description of a VP_E_* code. */
const char* vp_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* VARIOPATH_H */
