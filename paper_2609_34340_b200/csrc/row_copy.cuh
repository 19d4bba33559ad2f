// Row copy shared by the pack and the unpack: every source row is read once and written to each of its
// destination rows (given by a row map, -1 = none).  Rows of at least 2 KB that are 16-byte aligned travel
// global -> shared -> global as bulk asynchronous copies (TMA): one warp per CTA drives a ring of
// shared-memory stages, an mbarrier per stage signals the load, the stores of a source row form one bulk
// group whose read completion frees the stage, and the mbarrier wait is bounded.  Other rows take a
// plain vector-load kernel.  Included by the translation units that launch it.
#pragma once
#include <cuda_runtime.h>

#include "bulk_copy.cuh"
#include "vp_internal.h"

namespace {

constexpr int kPiece = 16384;              // bytes per bulk transfer (rows longer than this are split)
constexpr int kMinBulkRow = 2048;          // shorter rows use the plain-load kernel
constexpr unsigned kSpinLimit = 1u << 22;  // bounded mbarrier wait

// One warp per CTA.  A "unit" is one piece (<= kPiece bytes) of one source row.  Units are dealt to CTAs round
// robin.  Unit u is loaded into stage u % S, kLook units ahead of its stores.  The destination rows of a unit
// (lane = slot, up to 32 slots per round) are fetched one unit ahead of the load that needs them and kept in
// registers until the unit's stores, so no global-memory latency sits between two bulk copies.
template <int S>
__global__ void __launch_bounds__(32)
pack_copy_bulk_kernel(const char* __restrict__ rows, char* __restrict__ staged, const int32_t* __restrict__ dst_row,
                      const int32_t* __restrict__ flags, int T, int topk, long long row_bytes, int pieces,
                      int32_t* __restrict__ status) {
    constexpr int kLook = S / 2;
    static_assert(kLook == 3, "the destination-row registers below form a ring of three");
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) unsigned long long bars[S];
    const int lane = threadIdx.x;
    if (flags[0]) return;
    const unsigned long long stream_policy = l2_evict_first_policy();
    if (lane == 0) {
        for (int s = 0; s < S; s++) mbar_init(smem_u32(&bars[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const long long units = (long long)T * pieces;
    const long long count = units > blockIdx.x ? (units - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int rounds = (topk + 31) / 32;            // destinations are handled 32 slots at a time
    const bool one_round = rounds == 1;
    unsigned phase = 0;                              // parity per stage (bit s)
    unsigned loaded = 0;                             // stage holds a load that was issued (bit s)
    bool failed = false;
    // destination row of this lane's slot: for the unit whose load is issued next (fetched), and for the three
    // units in flight (r2 newest .. r0 oldest); used when all slots fit one round
    int fetched = -1, r0 = -1, r1 = -1, r2 = -1;
    if (one_round && count > 0 && lane < topk) fetched = dst_row[(long long)(blockIdx.x / pieces) * topk + lane];
    for (long long it = 0; it < count + kLook && !failed; it++) {
        int rows_m = r0;                             // unit it - kLook
        r0 = r1; r1 = r2; r2 = -1;
        if (it < count) {                            // ---- issue the load of unit `it`
            const long long u = blockIdx.x + it * gridDim.x;
            const long long t = u / pieces;
            const int s = (int)(it % S);
            bool any = false;
            if (one_round) {
                r2 = fetched;
                any = fetched >= 0;
                fetched = -1;
                if (it + 1 < count && lane < topk) fetched = dst_row[((u + gridDim.x) / pieces) * topk + lane];
            } else {
                for (int r = 0; r < rounds; r++) {
                    const int slot = r * 32 + lane;
                    any |= slot < topk && dst_row[t * topk + slot] >= 0;
                }
            }
            any = __any_sync(0xffffffffu, any);
            bulk_wait_read<S - kLook - 1>();         // every lane: its stores that last read this stage are done
            __syncwarp();
            if (lane == 0) {
                if (any) {
                    const int p = (int)(u % pieces);
                    const unsigned bytes = (unsigned)min((long long)kPiece, row_bytes - (long long)p * kPiece);
                    const unsigned bar = smem_u32(&bars[s]);
                    mbar_expect_tx(bar, bytes);
                    bulk_load_stream(smem_u32(ring + (size_t)s * kPiece), rows + t * row_bytes + (long long)p * kPiece, bytes, bar, stream_policy);
                }
            }
            loaded = any ? (loaded | (1u << s)) : (loaded & ~(1u << s));
        }
        const long long m = it - kLook;
        if (m >= 0) {                                // ---- unit m: wait for its load, issue its stores
            const long long u = blockIdx.x + m * gridDim.x;
            const long long t = u / pieces;
            const int p = (int)(u % pieces);
            const int s = (int)(m % S);
            if (loaded & (1u << s)) {
                const unsigned bar = smem_u32(&bars[s]);
                unsigned spins = 0;
                while (!mbar_try_wait(bar, (phase >> s) & 1u)) {
                    if (++spins > kSpinLimit) { failed = true; break; }
                }
                failed = __any_sync(0xffffffffu, failed);
                phase ^= 1u << s;
                if (!failed) loaded &= ~(1u << s);   // this stage's load has landed
                if (!failed) {
                    const unsigned bytes = (unsigned)min((long long)kPiece, row_bytes - (long long)p * kPiece);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    if (one_round) {
                        if (rows_m >= 0)
                            bulk_store_stream(staged + (long long)rows_m * row_bytes + (long long)p * kPiece,
                                              smem_u32(ring + (size_t)s * kPiece), bytes, stream_policy);
                    } else {
                        for (int r = 0; r < rounds; r++) {
                            const int slot = r * 32 + lane;
                            const int row = slot < topk ? dst_row[t * topk + slot] : -1;
                            if (row >= 0)
                                bulk_store_stream(staged + (long long)row * row_bytes + (long long)p * kPiece,
                                                  smem_u32(ring + (size_t)s * kPiece), bytes, stream_policy);
                        }
                    }
                }
            }
            bulk_commit();                           // one group per unit from every lane, empty or not
        }
    }
    bulk_wait_all();                                 // stores must finish before shared memory is released
    if (failed) {
        // Give-up path: no further loads were issued.  Loads already in flight must not land in shared memory that
        // the next CTA owns, so each is given one more bounded wait (the stage whose wait gave up had its parity
        // flipped: put it back first).  Then the status bit tells the caller that the output is incomplete.
        for (int s = 0; s < S; s++) {
            if (!(loaded & (1u << s))) continue;
            unsigned spins = 0;
            while (!mbar_try_wait(smem_u32(&bars[s]), ((phase >> s) & 1u) ^ 1u) && !mbar_try_wait(smem_u32(&bars[s]), (phase >> s) & 1u) &&
                   ++spins < (1u << 18)) {
            }
        }
        if (lane == 0) atomicOr(status, VP_ST_INTERNAL_TIMEOUT);
    }
}

// Plain-load path (short or unaligned rows): one warp per token, V-byte vectors.
template <typename V>
__global__ void __launch_bounds__(256)
pack_copy_plain_kernel(const char* __restrict__ rows, char* __restrict__ staged, const int32_t* __restrict__ dst_row,
                       const int32_t* __restrict__ flags, int T, int topk, long long row_bytes) {
    if (flags[0]) return;
    const int lane = threadIdx.x & 31;
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
    const long long vecs = row_bytes / (long long)sizeof(V);
    for (long long t = warp; t < T; t += n_warps) {
        const V* src = (const V*)(rows + t * row_bytes);
        for (int s0 = 0; s0 < topk; s0 += 8) {
            int row[8];
            bool any = false;
#pragma unroll
            for (int s = 0; s < 8; s++) {
                row[s] = (s0 + s < topk) ? dst_row[t * topk + s0 + s] : -1;
                any |= row[s] >= 0;
            }
            if (!any) continue;
            for (long long v = lane; v < vecs; v += 32) {
                const V x = src[v];
#pragma unroll
                for (int s = 0; s < 8; s++)
                    if (row[s] >= 0) ((V*)(staged + (long long)row[s] * row_bytes))[v] = x;
            }
        }
    }
}


// Enqueue the copy of `n_src` source rows, each to its up to `fanout` destination rows dst_row[src * fanout + slot].
// `flags[0] != 0` (device) turns the copy into a no-op.  Returns VP_OK or VP_E_CUDA.
inline int launch_row_copy(const void* rows, void* out, const int32_t* dst_row, const int32_t* flags, int n_src, int fanout,
                           long long row_bytes, int32_t* status, cudaStream_t stream) {
    // per device, once: the SM count and the bulk kernel's shared-memory limit (kept out of the per-call path)
    static int s_sms[64] = {0};
    static bool s_attr_set[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return VP_E_CUDA;
    const bool cached = dev >= 0 && dev < 64;
    int sms = cached ? s_sms[dev] : 0;
    if (!sms) {
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return VP_E_CUDA;
        if (cached) s_sms[dev] = sms;
    }
    const bool aligned16 = row_bytes % 16 == 0 && ((uintptr_t)rows & 15) == 0 && ((uintptr_t)out & 15) == 0;
    if (aligned16 && row_bytes >= kMinBulkRow) {
        constexpr int S = 6;
        const int pieces = (int)((row_bytes + kPiece - 1) / kPiece);
        const size_t smem = (size_t)S * kPiece;
        if (!cached || !s_attr_set[dev]) {
            if (cudaFuncSetAttribute(pack_copy_bulk_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
                return VP_E_CUDA;
            if (cached) s_attr_set[dev] = true;
        }
        pack_copy_bulk_kernel<S><<<sms * 2, 32, smem, stream>>>((const char*)rows, (char*)out, dst_row, flags, n_src, fanout,
                                                                row_bytes, pieces, status);
    } else {
        const int grid = sms * 8;
        const uintptr_t mix = (uintptr_t)rows | (uintptr_t)out | (uintptr_t)row_bytes;
        if (mix % 16 == 0)
            pack_copy_plain_kernel<uint4><<<grid, 256, 0, stream>>>((const char*)rows, (char*)out, dst_row, flags, n_src, fanout, row_bytes);
        else if (mix % 4 == 0)
            pack_copy_plain_kernel<uint32_t><<<grid, 256, 0, stream>>>((const char*)rows, (char*)out, dst_row, flags, n_src, fanout, row_bytes);
        else
            pack_copy_plain_kernel<uint8_t><<<grid, 256, 0, stream>>>((const char*)rows, (char*)out, dst_row, flags, n_src, fanout, row_bytes);
    }
    g_vp_launches++;
    return cudaGetLastError() == cudaSuccess ? VP_OK : VP_E_CUDA;
}

}  // namespace
