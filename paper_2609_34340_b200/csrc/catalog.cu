// Catalog loader: parses the topology / channel blobs, validates them against
// Eq. (3) and Eq. (4) of Section 4.1 and builds the device image the kernels read.
#include <algorithm>
#include <cstring>
#include <map>
#include <new>

#include "vp_internal.h"

std::atomic<long long> g_vp_launches{0};

namespace {

struct Reader {
    const uint8_t* p;
    size_t n;
    bool ok = true;
    uint32_t u32(size_t off) {
        if (off + 4 > n) { ok = false; return 0; }
        return (uint32_t)p[off] | ((uint32_t)p[off + 1] << 8) | ((uint32_t)p[off + 2] << 16) | ((uint32_t)p[off + 3] << 24);
    }
    uint16_t u16(size_t off) {
        if (off + 2 > n) { ok = false; return 0; }
        return (uint16_t)(p[off] | (p[off + 1] << 8));
    }
    uint8_t u8(size_t off) {
        if (off + 1 > n) { ok = false; return 0; }
        return p[off];
    }
};

struct HostInst {
    int a, d, kind, mult, n_res, cls;
    int64_t bw;
    int res[4];
};

int64_t gcd_i64(int64_t a, int64_t b) {
    while (b) { int64_t t = a % b; a = b; b = t; }
    return a;
}

template <typename T>
int upload(vp_catalog* c, const std::vector<T>& v, const T** out) {
    if (c->device < 0) { *out = nullptr; return VP_OK; }     // host-only handle: nothing is uploaded
    void* d = nullptr;
    // sizes are rounded up to 16 bytes (zero filled) so that the kernels may stage whole arrays with bulk copies
    size_t bytes = (std::max<size_t>(v.size(), 1) * sizeof(T) + 15) & ~(size_t)15;
    if (cudaMalloc(&d, bytes) != cudaSuccess) return VP_E_NOMEM;
    c->allocs.push_back(d);
    if (cudaMemset(d, 0, bytes) != cudaSuccess) return VP_E_CUDA;
    if (!v.empty() && cudaMemcpy(d, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) return VP_E_CUDA;
    *out = (const T*)d;
    return VP_OK;
}

}  // namespace

extern "C" void vp_free_catalog(vp_catalog* c) {
    if (!c) return;
    int prev = -1;
    cudaGetDevice(&prev);
    if (c->device >= 0 && cudaSetDevice(c->device) == cudaSuccess) {
        for (void* p : c->allocs) cudaFree(p);
        if (c->host_pipe_ready) {
            cudaStreamDestroy(c->copy_stream);
            for (cudaEvent_t e : c->host_ev) cudaEventDestroy(e);
        }
    }
    if (prev >= 0) cudaSetDevice(prev);
    delete c;
}

extern "C" int vp_catalog_argmax_classes(const vp_catalog* c, uint32_t* out, size_t capacity_words, size_t* words_needed) {
    if (!c || !words_needed) return VP_E_BAD_ARG;
    *words_needed = c->dec_host.size();
    if (!out) return VP_OK;
    if (capacity_words < c->dec_host.size()) return VP_E_WORKSPACE;
    if (!c->dec_host.empty()) memcpy(out, c->dec_host.data(), c->dec_host.size() * sizeof(uint32_t));
    return VP_OK;
}

extern "C" int vp_catalog_info(const vp_catalog* c, vp_info* out) {
    if (!c || !out) return VP_E_BAD_ARG;
    *out = c->info;
    return VP_OK;
}

extern "C" int vp_load_catalog(const void* topology, size_t topo_bytes, const void* channels, size_t chan_bytes,
                               int device, vp_catalog** out) {
    if (!topology || !channels || !out || device < -1) return VP_E_BAD_ARG;
    *out = nullptr;
    Reader t{(const uint8_t*)topology, topo_bytes}, h{(const uint8_t*)channels, chan_bytes};
    if (t.u32(0) != 0x50545056u || t.u32(4) != 1 || !t.ok) return VP_E_BAD_CATALOG;
    if (h.u32(0) != 0x48435056u || h.u32(4) != 1 || !h.ok) return VP_E_BAD_CATALOG;
    const int N = (int)t.u32(8), G = (int)t.u32(12), g = (int)t.u32(16), S = (int)t.u32(20);
    const int n_res = (int)t.u32(24), n_inst = (int)t.u32(28);
    if (!t.ok || N <= 0 || G <= 0 || g <= 0 || (long long)G * g != N || n_inst <= 0 || n_res < 0) return VP_E_BAD_CATALOG;
    if (N > VP_MAX_N || g > VP_MAX_GROUP || n_inst > 0xFFFE || n_res > 0xFFFF) return VP_E_UNSUPPORTED;
    if (topo_bytes < 32 + (size_t)n_inst * 20) return VP_E_BAD_CATALOG;

    // ---- path instances (Section 4.1), rate classes, lcm of rates
    std::vector<HostInst> inst(n_inst);
    std::vector<int64_t> rates;
    int64_t W = 1, bw_max = 0;
    for (int r = 0; r < n_inst; r++) {
        size_t o = 32 + (size_t)r * 20;
        HostInst& q = inst[r];
        q.a = t.u16(o); q.d = t.u16(o + 2); q.kind = t.u8(o + 4); q.n_res = t.u8(o + 5);
        q.mult = t.u16(o + 6); q.bw = t.u32(o + 8);
        if (q.a >= G || q.d >= G || q.n_res > 4 || q.bw <= 0 || q.mult < 1) return VP_E_BAD_CATALOG;
        for (int k = 0; k < q.n_res; k++) {
            q.res[k] = t.u16(o + 12 + 2 * k);
            if (q.res[k] >= n_res) return VP_E_BAD_CATALOG;
        }
        if (r > 0 && (inst[r - 1].a > q.a || (inst[r - 1].a == q.a && inst[r - 1].d > q.d))) return VP_E_BAD_CATALOG;
        auto it = std::find(rates.begin(), rates.end(), q.bw);
        if (it == rates.end()) { rates.push_back(q.bw); q.cls = (int)rates.size() - 1; }
        else q.cls = (int)(it - rates.begin());
        if (rates.size() > VP_MAX_CLASSES) return VP_E_UNSUPPORTED;
        W = W / gcd_i64(W, q.bw) * q.bw;
        if (W >= ((int64_t)1 << 20)) return VP_E_UNSUPPORTED;
        bw_max = std::max(bw_max, q.bw);
    }

    // ---- shapes and families
    if ((int)h.u32(8) != N) return VP_E_BAD_CATALOG;
    const int n_shapes = (int)h.u32(12), n_fam = (int)h.u32(16), total_nnz = (int)h.u32(20);
    if (!h.ok || n_shapes <= 0 || n_fam <= 0 || total_nnz <= 0) return VP_E_BAD_CATALOG;
    const size_t off_sptr = 24, off_nnz = off_sptr + 4 * ((size_t)n_shapes + 1);
    const size_t off_bptr = off_nnz + 8 * (size_t)total_nnz, off_fam = off_bptr + 4 * ((size_t)n_shapes + 1);
    if (chan_bytes < off_fam + 2 * (size_t)n_fam * N) return VP_E_BAD_CATALOG;
    std::vector<uint32_t> shape_ptr(n_shapes + 1), bucket_ptr(n_shapes + 1);
    for (int s = 0; s <= n_shapes; s++) {
        shape_ptr[s] = h.u32(off_sptr + 4 * (size_t)s);
        bucket_ptr[s] = h.u32(off_bptr + 4 * (size_t)s);
    }
    if (shape_ptr[0] != 0 || (int)shape_ptr[n_shapes] != total_nnz || bucket_ptr[0] != 0 || (int)bucket_ptr[n_shapes] != n_fam)
        return VP_E_BAD_CATALOG;

    std::vector<int> M((size_t)G * G, 0), cnt((size_t)G * G, 0), used(n_res + 1, 0), times(n_inst, 0);
    std::vector<int> rowsum(G), colsum(G);
    std::vector<char> seen((size_t)G * G, 0);
    std::vector<uint32_t> fam_slot((size_t)n_fam * N);
    std::vector<uint8_t> fam_cls((size_t)n_fam * N);
    std::vector<uint16_t> fam_in((size_t)n_fam * N);
    int max_nnz = 0, max_bucket = 0;
    for (int s = 0; s < n_shapes; s++) {
        if (shape_ptr[s + 1] <= shape_ptr[s] || bucket_ptr[s + 1] < bucket_ptr[s]) return VP_E_BAD_CATALOG;
        max_nnz = std::max(max_nnz, (int)(shape_ptr[s + 1] - shape_ptr[s]));
        max_bucket = std::max(max_bucket, (int)(bucket_ptr[s + 1] - bucket_ptr[s]));
        std::fill(rowsum.begin(), rowsum.end(), 0);
        std::fill(colsum.begin(), colsum.end(), 0);
        for (uint32_t e = shape_ptr[s]; e < shape_ptr[s + 1]; e++) {
            int a = h.u16(off_nnz + 8 * (size_t)e), d = h.u16(off_nnz + 8 * (size_t)e + 2), m = h.u16(off_nnz + 8 * (size_t)e + 4);
            if (a >= G || d >= G || m == 0 || M[(size_t)a * G + d] != 0) return VP_E_BAD_CATALOG;
            M[(size_t)a * G + d] = m;
            rowsum[a] += m; colsum[d] += m;
            seen[(size_t)a * G + d] = 1;
        }
        for (int a = 0; a < G; a++)
            if (rowsum[a] != g || colsum[a] != g) return VP_E_BAD_CATALOG;                  // Eq. (3)
        for (uint32_t f = bucket_ptr[s]; f < bucket_ptr[s + 1]; f++) {                      // Eq. (4)
            int fill[VP_MAX_N] = {0};
            int prev = -1;
            for (int r = 0; r < N; r++) {
                int id = h.u16(off_fam + 2 * ((size_t)f * N + r));
                if (id >= n_inst || id < prev) return VP_E_BAD_CATALOG;
                prev = id;
                const HostInst& q = inst[id];
                if (q.a != r / g) return VP_E_BAD_CATALOG;
                if (++cnt[(size_t)q.a * G + q.d] > M[(size_t)q.a * G + q.d]) return VP_E_BAD_CATALOG;
                if (++times[id] > q.mult) return VP_E_BAD_CATALOG;
                for (int k = 0; k < q.n_res; k++)
                    if (used[q.res[k]]++) return VP_E_BAD_CATALOG;
                if (fill[q.d] >= g) return VP_E_BAD_CATALOG;
                fam_slot[(size_t)f * N + r] = (uint32_t)id | ((uint32_t)q.d << 16) | ((uint32_t)q.cls << 24);
                fam_cls[(size_t)f * N + r] = (uint8_t)q.cls;
                fam_in[(size_t)f * N + q.d * g + fill[q.d]++] = (uint16_t)(r | (q.cls << 8));
            }
            for (int r = 0; r < N; r++) {   // N lanes with every count <= M_ad and sum M = N  =>  counts equal M
                const HostInst& q = inst[h.u16(off_fam + 2 * ((size_t)f * N + r))];
                cnt[(size_t)q.a * G + q.d] = 0;
                times[h.u16(off_fam + 2 * ((size_t)f * N + r))] = 0;
                for (int k = 0; k < q.n_res; k++) used[q.res[k]] = 0;
            }
        }
        for (uint32_t e = shape_ptr[s]; e < shape_ptr[s + 1]; e++)
            M[(size_t)h.u16(off_nnz + 8 * (size_t)e) * G + h.u16(off_nnz + 8 * (size_t)e + 2)] = 0;
    }
    if (!h.ok) return VP_E_BAD_CATALOG;
    int covered = 1;
    for (int a = 0; a < G; a++)
        for (int d = 0; d < G; d++)
            if ((a != d || g >= 2) && !seen[(size_t)a * G + d]) covered = 0;

    // ---- is every shape invariant under a shift of the node index?
    int sym = 0, P = 1;
    if (S >= 1 && G % S == 0 && G / S >= 2) {
        P = G / S;
        sym = 1;
        std::vector<int> Mfull((size_t)G * G, 0);
        for (int s = 0; s < n_shapes && sym; s++) {
            for (uint32_t e = shape_ptr[s]; e < shape_ptr[s + 1]; e++)
                Mfull[(size_t)h.u16(off_nnz + 8 * (size_t)e) * G + h.u16(off_nnz + 8 * (size_t)e + 2)] = h.u16(off_nnz + 8 * (size_t)e + 4);
            for (uint32_t e = shape_ptr[s]; e < shape_ptr[s + 1] && sym; e++) {
                int a = h.u16(off_nnz + 8 * (size_t)e), d = h.u16(off_nnz + 8 * (size_t)e + 2);
                int a2 = (a + S) % G, d2 = (d + S) % G;
                if (Mfull[(size_t)a2 * G + d2] != Mfull[(size_t)a * G + d]) sym = 0;
            }
            for (uint32_t e = shape_ptr[s]; e < shape_ptr[s + 1]; e++)
                Mfull[(size_t)h.u16(off_nnz + 8 * (size_t)e) * G + h.u16(off_nnz + 8 * (size_t)e + 2)] = 0;
        }
        if (!sym) P = 1;
    }

    // ---- Eq. (6) terms: (byte offset of the 64-bit table entry, lane count)
    std::vector<uint32_t> term_ptr(n_shapes + 1, 0), term;
    for (int s = 0; s < n_shapes; s++) {
        for (uint32_t e = shape_ptr[s]; e < shape_ptr[s + 1]; e++) {
            int a = h.u16(off_nnz + 8 * (size_t)e), d = h.u16(off_nnz + 8 * (size_t)e + 2), m = h.u16(off_nnz + 8 * (size_t)e + 4);
            if (sym) {
                if (a / S != 0) continue;                      // node 0 represents every node
                int delta = d / S, q = a % S, q2 = d % S;
                term.push_back((uint32_t)(((delta * S + q) * S + q2) * 8) | ((uint32_t)m << 16));
            } else {
                term.push_back((uint32_t)((a * G + d) * 8) | ((uint32_t)m << 16));
            }
        }
        term_ptr[s + 1] = (uint32_t)term.size();
    }

    // ---- quantum rule: resources every path of a group pair crosses
    std::vector<std::vector<uint16_t>> forced_cells(n_res);
    std::vector<uint32_t> forced_bw(std::max(n_res, 1), 0);
    {
        std::vector<int> common(n_res + 1);
        int r0 = 0;
        while (r0 < n_inst) {
            int r1 = r0;
            while (r1 < n_inst && inst[r1].a == inst[r0].a && inst[r1].d == inst[r0].d) r1++;
            std::fill(common.begin(), common.end(), 0);
            int64_t best = 0;
            for (int r = r0; r < r1; r++) {
                best = std::max(best, inst[r].bw);
                for (int k = 0; k < inst[r].n_res; k++) common[inst[r].res[k]]++;
            }
            for (int l = 0; l < n_res; l++)
                if (common[l] == r1 - r0) {
                    forced_cells[l].push_back((uint16_t)(inst[r0].a * G + inst[r0].d));
                    forced_bw[l] = (uint32_t)std::max<int64_t>(forced_bw[l], best);
                }
            r0 = r1;
        }
    }
    std::vector<uint32_t> forced_ptr(n_res + 1, 0);
    std::vector<uint16_t> forced_cell;
    for (int l = 0; l < n_res; l++) {
        forced_cell.insert(forced_cell.end(), forced_cells[l].begin(), forced_cells[l].end());
        forced_ptr[l + 1] = (uint32_t)forced_cell.size();
    }

    // ---- device image
    vp_catalog* c = new (std::nothrow) vp_catalog();
    if (!c) return VP_E_NOMEM;
    c->device = device;
    memset(c->memo, 0, sizeof(c->memo));
    c->memo_next = 0;
    c->host_pipe_ready = 0;
    int prev = -1;
    c->sm_count = 0;
    c->max_smem_optin = 0;
    if (device >= 0) {
        cudaGetDevice(&prev);
        if (cudaSetDevice(device) != cudaSuccess) { delete c; return VP_E_CUDA; }
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete c; return VP_E_CUDA; }
        c->sm_count = prop.multiProcessorCount;
        c->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    }
    DevCat& dc = c->dc;
    memset(&dc, 0, sizeof(dc));
    dc.N = N; dc.G = G; dc.g = g; dc.S = S; dc.P = P;
    dc.n_inst = n_inst; dc.n_shapes = n_shapes; dc.n_families = n_fam; dc.n_res = n_res;
    dc.n_classes = (int)rates.size(); dc.sym = sym; dc.tbl_size = sym ? P * S * S : G * G;
    dc.max_bucket = max_bucket; dc.bw_max = bw_max; dc.W = W;
    for (size_t k = 0; k < rates.size(); k++) { dc.class_bw[k] = rates[k]; dc.class_wdiv[k] = W / rates[k]; }
    int rc = VP_OK;
    if ((long long)dc.tbl_size * 8 > 65536) rc = VP_E_UNSUPPORTED;      // term words carry 16-bit byte offsets into the score table
    // fixed-stride copy of the terms (max_terms per shape, zero-count padding) so the scoring loop unrolls
    int max_terms = 0;
    for (int s = 0; s < n_shapes; s++) max_terms = std::max(max_terms, (int)(term_ptr[s + 1] - term_ptr[s]));
    std::vector<uint32_t> term_pad((size_t)n_shapes * max_terms, 0);
    for (int s = 0; s < n_shapes; s++)
        for (uint32_t e = term_ptr[s]; e < term_ptr[s + 1]; e++) term_pad[(size_t)s * max_terms + (e - term_ptr[s])] = term[e];
    dc.max_terms = max_terms;
    if (!rc) rc = upload(c, term_pad, &dc.term);
    {   // the same terms transposed ([term][shape], rows padded to 32 shapes): the layout the kernels keep in shared memory
        const int ns_pad = (n_shapes + 31) & ~31;
        std::vector<uint32_t> term_t((size_t)ns_pad * max_terms, 0);
        for (int s = 0; s < n_shapes; s++)
            for (int e = 0; e < max_terms; e++) term_t[(size_t)e * ns_pad + s] = term_pad[(size_t)s * max_terms + e];
        if (!rc) rc = upload(c, term_t, &dc.term_t);
    }
    if (sym) {   // row patterns: the terms of each shape split by source rail, distinct rows numbered
        std::map<std::vector<uint32_t>, int> ids;
        std::vector<std::vector<uint32_t>> rows;
        const int ns_pad = (n_shapes + 31) & ~31, words = (S + 1) / 2;
        std::vector<uint32_t> shape_pat((size_t)ns_pad * words, 0);
        size_t max_row = 1;
        bool fits = true;
        for (int s = 0; s < n_shapes && fits; s++)
            for (int q = 0; q < S; q++) {
                std::vector<uint32_t> row;
                for (uint32_t e = term_ptr[s]; e < term_ptr[s + 1]; e++) {
                    const uint32_t idx = (term[e] & 0xffffu) / 8;
                    if ((int)((idx / S) % S) == q) row.push_back(idx | (term[e] & 0xffff0000u));
                }
                auto it = ids.find(row);
                int id;
                if (it == ids.end()) {
                    id = (int)rows.size();
                    ids.emplace(row, id);
                    rows.push_back(row);
                    max_row = std::max(max_row, row.size());
                } else {
                    id = it->second;
                }
                if (id >= 65536) { fits = false; break; }
                shape_pat[(size_t)(q / 2) * ns_pad + s] |= (uint32_t)id << (16 * (q & 1));
            }
        if (fits) {
            std::vector<uint32_t> pat_term(rows.size() * max_row, 0);
            for (size_t p = 0; p < rows.size(); p++)
                for (size_t t = 0; t < rows[p].size(); t++) pat_term[p * max_row + t] = rows[p][t];
            dc.n_patterns = (int)rows.size();
            dc.max_row_terms = (int)max_row;
            if (!rc) rc = upload(c, pat_term, &dc.pat_term);
            if (!rc) rc = upload(c, shape_pat, &dc.shape_pat);
            // Two rails: when the shapes that share a first row are consecutive, and first rows fall into few classes
            // with the same list of second rows, the first maximum of Eq. (6) can be taken class by class.
            if (S == 2 && !rc) {
                std::vector<int> run_row, run_start;                       // first row and first shape of every run
                std::vector<std::vector<uint32_t>> run_list;               // its second rows, in shape order
                std::vector<char> seen(rows.size(), 0);
                bool ok = true;
                for (int s = 0; s < n_shapes && ok; s++) {
                    const int p0 = (int)(shape_pat[s] & 0xffffu), p1 = (int)(shape_pat[s] >> 16);
                    if (run_row.empty() || run_row.back() != p0) {
                        if (seen[p0]) ok = false;                           // a first row with two separate runs
                        seen[p0] = 1;
                        run_row.push_back(p0); run_start.push_back(s); run_list.emplace_back();
                    }
                    run_list.back().push_back((uint32_t)p1);
                }
                std::map<std::vector<uint32_t>, int> cls_of;
                std::vector<std::vector<uint32_t>> members, lists;          // per class: first row | run start << 16; second rows
                for (size_t r = 0; r < run_row.size() && ok; r++) {
                    auto it = cls_of.find(run_list[r]);
                    int cl;
                    if (it == cls_of.end()) {
                        cl = (int)members.size();
                        cls_of.emplace(run_list[r], cl);
                        members.emplace_back();
                        lists.push_back(run_list[r]);
                    } else {
                        cl = it->second;
                    }
                    members[cl].push_back((uint32_t)run_row[r] | (uint32_t)run_start[r] << 16);
                }
                // Units: 2 cl = the first rows of class cl, 2 cl + 1 = its second rows; each unit's entries fill whole
                // chunks of 32 (one warp each).  An entry carries the row's terms and its place within the unit.
                const int n = (int)members.size(), stride = (int)max_row + 1;
                size_t n_chunks = 0;
                for (int cl = 0; cl < n; cl++) n_chunks += (members[cl].size() + 31) / 32 + (lists[cl].size() + 31) / 32;
                if (ok && n <= 16 && n_chunks <= 32) {
                    constexpr int kHeader = 72;                            // 3 + (2 n + 1) + up to 32 chunk units <= 72
                    std::vector<uint32_t> dec(kHeader + n_chunks * 32 * stride, 0);
                    dec[0] = (uint32_t)n_chunks; dec[1] = (uint32_t)stride; dec[2] = kHeader;
                    size_t chunk = 0;
                    for (int unit = 0; unit < 2 * n; unit++) {
                        dec[3 + unit] = (uint32_t)chunk;
                        const std::vector<uint32_t>& src = unit & 1 ? lists[unit >> 1] : members[unit >> 1];
                        const size_t padded = (src.size() + 31) / 32 * 32;
                        for (size_t i = 0; i < padded; i++) {
                            uint32_t* ent = &dec[kHeader + (chunk * 32 + i) * stride];
                            if (i >= src.size()) { ent[stride - 1] = 0xffffffffu; continue; }    // padding: never wins
                            const std::vector<uint32_t>& row = rows[src[i] & 0xffffu];
                            for (size_t t = 0; t < row.size(); t++) ent[t] = row[t];
                            // tie-break word: the run start for a first row (runs are in shape order), the place for a second row
                            ent[stride - 1] = unit & 1 ? (uint32_t)i : src[i] >> 16;
                        }
                        for (size_t cc = chunk; cc < chunk + padded / 32; cc++) dec[3 + 2 * n + 1 + cc] = (uint32_t)unit;
                        chunk += padded / 32;
                    }
                    dec[3 + 2 * n] = (uint32_t)chunk;
                    dc.dec_classes = n;
                    dc.dec_words = (int)dec.size();
                    c->dec_host = dec;
                    rc = upload(c, dec, &dc.dec);
                }
            }
        }
    }
    if (!rc) rc = upload(c, bucket_ptr, &dc.bucket_ptr);
    if (!rc) rc = upload(c, fam_slot, &dc.fam_slot);
    if (!rc) rc = upload(c, fam_cls, &dc.fam_cls);
    if (!rc) rc = upload(c, fam_in, &dc.fam_in);
    dc.n_terms = (int)term.size();      // real (unpadded) multiply-adds of one scoring pass
    if (n_shapes < 65536) {             // inverted terms: entry -> (shape, count)
        std::vector<uint32_t> inv_ptr(dc.tbl_size + 1, 0), inv(term.size());
        for (uint32_t w : term) inv_ptr[(w & 0xffffu) / 8 + 1]++;
        for (int e = 0; e < dc.tbl_size; e++) inv_ptr[e + 1] += inv_ptr[e];
        std::vector<uint32_t> fill(inv_ptr.begin(), inv_ptr.end() - 1);
        for (int s = 0; s < n_shapes; s++)
            for (uint32_t e = term_ptr[s]; e < term_ptr[s + 1]; e++)
                inv[fill[(term[e] & 0xffffu) / 8]++] = (uint32_t)s | (term[e] & 0xffff0000u);
        if (!rc) rc = upload(c, inv_ptr, &dc.inv_ptr);
        if (!rc) rc = upload(c, inv, &dc.inv);
    }
    if (!rc) rc = upload(c, forced_ptr, &dc.forced_ptr);
    if (!rc) rc = upload(c, forced_cell, &dc.forced_cell);
    if (!rc) rc = upload(c, forced_bw, &dc.forced_bw);
    std::vector<uint32_t> inst_wdiv(n_inst);
    for (int r = 0; r < n_inst; r++) inst_wdiv[r] = (uint32_t)(W / inst[r].bw);
    if (!rc) rc = upload(c, inst_wdiv, &dc.inst_wdiv);
    if (rc) {
        vp_free_catalog(c);
        if (prev >= 0) cudaSetDevice(prev);
        return rc;
    }
    vp_info& I = c->info;
    I.N = N; I.G = G; I.g = g; I.groups_per_node = S; I.n_resources = n_res; I.n_instances = n_inst;
    I.n_shapes = n_shapes; I.n_families = n_fam; I.max_nnz = max_nnz; I.max_bucket = max_bucket;
    I.covered = covered; I.node_symmetric = sym; I.rate_lcm = W;
    I.row_patterns = dc.n_patterns; I.argmax_classes = dc.dec_classes;
    if (prev >= 0) cudaSetDevice(prev);
    *out = c;
    return VP_OK;
}

extern "C" int64_t vp_kernel_launch_count(void) { return g_vp_launches.load(); }

extern "C" const char* vp_strerror(int code) {
    switch (code) {
        case VP_OK: return "ok";
        case VP_E_BAD_ARG: return "bad argument";
        case VP_E_BAD_CATALOG: return "catalog blob malformed or violates the shape/family constraints";
        case VP_E_NOMEM: return "out of memory";
        case VP_E_CUDA: return "CUDA runtime error";
        case VP_E_WORKSPACE: return "workspace missing, misaligned or too small";
        case VP_E_UNSUPPORTED: return "catalog outside the supported limits (g <= 4, N <= 256, <= 8 path rates)";
        default: return "unknown error";
    }
}
