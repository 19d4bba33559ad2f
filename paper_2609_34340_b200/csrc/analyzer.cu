// vp_build_catalog: offline catalog construction (host code).  What it enumerates is Section 4.1's definition: every
// multiset of path instances that gives each group exactly g outgoing and g incoming lanes (Eq. 3 for its shape,
// Eq. 4 for the family) and uses no directed resource twice.
//
// The search is this build's own: families are assembled one SOURCE GROUP at a time.  A group's g lanes are a
// multiset over the instances that leave it (these are contiguous in the topology blob); the instances are walked in
// id order and each takes 0 .. min(multiplicity, lanes still missing, room left at its destination) lanes, provided
// its footprint is disjoint from the resources taken so far, which is one AND on a bitset.  Two cuts keep the walk
// small: a group is abandoned as soon as the instances not yet walked cannot supply its missing lanes, and the next
// group is only entered if every destination can still reach g with the lanes that later groups can send it.  A
// family is complete when the last group is filled.  PruneFamilies then drops, inside each bucket, exact duplicates
// and families that another family matches footprint by footprint with no lower and somewhere higher rates.
// Output order (what the scheduler's tie-breaks refer to): shapes by their sorted (a, d, count) list,
// families inside a bucket by their instance-id list.
#include <algorithm>
#include <cstring>
#include <map>
#include <vector>

#include "vp_internal.h"

namespace {

struct AInst {
    int a, d, mult, n_res;
    long long bw;
    int res[4];
};

struct Analyzer {
    int N, G, g, n_res;
    std::vector<AInst> inst;
    std::vector<int> group_begin;                           // instances leaving group a: group_begin[a] .. group_begin[a + 1]
    std::vector<int> supply_after;                          // lanes the instances after t, of t's own group, can still give
    std::vector<std::vector<int>> in_later;                 // in_later[a][d]: lanes groups a, a + 1, ... can send to d
    std::vector<std::vector<uint64_t>> footprint;           // per instance: its directed resources as a bitset
    std::vector<uint64_t> taken;                            // resources of the partial family
    std::vector<int> in_deg, chosen;
    std::vector<std::vector<uint16_t>> found;
    size_t limit;
    bool overflow = false;

    void prepare() {
        const int n = (int)inst.size(), words = (n_res + 63) / 64 + 1;
        group_begin.assign(G + 1, n);
        for (int r = n - 1; r >= 0; r--) group_begin[inst[r].a] = r;
        for (int a = G - 1; a >= 0; a--) group_begin[a] = std::min(group_begin[a], group_begin[a + 1]);
        supply_after.assign(n, 0);
        for (int a = 0; a < G; a++) {
            int later = 0;
            for (int r = group_begin[a + 1] - 1; r >= group_begin[a]; r--) { supply_after[r] = later; later += inst[r].mult; }
        }
        in_later.assign(G + 1, std::vector<int>(G, 0));
        for (int a = G - 1; a >= 0; a--) {
            in_later[a] = in_later[a + 1];
            for (int r = group_begin[a]; r < group_begin[a + 1]; r++) in_later[a][inst[r].d] += inst[r].mult;
        }
        footprint.assign(n, std::vector<uint64_t>(words, 0));
        for (int r = 0; r < n; r++)
            for (int k = 0; k < inst[r].n_res; k++) footprint[r][inst[r].res[k] >> 6] |= (uint64_t)1 << (inst[r].res[k] & 63);
        taken.assign(words, 0);
        in_deg.assign(G, 0);
        chosen.clear();
    }
    bool disjoint(int r) const {
        for (size_t w = 0; w < taken.size(); w++)
            if (taken[w] & footprint[r][w]) return false;
        return true;
    }
    // Group a still misses `need` lanes; instances from t on (of this group) may supply them.
    void fill_group(int a, int t, int need) {
        if (overflow) return;
        if (need == 0) {
            if (a + 1 == G) {                               // every group has sent g lanes; each must also have received g
                for (int d = 0; d < G; d++)
                    if (in_deg[d] != g) return;
                if (found.size() >= limit) { overflow = true; return; }
                found.emplace_back(chosen.begin(), chosen.end());
                return;
            }
            for (int d = 0; d < G; d++)                     // can the later groups still fill every destination?
                if (in_deg[d] + in_later[a + 1][d] < g) return;
            fill_group(a + 1, group_begin[a + 1], g);
            return;
        }
        if (t == group_begin[a + 1]) return;
        const AInst& r = inst[t];
        if (supply_after[t] >= need) fill_group(a, t + 1, need);            // no lane on this instance
        if (!disjoint(t)) return;
        const int most = std::min(std::min(r.mult, need), g - in_deg[r.d]);
        if (most < 1) return;
        for (size_t w = 0; w < taken.size(); w++) taken[w] |= footprint[t][w];
        for (int lanes = 1; lanes <= most; lanes++) {
            in_deg[r.d]++;
            chosen.push_back(t);
            if (supply_after[t] >= need - lanes) fill_group(a, t + 1, need - lanes);
        }
        for (int lanes = 0; lanes < most; lanes++) { in_deg[r.d]--; chosen.pop_back(); }
        for (size_t w = 0; w < taken.size(); w++) taken[w] &= ~footprint[t][w];
    }
};

typedef std::vector<std::pair<std::pair<int, int>, int>> Shape;   // sorted ((a, d), count)

uint32_t rd32(const uint8_t* p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24); }
uint16_t rd16(const uint8_t* p) { return (uint16_t)(p[0] | (p[1] << 8)); }
void wr32(std::vector<uint8_t>& o, uint32_t v) { for (int k = 0; k < 4; k++) o.push_back((uint8_t)(v >> (8 * k))); }
void wr16(std::vector<uint8_t>& o, uint16_t v) { o.push_back((uint8_t)v); o.push_back((uint8_t)(v >> 8)); }

// per group pair: the (sorted footprint, rate) of every lane, sorted; used by the dominance test
typedef std::map<std::pair<int, int>, std::vector<std::pair<std::vector<int>, long long>>> Signature;

Signature signature(const Analyzer& A, const std::vector<uint16_t>& fam) {
    Signature s;
    for (uint16_t id : fam) {
        const AInst& r = A.inst[id];
        std::vector<int> fp(r.res, r.res + r.n_res);
        std::sort(fp.begin(), fp.end());
        s[{r.a, r.d}].push_back({fp, r.bw});
    }
    for (auto& kv : s) std::sort(kv.second.begin(), kv.second.end());
    return s;
}

// x is dominated by y: same footprints lane by lane, y nowhere slower, somewhere faster
bool dominated(const Signature& x, const Signature& y) {
    bool strict = false;
    for (const auto& kv : x) {
        auto it = y.find(kv.first);
        if (it == y.end() || it->second.size() != kv.second.size()) return false;
        for (size_t k = 0; k < kv.second.size(); k++) {
            if (kv.second[k].first != it->second[k].first) return false;
            if (it->second[k].second < kv.second[k].second) return false;
            if (it->second[k].second > kv.second[k].second) strict = true;
        }
    }
    return strict;
}

// Reads a topology blob into an Analyzer (instances, degrees, suffix capacities).  kinds (optional) receives the
// instances' kind bytes.
int parse_topology(const void* topology, size_t topo_bytes, Analyzer& A, std::vector<int>* kinds) {
    const uint8_t* t = (const uint8_t*)topology;
    if (topo_bytes < 32 || rd32(t) != 0x50545056u || rd32(t + 4) != 1) return VP_E_BAD_CATALOG;
    A.N = (int)rd32(t + 8); A.G = (int)rd32(t + 12); A.g = (int)rd32(t + 16); A.n_res = (int)rd32(t + 24);
    const int n_inst = (int)rd32(t + 28);
    if (A.N <= 0 || A.G <= 0 || A.g <= 0 || (long long)A.G * A.g != A.N || n_inst <= 0 || n_inst > 0xFFFE || A.n_res < 0 ||
        A.N > 0xFFFF || topo_bytes < 32 + (size_t)n_inst * 20)
        return VP_E_BAD_CATALOG;
    A.inst.resize(n_inst);
    if (kinds) kinds->resize(n_inst);
    for (int r = 0; r < n_inst; r++) {
        const uint8_t* p = t + 32 + (size_t)r * 20;
        AInst& q = A.inst[r];
        q.a = rd16(p); q.d = rd16(p + 2); q.n_res = p[5]; q.mult = rd16(p + 6); q.bw = rd32(p + 8);
        if (kinds) (*kinds)[r] = p[4];
        if (q.a >= A.G || q.d >= A.G || q.n_res > 4 || q.mult < 1 || q.bw <= 0) return VP_E_BAD_CATALOG;
        for (int k = 0; k < q.n_res; k++) {
            q.res[k] = rd16(p + 12 + 2 * k);
            if (q.res[k] >= A.n_res) return VP_E_BAD_CATALOG;
        }
        if (r > 0 && (A.inst[r - 1].a > q.a || (A.inst[r - 1].a == q.a && A.inst[r - 1].d > q.d))) return VP_E_BAD_CATALOG;
    }
    return VP_OK;
}

// Buckets the families in A.found by shape, applies PruneFamilies inside each bucket and writes the channels blob in
// canonical order (shapes by their sorted (a, d, count) list, families by their instance-id list).
int write_catalog(Analyzer& A, void* channels_out, size_t capacity_bytes, size_t* bytes_needed, int32_t* n_shapes_out,
                  int32_t* n_families_out) {
    std::map<Shape, std::vector<std::vector<uint16_t>>> buckets;
    for (auto& fam : A.found) {
        std::map<std::pair<int, int>, int> cnt;
        for (uint16_t id : fam) cnt[{A.inst[id].a, A.inst[id].d}]++;
        buckets[Shape(cnt.begin(), cnt.end())].push_back(fam);
    }
    size_t n_fam = 0, total_nnz = 0;
    for (auto& kv : buckets) {
        auto& fams = kv.second;
        std::sort(fams.begin(), fams.end());
        fams.erase(std::unique(fams.begin(), fams.end()), fams.end());
        std::vector<Signature> sig;
        for (auto& f : fams) sig.push_back(signature(A, f));
        std::vector<std::vector<uint16_t>> keep;
        for (size_t x = 0; x < fams.size(); x++) {
            bool dom = false;
            for (size_t y = 0; y < fams.size() && !dom; y++)
                if (y != x && dominated(sig[x], sig[y])) dom = true;
            if (!dom) keep.push_back(fams[x]);
        }
        fams.swap(keep);
        n_fam += fams.size();
        total_nnz += kv.first.size();
    }
    std::vector<uint8_t> o;
    wr32(o, 0x48435056u); wr32(o, 1); wr32(o, (uint32_t)A.N); wr32(o, (uint32_t)buckets.size());
    wr32(o, (uint32_t)n_fam); wr32(o, (uint32_t)total_nnz);
    uint32_t run = 0;
    for (auto& kv : buckets) { wr32(o, run); run += (uint32_t)kv.first.size(); }
    wr32(o, run);
    for (auto& kv : buckets)
        for (auto& e : kv.first) { wr16(o, (uint16_t)e.first.first); wr16(o, (uint16_t)e.first.second); wr16(o, (uint16_t)e.second); wr16(o, 0); }
    run = 0;
    for (auto& kv : buckets) { wr32(o, run); run += (uint32_t)kv.second.size(); }
    wr32(o, run);
    for (auto& kv : buckets)
        for (auto& f : kv.second)
            for (uint16_t id : f) wr16(o, id);
    *bytes_needed = o.size();
    if (n_shapes_out) *n_shapes_out = (int32_t)buckets.size();
    if (n_families_out) *n_families_out = (int32_t)n_fam;
    if (!channels_out || capacity_bytes < o.size()) return channels_out ? VP_E_WORKSPACE : VP_OK;
    memcpy(channels_out, o.data(), o.size());
    return VP_OK;
}

}  // namespace

extern "C" int vp_build_catalog(const void* topology, size_t topo_bytes, void* channels_out, size_t capacity_bytes,
                                size_t* bytes_needed, int32_t* n_shapes_out, int32_t* n_families_out) {
    if (!topology || !bytes_needed) return VP_E_BAD_ARG;
    Analyzer A;
    int rc = parse_topology(topology, topo_bytes, A, nullptr);
    if (rc) return rc;
    A.prepare();
    A.limit = (size_t)1 << 22;                              // more families than this is not a usable catalog
    A.fill_group(0, A.group_begin[0], A.g);
    if (A.overflow) return VP_E_UNSUPPORTED;
    if (A.found.empty()) return VP_E_BAD_CATALOG;
    return write_catalog(A, channels_out, capacity_bytes, bytes_needed, n_shapes_out, n_families_out);
}

// A catalog for many nodes without the exponential search: one per-node TEMPLATE applied to every node, so that every
// family is invariant under a shift of the node index.  (The paper's search, Algorithm 1, grows exponentially with the
// node count; its Table 3 catalogs for 16 to 32 nodes have a few hundred shapes, which a complete enumeration cannot
// give.  This construction is this library's reading; it needs two switch-local groups per node, each with one
// network path to every other group and one path to its sibling group.)  A template gives each of the two groups q of a
// node a network target "none" or (delta, q2) = group q2 of node (n + delta) mod P -- delta = 0 needs q2 != q, and the two
// groups must not target the same q2 -- plus one flag per direction of the sibling path; a group must send as many
// such lanes as it receives, and switch-local lanes fill the rest of its g slots.
extern "C" int vp_build_template_catalog(const void* topology, size_t topo_bytes, void* channels_out, size_t capacity_bytes,
                                         size_t* bytes_needed, int32_t* n_shapes_out, int32_t* n_families_out) {
    if (!topology || !bytes_needed) return VP_E_BAD_ARG;
    Analyzer A;
    std::vector<int> kinds;
    int rc = parse_topology(topology, topo_bytes, A, &kinds);
    if (rc) return rc;
    const uint8_t* t = (const uint8_t*)topology;
    const int S = (int)rd32(t + 20);
    if (S != 2 || A.G % S) return VP_E_UNSUPPORTED;
    const int P = A.G / S, g = A.g;
    std::map<std::pair<std::pair<int, int>, int>, int> by_key;          // (a, d, kind) -> instance id
    for (int r = 0; r < (int)A.inst.size(); r++) by_key[{{A.inst[r].a, A.inst[r].d}, kinds[r]}] = r;
    auto find = [&](int a, int d, int kind) {
        auto it = by_key.find({{a, d}, kind});
        return it == by_key.end() ? -1 : it->second;
    };
    struct Opt { int delta, q2; };                                       // delta < 0: no network lane
    std::vector<Opt> opts[2];
    for (int q = 0; q < S; q++) {
        opts[q].push_back({-1, 0});
        for (int delta = 0; delta < P; delta++)
            for (int q2 = 0; q2 < S; q2++)
                if (!(delta == 0 && q2 == q)) opts[q].push_back({delta, q2});
    }
    for (const Opt& n0 : opts[0])
        for (const Opt& n1 : opts[1])
            for (int p01 = 0; p01 < 2; p01++)
                for (int p10 = 0; p10 < 2; p10++) {
                    if (n0.delta >= 0 && n1.delta >= 0 && n0.q2 == n1.q2) continue;
                    const Opt nic[2] = {n0, n1};
                    const int out[2] = {p01 + (n0.delta >= 0), p10 + (n1.delta >= 0)};
                    const int inn[2] = {p10 + (n0.delta >= 0 && n0.q2 == 0) + (n1.delta >= 0 && n1.q2 == 0),
                                        p01 + (n0.delta >= 0 && n0.q2 == 1) + (n1.delta >= 0 && n1.q2 == 1)};
                    if (out[0] != inn[0] || out[1] != inn[1] || std::max(out[0], out[1]) > g) continue;
                    if (g < 2 && std::min(out[0], out[1]) < g) continue;
                    std::vector<uint16_t> fam;
                    bool ok = true;
                    for (int node = 0; node < P && ok; node++)
                        for (int q = 0; q < S && ok; q++) {
                            const int a = node * S + q;
                            if (g - out[q] > 0) {
                                const int pix = find(a, a, 0);
                                if (pix < 0) { ok = false; break; }
                                for (int k = 0; k < g - out[q]; k++) fam.push_back((uint16_t)pix);
                            }
                            if (q == 0 ? p01 : p10) {
                                const int pxb = find(a, node * S + (1 - q), 1);
                                if (pxb < 0) { ok = false; break; }
                                fam.push_back((uint16_t)pxb);
                            }
                            if (nic[q].delta >= 0) {
                                const int d = ((node + nic[q].delta) % P) * S + nic[q].q2;
                                const int id = find(a, d, 2);
                                if (id < 0) { ok = false; break; }
                                fam.push_back((uint16_t)id);
                            }
                        }
                    if (!ok) return VP_E_UNSUPPORTED;             // the topology lacks a path the template needs
                    std::sort(fam.begin(), fam.end());
                    A.found.push_back(fam);
                }
    if (A.found.empty()) return VP_E_BAD_CATALOG;
    return write_catalog(A, channels_out, capacity_bytes, bytes_needed, n_shapes_out, n_families_out);
}

namespace {
}  // namespace

// PrunePaths of Section 4.1 ("Pruning and search cost"), the filter that runs before the search: a path instance r
// is dropped when another instance r' of the same group pair has a footprint L(r') that is a subset of L(r) and a
// rate bw(r') >= bw(r), with at least one of the two strict.  The survivors keep their order.
extern "C" int vp_prune_paths(const void* topology, size_t topo_bytes, void* topology_out, size_t capacity_bytes,
                              size_t* bytes_needed, int32_t* n_kept_out) {
    if (!topology || !bytes_needed) return VP_E_BAD_ARG;
    const uint8_t* t = (const uint8_t*)topology;
    if (topo_bytes < 32 || rd32(t) != 0x50545056u || rd32(t + 4) != 1) return VP_E_BAD_CATALOG;
    const int n_inst = (int)rd32(t + 28);
    if (n_inst < 0 || n_inst > 0xFFFE || topo_bytes < 32 + (size_t)n_inst * 20) return VP_E_BAD_CATALOG;
    struct P { int a, d, n_res; long long bw; int res[4]; };
    std::vector<P> inst(n_inst);
    for (int r = 0; r < n_inst; r++) {
        const uint8_t* p = t + 32 + (size_t)r * 20;
        P& q = inst[r];
        q.a = rd16(p); q.d = rd16(p + 2); q.n_res = p[5]; q.bw = rd32(p + 8);
        if (q.n_res > 4) return VP_E_BAD_CATALOG;
        for (int k = 0; k < q.n_res; k++) q.res[k] = rd16(p + 12 + 2 * k);
    }
    auto subset = [](const P& x, const P& y) {               // L(x) is a subset of L(y)
        for (int i = 0; i < x.n_res; i++) {
            bool found = false;
            for (int k = 0; k < y.n_res; k++) found |= x.res[i] == y.res[k];
            if (!found) return false;
        }
        return true;
    };
    std::vector<int> keep;
    for (int r = 0; r < n_inst; r++) {
        bool dominated = false;
        for (int o = 0; o < n_inst && !dominated; o++) {
            if (o == r || inst[o].a != inst[r].a || inst[o].d != inst[r].d) continue;
            if (!subset(inst[o], inst[r]) || inst[o].bw < inst[r].bw) continue;
            const bool strict = !subset(inst[r], inst[o]) || inst[o].bw > inst[r].bw;
            if (strict) dominated = true;
        }
        if (!dominated) keep.push_back(r);
    }
    *bytes_needed = 32 + keep.size() * 20;
    if (n_kept_out) *n_kept_out = (int32_t)keep.size();
    if (!topology_out || capacity_bytes < *bytes_needed) return topology_out ? VP_E_WORKSPACE : VP_OK;
    uint8_t* o = (uint8_t*)topology_out;
    memcpy(o, t, 32);
    const uint32_t n = (uint32_t)keep.size();
    for (int k = 0; k < 4; k++) o[28 + k] = (uint8_t)(n >> (8 * k));
    for (size_t i = 0; i < keep.size(); i++) memcpy(o + 32 + i * 20, t + 32 + (size_t)keep[i] * 20, 20);
    return VP_OK;
}
