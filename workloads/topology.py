"""Topology and channel-catalog inputs (Section 3 model setup, Section 4.1).

The online scheduler takes the catalog as a given input (Algorithm 2,
"Require: complete catalog tree").  This module builds such inputs:

* PCIe-tree topologies: ``P`` nodes, two PCIe switches per node, ``g`` GPUs and
  one NIC per switch.  A rank group is one switch (Section 4.1, "switch-local
  rank groups").  Directed shared resources per group ``a``: the switch uplink in
  both directions (``up``, ``down``) and the NIC in both directions (``NICtx``,
  ``NICrx``); endpoint GPU-to-switch links are not modelled (Section 3).
  Group-level path instances: PIX (same switch, empty footprint, may be used by
  up to ``g`` lanes), PXB (other switch of the same node, footprint
  ``{up(a), down(d)}``) and NIC (any other group, footprint
  ``{NICtx(a), NICrx(d)}``).
* the complete family catalog of a topology by the pruned binary DFS of
  Algorithm 1 with ``PrunePaths`` / ``PruneFamilies``;
* a node-template ("symmetric") catalog for deployments whose complete family
  set is too large to enumerate: every node applies the same template.

Everything is serialised into two little-endian byte blobs, the only thing the
oracle and the CUDA library both read.

Blob layouts
------------
topology: ``u32 magic 'VPTP', u32 version, u32 N, u32 G, u32 g,
u32 groups_per_node, u32 n_resources, u32 n_instances`` then per instance 20
bytes ``u16 src_group, u16 dst_group, u8 kind, u8 n_res, u16 mult, u32 bw,
u16 res[4]``.  Instance ids are positions in this list, which is sorted by
``(src_group, dst_group, kind)``.  Ranks of group ``a`` are ``a*g .. a*g+g-1``.

channels: ``u32 magic 'VPCH', u32 version, u32 N, u32 n_shapes, u32 n_families,
u32 total_nnz``; ``u32 shape_ptr[n_shapes+1]``; ``total_nnz`` records
``u16 a, u16 d, u16 count, u16 pad``; ``u32 bucket_ptr[n_shapes+1]`` (families
are stored grouped by shape, so the families of shape ``s`` are the global
family ids ``bucket_ptr[s] .. bucket_ptr[s+1]-1``, in tie-break order);
``u16 fam_inst[n_families][N]`` ascending instance ids, a multi-lane instance
repeated once per lane.
"""
from __future__ import annotations

import struct
from dataclasses import dataclass, field
from itertools import product
from typing import Dict, List, Sequence, Tuple

import numpy as np

KIND_PIX, KIND_PXB, KIND_NIC = 0, 1, 2
TOPO_MAGIC = 0x50545056  # 'VPTP'
CHAN_MAGIC = 0x48435056  # 'VPCH'
BLOB_VERSION = 1


@dataclass(frozen=True)
class Instance:
    """One group-level path instance r in R_ad (Section 4.1)."""

    src_group: int
    dst_group: int
    kind: int
    bw: int  # bytes per nanosecond (= GB/s)
    mult: int  # how many lanes of one family may use it (PIX: g, else 1)
    res: Tuple[int, ...]  # directed shared resources L(r)


@dataclass
class Topology:
    N: int
    G: int
    g: int
    groups_per_node: int
    n_resources: int
    instances: List[Instance]

    def blob(self) -> bytes:
        out = [struct.pack("<8I", TOPO_MAGIC, BLOB_VERSION, self.N, self.G, self.g,
                           self.groups_per_node, self.n_resources, len(self.instances))]
        for r in self.instances:
            res = list(r.res) + [0] * (4 - len(r.res))
            out.append(struct.pack("<HHBBHI4H", r.src_group, r.dst_group, r.kind,
                                   len(r.res), r.mult, r.bw, *res))
        return b"".join(out)


@dataclass
class Catalog:
    topology: Topology
    shapes: List[List[Tuple[int, int, int]]]  # per shape: sorted (a, d, count)
    buckets: List[List[Tuple[int, ...]]]  # per shape: families (N instance ids)
    families: List[Tuple[int, ...]] = field(init=False)
    bucket_ptr: List[int] = field(init=False)

    def __post_init__(self) -> None:
        self.families = [f for b in self.buckets for f in b]
        ptr = [0]
        for b in self.buckets:
            ptr.append(ptr[-1] + len(b))
        self.bucket_ptr = ptr

    @property
    def n_shapes(self) -> int:
        return len(self.shapes)

    @property
    def n_families(self) -> int:
        return len(self.families)

    def blob(self) -> bytes:
        N = self.topology.N
        shape_ptr = [0]
        for s in self.shapes:
            shape_ptr.append(shape_ptr[-1] + len(s))
        out = [struct.pack("<6I", CHAN_MAGIC, BLOB_VERSION, N, self.n_shapes,
                           self.n_families, shape_ptr[-1])]
        out.append(np.asarray(shape_ptr, dtype="<u4").tobytes())
        nnz = np.zeros((shape_ptr[-1], 4), dtype="<u2")
        k = 0
        for s in self.shapes:
            for (a, d, c) in s:
                nnz[k, 0], nnz[k, 1], nnz[k, 2] = a, d, c
                k += 1
        out.append(nnz.tobytes())
        out.append(np.asarray(self.bucket_ptr, dtype="<u4").tobytes())
        fam = np.asarray(self.families, dtype="<u2").reshape(self.n_families, N)
        out.append(fam.tobytes())
        return b"".join(out)


# --------------------------------------------------------------------------
# topologies
# --------------------------------------------------------------------------

def _res_id(group: int, which: int) -> int:
    """which: 0 uplink towards the root, 1 downlink from the root, 2 NIC transmit, 3 NIC receive."""
    return group * 4 + which


def prune_paths(cands: Sequence[Instance]) -> List[Instance]:
    """PrunePaths (Section 4.1): drop r when another r' of the same group pair has
    L(r') a subset of L(r) and bw(r') >= bw(r), with at least one strict."""
    keep = []
    for r in cands:
        dominated = False
        for o in cands:
            if o is r or (o.src_group, o.dst_group) != (r.src_group, r.dst_group):
                continue
            if set(o.res) <= set(r.res) and o.bw >= r.bw and (set(o.res) < set(r.res) or o.bw > r.bw):
                dominated = True
                break
        if not dominated:
            keep.append(r)
    return keep


def tree_topology(nodes: int, g: int = 4, pcie_bw: int = 64, nic_bw: int = 64,
                  switches_per_node: int = 2) -> Topology:
    """PCIe tree: ``nodes`` x ``switches_per_node`` switches x ``g`` GPUs, one NIC per switch.

    A GPU reaches the network only through its own switch's NIC; the inter-node
    fabric is non-blocking, so a NIC path's footprint is the two NIC directions.
    """
    S = switches_per_node
    G = nodes * S
    cands: List[Instance] = []
    for a in range(G):
        for d in range(G):
            same_node = (a // S) == (d // S)
            if a == d:
                if g >= 2:
                    cands.append(Instance(a, d, KIND_PIX, pcie_bw, g, ()))
                # NIC loop-back through the own switch: dominated by PIX, removed below
                cands.append(Instance(a, d, KIND_NIC, nic_bw, 1, (_res_id(a, 2), _res_id(d, 3))))
                continue
            if same_node:
                cands.append(Instance(a, d, KIND_PXB, pcie_bw, 1, (_res_id(a, 0), _res_id(d, 1))))
            cands.append(Instance(a, d, KIND_NIC, nic_bw, 1, (_res_id(a, 2), _res_id(d, 3))))
    inst = prune_paths(cands)
    if g < 2:  # a one-GPU switch has no valid same-switch pair (i != j)
        inst = [r for r in inst if r.src_group != r.dst_group]
    inst.sort(key=lambda r: (r.src_group, r.dst_group, r.kind))
    return Topology(N=G * g, G=G, g=g, groups_per_node=S, n_resources=4 * G, instances=inst)


def ring_topology(nodes: int, switches_per_node: int = 4, g: int = 2, pcie_bw: int = 64, nic_bw: int = 64) -> Topology:
    """PCIe ring (Table 2 lists one platform with a "Ring" PCIe topology and says no more; this is the plainest
    reading): the switches of a node form a ring, each with ``g`` GPUs and one NIC.  Directed shared resources per
    switch: its clockwise and its counter-clockwise ring link, NIC transmit, NIC receive.  Group-level path
    instances: PIX (same switch), one ring path per direction to every other switch of the node (footprint = the
    ring links it crosses, at most four), NIC to every other group; ``PrunePaths`` then removes dominated ones."""
    S = switches_per_node
    G = nodes * S
    cands: List[Instance] = []
    for a in range(G):
        node, sa = divmod(a, S)
        for d in range(G):
            if a == d:
                if g >= 2:
                    cands.append(Instance(a, d, KIND_PIX, pcie_bw, g, ()))
                continue
            if d // S == node:
                sd = d % S
                cw = [_res_id(node * S + (sa + k) % S, 0) for k in range((sd - sa) % S)]
                ccw = [_res_id(node * S + (sa - k) % S, 1) for k in range((sa - sd) % S)]
                for links in (cw, ccw):
                    if len(links) <= 4:
                        cands.append(Instance(a, d, KIND_PXB, pcie_bw, 1, tuple(links)))
            cands.append(Instance(a, d, KIND_NIC, nic_bw, 1, (_res_id(a, 2), _res_id(d, 3))))
    inst = prune_paths(cands)
    inst.sort(key=lambda r: (r.src_group, r.dst_group, r.kind, len(r.res), r.res))
    return Topology(N=G * g, G=G, g=g, groups_per_node=S, n_resources=4 * G, instances=inst)


def crossbar_topology(n: int, bw: int = 64) -> Topology:
    """One switch with ``n`` GPUs: a single group, every pair on a PIX path."""
    return Topology(N=n, G=1, g=n, groups_per_node=1, n_resources=0,
                    instances=[Instance(0, 0, KIND_PIX, bw, n, ())])


# --------------------------------------------------------------------------
# catalogs
# --------------------------------------------------------------------------

def _shape_of(topo: Topology, fam: Sequence[int]) -> Tuple[Tuple[int, int, int], ...]:
    cnt: Dict[Tuple[int, int], int] = {}
    for r in fam:
        i = topo.instances[r]
        cnt[(i.src_group, i.dst_group)] = cnt.get((i.src_group, i.dst_group), 0) + 1
    return tuple(sorted((a, d, c) for (a, d), c in cnt.items()))


def _prune_families(topo: Topology, fams: List[Tuple[int, ...]]) -> List[Tuple[int, ...]]:
    """PruneFamilies (Section 4.1) within one shape: exact duplicates, and families
    whose instances pair up per group pair with identical footprints and no
    lower rates against another family that is strictly faster somewhere."""
    uniq = sorted(set(fams))

    def signature(f):
        sig: Dict[Tuple[int, int], List[Tuple[Tuple[int, ...], int]]] = {}
        for r in f:
            i = topo.instances[r]
            sig.setdefault((i.src_group, i.dst_group), []).append((tuple(sorted(i.res)), i.bw))
        return {k: sorted(v) for k, v in sig.items()}

    sigs = [signature(f) for f in uniq]
    keep = []
    for x, sx in zip(uniq, sigs):
        dominated = False
        for y, sy in zip(uniq, sigs):
            if y is x:
                continue
            ok, strict = True, False
            for k in sx:
                fx, fy = sx[k], sy[k]
                if [t[0] for t in fx] != [t[0] for t in fy]:
                    ok = False
                    break
                for (_, bx), (_, by) in zip(fx, fy):
                    if by < bx:
                        ok = False
                    if by > bx:
                        strict = True
                if not ok:
                    break
            if ok and strict:
                dominated = True
                break
        if not dominated:
            keep.append(x)
    return keep


def _assemble(topo: Topology, fams: Sequence[Tuple[int, ...]], prune: bool = True) -> Catalog:
    by_shape: Dict[Tuple[Tuple[int, int, int], ...], List[Tuple[int, ...]]] = {}
    for f in fams:
        by_shape.setdefault(_shape_of(topo, f), []).append(tuple(f))
    shapes = sorted(by_shape)
    buckets = []
    for s in shapes:
        b = _prune_families(topo, by_shape[s]) if prune else sorted(set(by_shape[s]))
        buckets.append(b)
    return Catalog(topo, [list(s) for s in shapes], buckets)


def complete_catalog(topo: Topology) -> Catalog:
    """Algorithm 1: every resource-disjoint instance set that gives each group
    exactly ``g`` outgoing and ``g`` incoming lanes."""
    inst, G, g = topo.instances, topo.G, topo.g
    m = len(inst)
    # capacity still available from instance t onwards, per group (SuffixOK)
    out_suffix = np.zeros((m + 1, G), dtype=np.int64)
    in_suffix = np.zeros((m + 1, G), dtype=np.int64)
    for t in range(m - 1, -1, -1):
        out_suffix[t] = out_suffix[t + 1]
        in_suffix[t] = in_suffix[t + 1]
        out_suffix[t, inst[t].src_group] += inst[t].mult
        in_suffix[t, inst[t].dst_group] += inst[t].mult
    res_mask = [sum(1 << x for x in r.res) for r in inst]
    out_deg = [0] * G
    in_deg = [0] * G
    chosen: List[int] = []
    found: List[Tuple[int, ...]] = []

    def explore(t: int, used: int) -> None:
        if all(x == g for x in out_deg) and all(x == g for x in in_deg):  # Complete
            found.append(tuple(chosen))
            return
        if t >= m:
            return
        for a in range(G):  # SuffixOK
            if out_deg[a] + out_suffix[t, a] < g or in_deg[a] + in_suffix[t, a] < g:
                return
        r = inst[t]
        explore(t + 1, used)  # exclude branch
        # include branch, once per admissible lane count (CanAdd: degree limits + disjointness)
        if used & res_mask[t]:
            return
        added = 0
        for c in range(1, r.mult + 1):
            if out_deg[r.src_group] + 1 > g or in_deg[r.dst_group] + 1 > g:
                break
            out_deg[r.src_group] += 1
            in_deg[r.dst_group] += 1
            chosen.append(t)
            added += 1
            explore(t + 1, used | res_mask[t])
        for _ in range(added):
            out_deg[r.src_group] -= 1
            in_deg[r.dst_group] -= 1
            chosen.pop()

    explore(0, 0)
    return _assemble(topo, found)


def node_template_catalog(topo: Topology) -> Catalog:
    """Symmetric catalog: one per-node template applied to every node.

    A template gives each of the two rails ``q`` a NIC target ``none`` or
    ``(delta, q2)`` = "send to rail ``q2`` of node ``(n+delta) mod P``" (``delta=0``
    needs ``q2 != q``), the targets of the two rails using different ``q2``, plus
    two PXB flags; each rail must send as many non-PIX lanes as it receives,
    and PIX lanes fill the rest.
    """
    S = topo.groups_per_node
    if S != 2:
        raise ValueError("node templates are defined for two switches per node")
    P = topo.G // S
    g = topo.g
    by_key = {(r.src_group, r.dst_group, r.kind): i for i, r in enumerate(topo.instances)}
    nic_opts: List[List] = []
    for q in range(S):
        opts = [None]
        for delta in range(P):
            for q2 in range(S):
                if delta == 0 and q2 == q:
                    continue
                opts.append((delta, q2))
        nic_opts.append(opts)
    fams = []
    for n0, n1, p01, p10 in product(nic_opts[0], nic_opts[1], (0, 1), (0, 1)):
        nic = (n0, n1)
        if n0 is not None and n1 is not None and n0[1] == n1[1]:
            continue
        out = [p01 + (n0 is not None), p10 + (n1 is not None)]
        inn = [p10 + sum(1 for t in nic if t is not None and t[1] == 0),
               p01 + sum(1 for t in nic if t is not None and t[1] == 1)]
        if out != inn or max(out) > g:
            continue
        if g < 2 and min(out) < g:
            continue
        fam: List[int] = []
        for node in range(P):
            for q in range(S):
                a = node * S + q
                fam += [by_key[(a, a, KIND_PIX)]] * (g - out[q])
                if (p01, p10)[q]:
                    fam.append(by_key[(a, node * S + (1 - q), KIND_PXB)])
                if nic[q] is not None:
                    d = ((node + nic[q][0]) % P) * S + nic[q][1]
                    fam.append(by_key[(a, d, KIND_NIC)])
        fams.append(tuple(sorted(fam)))
    return _assemble(topo, fams)


def crossbar_catalog(topo: Topology) -> Catalog:
    """The single shape [g] and single family (g PIX lanes) of a one-switch topology."""
    return Catalog(topo, [[(0, 0, topo.g)]], [[tuple([0] * topo.g)]])
