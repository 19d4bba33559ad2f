"""Pins for the oracle's channel model and for the catalog inputs (no GPU)."""
import os
import struct

import numpy as np
import pytest

from workloads.topology import (KIND_NIC, KIND_PIX, KIND_PXB, complete_catalog, crossbar_catalog,
                                crossbar_topology, node_template_catalog, tree_topology)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def _oc(oracle_lib, cat):
    return oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())


def test_table3_row1_catalog_size(oracle_lib):
    """Table 3, 8-GPU tree node: 3 shapes and 6 families."""
    shapes, fams = (int(x) for x in _golden("table3_row1.txt")[0])
    cat = complete_catalog(tree_topology(1, g=4))
    assert (cat.n_shapes, cat.n_families) == (shapes, fams)
    oc = _oc(oracle_lib, cat)
    assert (oc.n_shapes, oc.n_families) == (shapes, fams)
    assert oc.check() == 0 and oc.covers()


def test_node_template_equals_complete_for_one_node():
    a = complete_catalog(tree_topology(1))
    b = node_template_catalog(tree_topology(1))
    assert a.shapes == b.shapes and a.buckets == b.buckets


@pytest.mark.parametrize("nodes,kind,counts", [(2, "complete", (89, 152)), (2, "template", (15, 20)),
                                                (8, "template", (255, 272))])
def test_catalogs_satisfy_eq3_eq4(oracle_lib, nodes, kind, counts):
    topo = tree_topology(nodes)
    cat = complete_catalog(topo) if kind == "complete" else node_template_catalog(topo)
    assert (cat.n_shapes, cat.n_families) == counts
    oc = _oc(oracle_lib, cat)
    assert oc.check() == 0          # Eq. (3) for every shape, Eq. (4) for every family
    assert oc.covers()


def test_template_families_are_a_subset_of_the_complete_catalog():
    topo = tree_topology(2)
    full = set(complete_catalog(topo).families)
    assert set(node_template_catalog(topo).families) <= full


def test_complete_catalog_matches_brute_force_subset_enumeration():
    """Algorithm 1 must find every instance multiset with g in/out lanes per group and disjoint
    footprints: compare with plain enumeration on the 2x2-GPU node."""
    from itertools import combinations_with_replacement
    topo = tree_topology(1, g=2)
    inst = topo.instances
    want = set()
    for fam in combinations_with_replacement(range(len(inst)), topo.N):
        out = [0] * topo.G
        inn = [0] * topo.G
        used = []
        ok = True
        for r in set(fam):
            if fam.count(r) > inst[r].mult:
                ok = False
        for r in fam:
            out[inst[r].src_group] += 1
            inn[inst[r].dst_group] += 1
            used += list(inst[r].res)
        if ok and out == [topo.g] * topo.G and inn == [topo.g] * topo.G and len(used) == len(set(used)):
            want.add(tuple(fam))
    assert set(complete_catalog(topo).families) == want


def test_corrupted_catalogs_fail_the_checks(oracle_lib):
    cat = complete_catalog(tree_topology(1))
    topo_blob, blob = cat.topology.blob(), bytearray(cat.blob())
    n_shapes, n_fam, nnz = struct.unpack_from("<3I", blob, 12)
    nnz_off = 24 + 4 * (n_shapes + 1)
    fam_off = nnz_off + 8 * nnz + 4 * (n_shapes + 1)
    # unbalanced shape: bump one lane count (Eq. 3)
    bad = bytearray(blob)
    struct.pack_into("<H", bad, nnz_off + 4, struct.unpack_from("<H", bad, nnz_off + 4)[0] + 1)
    assert oracle_lib.OracleCatalog(topo_blob, bytes(bad)).check() == 3
    # family using one PXB instance twice: same directed resources twice (Eq. 4)
    inst = cat.topology.instances
    pxb01 = next(i for i, r in enumerate(inst) if r.kind == KIND_PXB and r.src_group == 0)
    nic01 = next(i for i, r in enumerate(inst) if r.kind == KIND_NIC and r.src_group == 0)
    fams = np.frombuffer(bytes(blob), dtype="<u2", offset=fam_off).reshape(n_fam, 8).copy()
    f = next(i for i in range(n_fam) if pxb01 in fams[i] and nic01 in fams[i])
    fams[f][list(fams[f]).index(nic01)] = pxb01
    fams[f].sort()
    bad = bytearray(blob)
    bad[fam_off:] = fams.astype("<u2").tobytes()
    assert oracle_lib.OracleCatalog(topo_blob, bytes(bad)).check() == 4
    # truncated blob
    with pytest.raises(ValueError):
        oracle_lib.OracleCatalog(topo_blob, bytes(blob[:-4]))


def test_fig1_aggregate_bandwidths(oracle_lib):
    """Figure 1: 6 GPUs on two switches, PCIe 64 / NIC 50 GB/s.  Stages A and B use the cyclic
    matching i -> (i+3) mod 6; A puts all six transfers on PXB (128 GB/s, contended), B moves one
    transfer per direction to the NIC (228, PXB still contended), C is a feasible channel with two
    PIX, two PXB and two NIC lanes (356)."""
    g = _golden("fig1_aggregate_bw.txt")
    want_a, want_b, want_c = (int(x) for x in g[0])
    pcie, nic = int(g[1][0]), int(g[2][0])
    topo = tree_topology(1, g=3, pcie_bw=pcie, nic_bw=nic)
    cat = complete_catalog(topo)
    oc = _oc(oracle_lib, cat)
    ids = {(r.src_group, r.dst_group, r.kind): i for i, r in enumerate(topo.instances)}
    cyc = [(i + 3) % 6 for i in range(6)]
    pxb = [ids[(i // 3, cyc[i] // 3, KIND_PXB)] for i in range(6)]
    assert oc.aggregate_bw(cyc, pxb) == want_a
    assert oc.lanes_feasible(cyc, pxb) in (4, 5)       # one path / one directed resource used twice
    mixed = list(pxb)
    mixed[0] = ids[(0, 1, KIND_NIC)]
    mixed[3] = ids[(1, 0, KIND_NIC)]
    assert oc.aggregate_bw(cyc, mixed) == want_b
    assert oc.lanes_feasible(cyc, mixed) in (4, 5)
    # joint peer-path selection: 0->1 PIX, 1->3 PXB, 2->4 NIC, 3->0 PXB, 4->5 PIX, 5->2 NIC
    dst = [1, 3, 4, 0, 5, 2]
    path = [ids[(0, 0, KIND_PIX)], ids[(0, 1, KIND_PXB)], ids[(0, 1, KIND_NIC)],
            ids[(1, 0, KIND_PXB)], ids[(1, 1, KIND_PIX)], ids[(1, 0, KIND_NIC)]]
    assert oc.lanes_feasible(dst, path) == 0
    assert oc.aggregate_bw(dst, path) == want_c
    # that channel's shape [[1,2],[2,1]] is in the catalog
    assert [(0, 0, 1), (0, 1, 2), (1, 0, 2), (1, 1, 1)] in cat.shapes


def test_feasibility_rejections(oracle_lib):
    topo = tree_topology(1)
    oc = _oc(oracle_lib, complete_catalog(topo))
    ids = {(r.src_group, r.dst_group, r.kind): i for i, r in enumerate(topo.instances)}
    idle = [-1] * 8
    none = [0xFFFF] * 8
    assert oc.lanes_feasible(idle, none) == 0
    d, p = list(idle), list(none)
    d[0], p[0] = 0, ids[(0, 0, KIND_PIX)]
    assert oc.lanes_feasible(d, p) == 1                  # self transfer
    d[0], p[0] = 5, ids[(0, 0, KIND_PIX)]
    assert oc.lanes_feasible(d, p) == 2                  # path does not connect the groups
    d[0], p[0] = 5, ids[(0, 1, KIND_PXB)]
    d[1], p[1] = 5, ids[(0, 1, KIND_NIC)]
    assert oc.lanes_feasible(d, p) == 3                  # two lanes into one rank
    d[1], p[1] = 6, ids[(0, 1, KIND_PXB)]
    assert oc.lanes_feasible(d, p) in (4, 5)             # same instance / same resources twice
    d[1], p[1] = 6, ids[(0, 1, KIND_NIC)]
    assert oc.lanes_feasible(d, p) == 0


def test_crossbar_catalog(oracle_lib):
    cat = crossbar_catalog(crossbar_topology(5))
    oc = _oc(oracle_lib, cat)
    assert oc.check() == 0 and oc.covers()
    assert (oc.n_shapes, oc.n_families, oc.G, oc.g) == (1, 1, 1, 5)
