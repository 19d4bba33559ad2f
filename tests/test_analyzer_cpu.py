"""vp_build_catalog (Algorithm 1 in the library, host code): pins and agreement with the input generator."""
import os
import time

import pytest

from workloads.topology import (complete_catalog, crossbar_catalog, crossbar_topology, ring_topology, tree_topology, Topology,
                                Instance)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def vp():
    from paper_2609_34340_b200.build import build
    build()
    import paper_2609_34340_b200 as vp
    return vp


def test_table3_row1(vp, oracle_lib):
    with open(os.path.join(GOLDEN, "table3_row1.txt")) as f:
        shapes, fams = (int(x) for x in [ln for ln in f if not ln.startswith("#")][0].split())
    topo = tree_topology(1)
    blob, ns, nf = vp.build_catalog(topo.blob())
    assert (ns, nf) == (shapes, fams)
    oc = oracle_lib.OracleCatalog(topo.blob(), blob)
    assert oc.check() == 0 and oc.covers()          # Eq. (3), Eq. (4) by the oracle's own checker


@pytest.mark.parametrize("make", [
    lambda: tree_topology(1), lambda: tree_topology(1, g=3, pcie_bw=64, nic_bw=50), lambda: tree_topology(1, g=2),
    lambda: tree_topology(2, g=2), lambda: tree_topology(2, g=1), lambda: tree_topology(2), lambda: tree_topology(3, g=2),
    lambda: crossbar_topology(4)])
def test_same_blob_as_the_python_generator(vp, oracle_lib, make):
    topo = make()
    ref = crossbar_catalog(topo) if topo.G == 1 else complete_catalog(topo)
    blob, ns, nf = vp.build_catalog(topo.blob())
    assert (ns, nf) == (ref.n_shapes, ref.n_families)
    assert blob == ref.blob()
    assert oracle_lib.OracleCatalog(topo.blob(), blob).check() == 0


def test_rate_dominance_pruning(vp):
    """Two parallel paths with the same footprint between two one-GPU switches: the slower family goes."""
    inst = [Instance(0, 1, 1, 64, 1, (0,)), Instance(0, 1, 1, 32, 1, (0,)), Instance(1, 0, 1, 64, 1, (1,))]
    topo = Topology(N=2, G=2, g=1, groups_per_node=2, n_resources=2, instances=inst)
    blob, ns, nf = vp.build_catalog(topo.blob())
    assert (ns, nf) == (1, 1)
    ref = complete_catalog(topo)
    assert blob == ref.blob() and ref.families == [(0, 2)]


def test_errors_and_size_query(vp):
    import ctypes as C
    lib = vp.binding._load()
    topo = tree_topology(1).blob()
    need = C.c_size_t(0)
    assert lib.vp_build_catalog(topo, len(topo), None, 0, C.byref(need), None, None) == 0 and need.value > 24
    small = C.create_string_buffer(8)
    assert lib.vp_build_catalog(topo, len(topo), small, 8, C.byref(need), None, None) == vp.E_WORKSPACE
    assert lib.vp_build_catalog(topo[:40], 40, None, 0, C.byref(need), None, None) == vp.E_BAD_CATALOG
    assert lib.vp_build_catalog(None, 0, None, 0, C.byref(need), None, None) == vp.E_BAD_ARG
    # a switch that cannot reach anything admits no family
    lonely = Topology(N=2, G=2, g=1, groups_per_node=2, n_resources=1, instances=[Instance(0, 1, 1, 64, 1, (0,))])
    lb = lonely.blob()
    assert lib.vp_build_catalog(lb, len(lb), None, 0, C.byref(need), None, None) == vp.E_BAD_CATALOG


def test_construction_time_is_small(vp):
    """Context: the paper reports 0.8 s (8 GPUs) and 4.95 s (16 GPUs) for its analyzer (Table 3)."""
    topo = tree_topology(2).blob()
    t0 = time.perf_counter()
    _, ns, nf = vp.build_catalog(topo)
    dt = time.perf_counter() - t0
    assert (ns, nf) == (89, 152) and dt < 2.0


def test_prune_paths_matches_the_definition(vp):
    """vp_prune_paths against the definition written out: r goes when some r' of the same group pair has
    L(r') within L(r) and bw(r') >= bw(r), one of them strictly (Section 4.1, pruning)."""
    import random
    from workloads.topology import prune_paths
    rng = random.Random(5)
    base = tree_topology(2, pcie_bw=64, nic_bw=50)
    cands = list(base.instances)
    for r in list(base.instances):
        if not r.res:
            continue
        cands.append(Instance(r.src_group, r.dst_group, r.kind, r.bw - 1, 1, r.res))                     # slower twin: dominated
        cands.append(Instance(r.src_group, r.dst_group, r.kind, r.bw, 1, r.res + (base.n_resources,)))   # extra resource: dominated
        cands.append(Instance(r.src_group, r.dst_group, r.kind, r.bw + 9, 1, r.res + (base.n_resources + 1,)))  # faster but wider: stays
        cands.append(Instance(r.src_group, r.dst_group, r.kind, r.bw, 1, r.res))                         # exact twin: both stay
    rng.shuffle(cands)
    cands.sort(key=lambda r: (r.src_group, r.dst_group))
    topo = Topology(base.N, base.G, base.g, base.groups_per_node, base.n_resources + 2, cands)
    want = Topology(base.N, base.G, base.g, base.groups_per_node, base.n_resources + 2, prune_paths(cands))
    got = vp.prune_paths(topo.blob())
    assert got == want.blob()
    assert len(want.instances) < len(cands)
    # the instances a generator hands to Algorithm 1 are already a fixed point
    assert vp.prune_paths(base.blob()) == base.blob()
    # same-switch NIC loop-back next to the switch-local path: the textbook dominated candidate
    pix = Instance(0, 0, 0, 64, 4, ())
    loop = Instance(0, 0, 2, 64, 1, (2, 3))
    two = Topology(4, 1, 4, 1, 4, [pix, loop])
    assert vp.prune_paths(two.blob()) == Topology(4, 1, 4, 1, 4, [pix]).blob()


@pytest.mark.parametrize("nodes,g,nic_bw", [(3, 4, 64), (4, 4, 50), (8, 4, 64), (12, 4, 64), (3, 3, 50), (5, 2, 64), (32, 4, 64)])
def test_template_catalog_same_blob_as_the_python_generator(vp, oracle_lib, nodes, g, nic_bw):
    from workloads.topology import node_template_catalog
    topo = tree_topology(nodes, g=g, nic_bw=nic_bw)
    want = node_template_catalog(topo)
    blob, ns, nf = vp.build_template_catalog(topo.blob())
    assert (ns, nf) == (want.n_shapes, want.n_families)
    assert blob == want.blob()
    if nodes <= 8:                                   # Eq. (3), Eq. (4) by the oracle's own checker
        oc = oracle_lib.OracleCatalog(topo.blob(), blob)
        assert oc.check() == 0 and oc.covers()
    if nodes == 8:
        assert (ns, nf) == (255, 272)
    if nodes == 32:
        assert (ns, nf) == (4095, 4160)


def test_template_catalog_needs_two_groups_per_node(vp):
    with pytest.raises(vp.VpError) as e:
        vp.build_template_catalog(crossbar_topology(4).blob())
    assert e.value.code == vp.E_UNSUPPORTED


def _brute_force_families(topo):
    """Every family of a topology by plain enumeration, written from the definition alone (Section 4.1): each group
    picks g lanes among the instances that leave it; a pick is a family when every group also receives g lanes and no
    directed resource is used twice.  Independent of both catalog builders."""
    from itertools import combinations_with_replacement, product
    per_group = []
    for a in range(topo.G):
        ids = [i for i, r in enumerate(topo.instances) if r.src_group == a]
        picks = [c for c in combinations_with_replacement(ids, topo.g)
                 if all(c.count(i) <= topo.instances[i].mult for i in set(c))]
        per_group.append(picks)
    fams = set()
    for combo in product(*per_group):
        fam = tuple(sorted(i for c in combo for i in c))
        inn = [0] * topo.G
        used = []
        for i in fam:
            inn[topo.instances[i].dst_group] += 1
            used += list(topo.instances[i].res)
        if inn == [topo.g] * topo.G and len(used) == len(set(used)):
            fams.add(fam)
    return fams


def _shape_count(topo, fams):
    shapes = set()
    for f in fams:
        cnt = {}
        for i in f:
            key = (topo.instances[i].src_group, topo.instances[i].dst_group)
            cnt[key] = cnt.get(key, 0) + 1
        shapes.add(tuple(sorted(cnt.items())))
    return len(shapes)


@pytest.mark.parametrize("make", [lambda: tree_topology(2, g=2), lambda: ring_topology(1, switches_per_node=4, g=2),
                                  lambda: ring_topology(1, switches_per_node=3, g=2, pcie_bw=64, nic_bw=50)])
def test_counts_against_plain_enumeration(vp, oracle_lib, make):
    """The two-node tree (g = 2) and one-node rings: the library's catalog holds exactly the families that plain
    enumeration from the definition finds (all rates equal per kind, so PruneFamilies removes nothing but duplicates)."""
    topo = make()
    want = _brute_force_families(topo)
    blob, ns, nf = vp.build_catalog(topo.blob())
    oc = oracle_lib.OracleCatalog(topo.blob(), blob)
    assert oc.check() == 0 and oc.covers()
    got = {tuple(int(x) for x in row) for row in oc.families()}
    assert got == want and nf == len(want) and ns == _shape_count(topo, want)


def test_ring_topology_through_prune_build_and_oracle(vp, oracle_lib):
    """A ring of PCIe switches: candidate paths -> vp_prune_paths -> vp_build_catalog -> the oracle's Eq. (3)/(4)
    checker, coverage, and a schedule whose plans are valid (conservation, Eq. 1, Eq. 9)."""
    import numpy as np
    from workloads import SchedParams
    topo = ring_topology(1, switches_per_node=4, g=2)
    pruned = vp.prune_paths(topo.blob())
    assert pruned == topo.blob()                                         # the generator already pruned: a fixed point
    blob, ns, nf = vp.build_catalog(pruned)
    oc = oracle_lib.OracleCatalog(pruned, blob)
    assert oc.check() == 0 and oc.covers() and ns > 3 and nf >= ns
    # two ring paths per switch pair, one per direction: neither footprint contains the other, so PrunePaths keeps both
    inst = oc.instances()
    assert sorted(len(r[5]) for r in inst if (r[0], r[1], r[2]) == (0, 2, 1)) == [2, 2]
    assert sorted(len(r[5]) for r in inst if (r[0], r[1], r[2]) == (0, 1, 1)) == [1, 3]
    rng = np.random.default_rng(8)
    for _ in range(4):
        D = (rng.integers(0, 40, size=(8, 8)) * (rng.random((8, 8)) < 0.7) * 64).astype(np.int64)
        np.fill_diagonal(D, 0)
        plan = oc.schedule(D, SchedParams(granule_bytes=64).resolved(8))
        assert plan["status"] == 0 and oc.check_plan(D, plan, int(plan["tau_ns"]), 64) == 0


def test_catalog_scale_report(vp, capsys):
    """Catalog scale and build time per topology, in the manner of Table 3 (shapes, families, KiB, seconds); only the
    one-node row is a pin (3 shapes / 6 families), the rest is a report."""
    rows = []
    for name, topo in [("1 node, tree 2 x 4", tree_topology(1)), ("2 nodes, tree 2 x 4", tree_topology(2)),
                       ("3 nodes, tree 2 x 2", tree_topology(3, g=2)), ("1 node, ring 4 x 2", ring_topology(1, 4, 2)),
                       ("1 node, ring 5 x 2", ring_topology(1, 5, 2))]:
        t0 = time.perf_counter()
        blob, ns, nf = vp.build_catalog(topo.blob())
        rows.append((name, topo.N, ns, nf, len(blob) / 1024, time.perf_counter() - t0))
    with capsys.disabled():
        print()
        for name, n, ns, nf, kib, sec in rows:
            print(f"    {name:22s} N={n:3d}  shapes {ns:6d}  families {nf:7d}  {kib:9.1f} KiB  {sec:7.3f} s")
    assert rows[0][2:4] == (3, 6)
