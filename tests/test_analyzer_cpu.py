"""vp_build_catalog (Algorithm 1 in the library, host code): pins and agreement with the input generator."""
import os
import time

import pytest

from workloads.topology import (complete_catalog, crossbar_catalog, crossbar_topology, tree_topology, Topology, Instance)

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
