"""GPU parity: vp_schedule_batch (through the C ABI) against the CPU oracle, bit for bit."""
import os

import numpy as np
import pytest
import torch

from workloads import (SchedParams as WParams, complete_catalog, crossbar_catalog, crossbar_topology,
                       node_template_catalog, tree_topology, uniform_demand)
from workloads.configs import build_config
from workloads.topology import Catalog

pytestmark = pytest.mark.gpu

KEYS = ("status", "n_steps", "tau_ns", "chan_id", "lane_dst", "lane_inst", "lane_bytes", "send_off", "recv_off")


@pytest.fixture(scope="module")
def vp():
    import paper_2609_34340_b200 as vp
    assert torch.cuda.is_available(), "these tests need a GPU"
    assert os.path.exists(vp.library_path()), "libvariopath.so has not been built"
    return vp


def _params(vp, w: WParams):
    return vp.SchedParams(lambda_ns=w.lambda_ns, granule_bytes=w.granule_bytes, k_target=w.k_target,
                          n_start=w.n_start, i_aa=w.i_aa, k_max=w.k_max)


def _both(vp, oracle_lib, cat, demand, wparams, tau=None, threads=8):
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    D = torch.as_tensor(demand, dtype=torch.int64)
    tau_t = None if tau is None else torch.as_tensor(tau, dtype=torch.int64).cuda()
    plan = vp.schedule_batch(dc, _params(vp, wparams), D.cuda().contiguous(), tau_t)
    torch.cuda.synchronize()
    got = plan.cpu()
    want = oc.schedule_batch(D.numpy(), wparams, tau_in=None if tau is None else np.asarray(tau), threads=threads)
    return got, want, oc, dc


def _assert_same(got, want, which=None):
    for k in KEYS:
        g, w = got[k], want[k]
        if which is not None:
            g, w = g[which], w[which]
        if not np.array_equal(g, w):
            bad = np.argwhere(np.asarray(g) != np.asarray(w))
            raise AssertionError(f"{k} differs at {bad[:5].tolist()} ({len(bad)} entries); "
                                 f"got {np.asarray(g)[tuple(bad[0])]} want {np.asarray(w)[tuple(bad[0])]}")


def _random_batch(rng, B, N, u, hi, density):
    D = rng.integers(0, hi + 1, size=(B, N, N)) * (rng.random((B, N, N)) < density) * u
    for b in range(B):
        np.fill_diagonal(D[b], 0)
    return D.astype(np.int64)


TOPOS = {
    "node8": lambda: complete_catalog(tree_topology(1)),
    "node8_64_50": lambda: complete_catalog(tree_topology(1, pcie_bw=64, nic_bw=50)),
    "fig1_g3": lambda: complete_catalog(tree_topology(1, g=3, pcie_bw=64, nic_bw=50)),
    "g2_two_nodes": lambda: complete_catalog(tree_topology(2, g=2)),
    "g1_two_nodes": lambda: complete_catalog(tree_topology(2, g=1)),
    "two_nodes": lambda: complete_catalog(tree_topology(2)),
    "two_nodes_64_50": lambda: complete_catalog(tree_topology(2, pcie_bw=64, nic_bw=50)),
    "template_4_nodes": lambda: node_template_catalog(tree_topology(4)),
    "template_3_nodes_g3": lambda: node_template_catalog(tree_topology(3, g=3, nic_bw=50)),
    "template_3_nodes_64_50": lambda: node_template_catalog(tree_topology(3, pcie_bw=64, nic_bw=50)),
    "crossbar4": lambda: crossbar_catalog(crossbar_topology(4)),
}


@pytest.mark.parametrize("name", sorted(TOPOS))
def test_random_demands_match_oracle(vp, oracle_lib, name):
    cat = TOPOS[name]()
    N = cat.topology.N
    rng = np.random.default_rng(sum(map(ord, name)))
    for u, hi, density, lam in [(256, 3, 1.0, 8000), (1, 100000, 0.5, 0), (4096, 50, 0.15, 123), (64, 1, 0.05, 8000)]:
        D = _random_batch(rng, 37, N, u, hi, density)
        D[5] = 0                                     # an empty matrix inside the batch
        w = WParams(lambda_ns=lam, granule_bytes=u, n_start=0).resolved(N)
        got, want, oc, _ = _both(vp, oracle_lib, cat, D, w)
        assert (want["status"] == 0).all()
        _assert_same(got, want)


def test_parameters_and_tau_override(vp, oracle_lib):
    cat = complete_catalog(tree_topology(2))
    rng = np.random.default_rng(3)
    D = _random_batch(rng, 16, 16, 512, 200, 0.7)
    for w in [WParams(granule_bytes=512, n_start=1, i_aa=1, k_target=16, k_max=200),
              WParams(granule_bytes=512, n_start=2, i_aa=5, k_target=48, k_max=300),
              WParams(granule_bytes=512, n_start=7, i_aa=2, k_target=5, k_max=64, lambda_ns=0)]:
        tau = rng.integers(0, 3, size=16) * rng.integers(1, 5000, size=16)   # 0 = derive
        got, want, *_ = _both(vp, oracle_lib, cat, D, w.resolved(16), tau=tau)
        _assert_same(got, want)


def test_status_codes_and_partial_plans(vp, oracle_lib):
    cat = complete_catalog(tree_topology(1))
    good = uniform_demand(8, 6400).numpy()
    D = np.stack([good] * 8)
    D[1, 2, 2] = 64                 # diagonal
    D[2, 1, 3] = -64                # negative
    D[3, 1, 3] = 65                 # not a granule multiple
    D[4, 1, 3] = 1 << 40            # overflow risk
    D[5, 0, 0] = -1; D[5, 4, 5] = 3  # several flags at once
    tau = np.zeros(8, np.int64); tau[6] = (1 << 40) + 1
    w = WParams(granule_bytes=64).resolved(8)
    got, want, *_ = _both(vp, oracle_lib, cat, D, w, tau=tau)
    _assert_same(got, want)
    assert got["status"].tolist() == [0, vp.ST_DIAG_NONZERO, vp.ST_NEGATIVE, vp.ST_NOT_GRANULE, vp.ST_OVERFLOW_RISK,
                                      vp.ST_NEGATIVE | vp.ST_NOT_GRANULE, vp.ST_BAD_TAU, 0]
    # step limit
    w = WParams(granule_bytes=64, k_max=5).resolved(8)
    got, want, *_ = _both(vp, oracle_lib, cat, D[:1], w)
    _assert_same(got, want)
    assert got["status"][0] == vp.ST_STEP_LIMIT and got["n_steps"][0] == 5
    # uncovered: a catalog with the all-PIX shape only
    only_pix = Catalog(cat.topology, [cat.shapes[-1]], [cat.buckets[-1]])
    got, want, _, dc = _both(vp, oracle_lib, only_pix, D[:1], WParams(granule_bytes=64).resolved(8))
    _assert_same(got, want)
    assert got["status"][0] == vp.ST_UNCOVERED and dc.covered == 0


def test_library_rejects_bad_arguments(vp):
    cat = complete_catalog(tree_topology(1))
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    D = uniform_demand(8, 64).unsqueeze(0).cuda()
    with pytest.raises(vp.VpError) as e:
        vp.schedule_batch(dc, vp.SchedParams(granule_bytes=0), D)
    assert e.value.code == vp.E_BAD_ARG
    with pytest.raises(vp.VpError) as e:
        vp.schedule_batch(dc, vp.SchedParams(), D, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == vp.E_WORKSPACE
    with pytest.raises(vp.VpError) as e:
        vp.load_catalog(cat.topology.blob(), cat.blob()[:-2])
    assert e.value.code == vp.E_BAD_CATALOG
    big = crossbar_catalog(crossbar_topology(6))
    with pytest.raises(vp.VpError) as e:
        vp.load_catalog(big.topology.blob(), big.blob())
    assert e.value.code == vp.E_UNSUPPORTED
    info = dc
    assert (info.N, info.G, info.g, info.n_shapes, info.n_families, info.covered) == (8, 2, 4, 3, 6, 1)


def test_deterministic_and_batch_independent(vp, oracle_lib):
    c = build_config(2, device="cuda", batch=24)
    cat = c["catalog"]
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    p = _params(vp, c["params"])
    D = c["demand"].cuda()
    a = vp.schedule_batch(dc, p, D).cpu()
    b = vp.schedule_batch(dc, p, D).cpu()
    one = [vp.schedule_batch(dc, p, D[i:i + 1].contiguous()).cpu() for i in (0, 7, 23)]
    torch.cuda.synchronize()
    for k in KEYS:
        assert np.array_equal(a[k], b[k])
        for i, o in zip((0, 7, 23), one):
            assert np.array_equal(a[k][i], o[k][0])


def test_host_buffer_variant(vp, oracle_lib):
    c = build_config(1, device="cuda", batch=8)
    cat = c["catalog"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    plan = vp.schedule_batch_host(dc, _params(vp, c["params"]), c["demand"].pin_memory())
    want = oc.schedule_batch(c["demand"].numpy(), c["params"])
    _assert_same(plan.cpu(), want)


def test_host_buffer_variant_used_rows_only(vp, oracle_lib):
    """vp_schedule_batch_host_used: rows below n_steps (and offset row n_steps) equal the oracle's; rows beyond keep what
    the host buffers held before the call."""
    c = build_config(2, device="cuda", batch=9, token_scale=0.5)
    cat = c["catalog"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    p = _params(vp, c["params"])
    plan = vp.Plan.empty(9, 16, p.k_max, "cpu", pin=True)
    marks = dict(chan_id=-77, lane_dst=-55, lane_inst=1234, lane_bytes=-99, send_off=-11, recv_off=-13)
    for name, v in marks.items():
        getattr(plan, name).fill_(v)
    vp.schedule_batch_host(dc, p, c["demand"].pin_memory(), plan=plan, used_only=True)
    want = oc.schedule_batch(c["demand"].numpy(), c["params"])
    got = plan.cpu()
    assert np.array_equal(got["n_steps"], want["n_steps"]) and np.array_equal(got["status"], want["status"])
    assert np.array_equal(got["tau_ns"], want["tau_ns"])
    for b in range(9):
        K = int(want["n_steps"][b])
        assert 0 < K < p.k_max - 1
        for name in ("chan_id", "lane_dst", "lane_inst", "lane_bytes"):
            assert np.array_equal(got[name][b][:K], want[name][b][:K]), (name, b)
            assert (got[name][b][K:] == (marks[name] if name != "lane_inst" else 1234)).all(), (name, b)
        for name in ("send_off", "recv_off"):
            assert np.array_equal(got[name][b][:K + 1], want[name][b][:K + 1]), (name, b)
            assert (got[name][b][K + 1:] == marks[name]).all(), (name, b)


@pytest.mark.parametrize("used_only", [False, True])
def test_host_buffer_variant_in_chunks(vp, oracle_lib, used_only):
    """Batches of 64 matrices and more go through the host-buffer call in chunks, two in flight on two streams (ragged
    last chunk, tau given per matrix, one invalid matrix): the same plans as the oracle's, chunk by chunk."""
    c = build_config(2, device="cuda", batch=203, token_scale=0.25)
    cat = c["catalog"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    p = _params(vp, c["params"])
    D = c["demand"].clone()
    D[77, 3, 3] = c["params"].granule_bytes              # an invalid matrix in the middle chunk
    tau = torch.zeros(203, dtype=torch.int64)
    tau[::5] = 40_000                                   # a given quantum for every fifth matrix
    plan = vp.Plan.empty(203, 16, p.k_max, "cpu", pin=True)
    for name in ("chan_id", "lane_dst", "lane_inst", "lane_bytes", "send_off", "recv_off"):
        getattr(plan, name).fill_(-7 if name != "lane_inst" else 777)
    for _ in range(2):                                  # the second call reuses the streams and events of the first
        vp.schedule_batch_host(dc, p, D.pin_memory(), tau.pin_memory(), plan=plan, used_only=used_only)
    want = oc.schedule_batch(D.numpy(), c["params"], tau_in=tau.numpy(), threads=os.cpu_count())
    got = plan.cpu()
    assert got["status"][77] == vp.ST_DIAG_NONZERO and got["n_steps"][77] == 0
    assert (np.delete(got["status"], 77)[np.delete(tau.numpy(), 77) == 0] == 0).all()   # (a small given quantum may hit k_max)
    if not used_only:
        _assert_same(got, want)
        return
    for key in ("n_steps", "status", "tau_ns"):
        assert np.array_equal(got[key], want[key]), key
    for b in range(203):
        K = int(want["n_steps"][b])
        for name in ("chan_id", "lane_dst", "lane_inst", "lane_bytes"):
            assert np.array_equal(got[name][b][:K], want[name][b][:K]), (name, b)
            assert (got[name][b][K:] == (-7 if name != "lane_inst" else 777)).all(), (name, b)
        for name in ("send_off", "recv_off"):
            assert np.array_equal(got[name][b][:K + 1], want[name][b][:K + 1]), (name, b)
            assert (got[name][b][K + 1:] == -7).all(), (name, b)


@pytest.mark.parametrize("idx", [1, 2])
def test_config_full_batch(vp, oracle_lib, idx):
    c = build_config(idx, device="cuda")
    got, want, oc, _ = _both(vp, oracle_lib, c["catalog"], c["demand"], c["params"], threads=os.cpu_count())
    assert (want["status"] == 0).all()
    _assert_same(got, want)


def _validate_all(oc, D, got, granule):
    for b in range(D.shape[0]):
        plan = {k: got[k][b] for k in KEYS}
        assert got["status"][b] == 0, f"matrix {b}: status {got['status'][b]} after {got['n_steps'][b]} steps"
        assert oc.check_plan(D[b], plan, int(got["tau_ns"][b]), granule) == 0, f"matrix {b} invalid"
        K = int(got["n_steps"][b])
        assert (got["send_off"][b][K] == D[b].sum(1)).all() and (got["recv_off"][b][K] == D[b].sum(0)).all()


def test_config3_full_batch(vp, oracle_lib):
    """1024 matrices, N=64: all 1024 plans are compared with the oracle's bit for bit (and checked for validity)."""
    c = build_config(3, device="cuda")
    cat, w = c["catalog"], c["params"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    assert dc.node_symmetric == 1
    D = c["demand"]
    got = vp.schedule_batch(dc, _params(vp, w), D.cuda()).cpu()
    Dn = D.numpy()
    _validate_all(oc, Dn, got, w.granule_bytes)
    want = oc.schedule_batch(Dn, w, threads=os.cpu_count())
    _assert_same(got, want)


CONFIG4_COMPARED = 1024


def test_config4_full_batch(vp, oracle_lib):
    """4096 matrices, N=256, scheduled in sub-batches that reuse the output buffers.  Every plan is checked for
    validity; 1024 of them (every fourth matrix of the seeded shuffle) are compared with the oracle's bit for bit,
    which covers every class of the recipe many times over: sequence-parallel matrices, MoE matrices of each
    popularity exponent, token counts from 1 to 16384 per GPU."""
    c = build_config(4, device="cuda")
    cat, w = c["catalog"], c["params"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    assert dc.node_symmetric == 1 and (dc.n_shapes, dc.n_families) == (4095, 4160)
    D = c["demand"]
    p = _params(vp, w)
    sub = 128
    stride = D.shape[0] // CONFIG4_COMPARED
    plan = vp.Plan.empty(sub, 256, p.k_max, "cuda")
    kept = {k: [] for k in KEYS}
    for lo in range(0, D.shape[0], sub):
        part = D[lo:lo + sub]
        plan = vp.schedule_batch(dc, p, part.cuda().contiguous(), plan=plan)
        got = plan.cpu()
        _validate_all(oc, part.numpy(), got, w.granule_bytes)
        for k in KEYS:
            kept[k].append(np.array(got[k][::stride], copy=True))
    Dn = D.numpy()[::stride]
    # the recipe's classes are all among the compared matrices
    cross_node = np.array([m.reshape(32, 8, 32, 8).sum(axis=(1, 3))[~np.eye(32, dtype=bool)].any() for m in Dn])
    per_rank = Dn.sum(axis=2).max(axis=1) // w.granule_bytes
    assert (~cross_node).sum() > 300 and cross_node.sum() > 300                   # sequence-parallel and MoE
    assert (per_rank[cross_node] <= 8 * 56 * 2).any() and (per_rank[cross_node] > 8 * 56 * 4096).any()   # few and many tokens
    # interleaved split so that every oracle thread gets the same mix of long and short decompositions
    n_thr = os.cpu_count() or 1
    order = np.concatenate([np.arange(t, len(Dn), n_thr) for t in range(n_thr)])
    want = oc.schedule_batch(np.ascontiguousarray(Dn[order]), w, threads=n_thr)
    gotc = {k: np.concatenate(kept[k])[order] for k in KEYS}
    _assert_same(gotc, want)


def test_extreme_values_stay_exact(vp, oracle_lib):
    """Entries just below 2^40, lambda just below 2^40, tau at its limit, mixed rates (rate lcm 1600):
    the 128-bit utility compare and the 64-bit byte path must agree with the oracle's __int128."""
    cat = complete_catalog(tree_topology(2, pcie_bw=64, nic_bw=50))
    rng = np.random.default_rng(17)
    big = (1 << 40) - 1
    D = np.zeros((6, 16, 16), np.int64)
    D[0] = rng.integers(big - 1000, big + 1, size=(16, 16))
    D[1] = rng.integers(0, 2, size=(16, 16)) * big
    D[2] = rng.integers(0, big + 1, size=(16, 16))
    D[3, 0, 9] = big
    D[4] = rng.integers(0, 3, size=(16, 16))
    D[5] = rng.integers(big // 2, big, size=(16, 16)) * (rng.random((16, 16)) < 0.2)
    for b in range(6):
        np.fill_diagonal(D[b], 0)
    tau = np.array([0, 0, 1 << 40, 1, 0, 12345], np.int64)
    w = WParams(lambda_ns=(1 << 40) - 1, granule_bytes=1, k_target=7, k_max=400).resolved(16)
    got, want, *_ = _both(vp, oracle_lib, cat, D, w, tau=tau)
    _assert_same(got, want)
    assert (got["status"] & ~vp.ST_STEP_LIMIT == 0).all()
    # the same matrices scaled to a 4096-byte granule take the 32-bit unit path where capacities allow
    D2 = (D // 4096) * 4096
    w2 = WParams(lambda_ns=0, granule_bytes=4096, k_target=48, k_max=400).resolved(16)
    got, want, *_ = _both(vp, oracle_lib, cat, D2, w2)
    _assert_same(got, want)


def _tiled_case(vp, oracle_lib, cat, base, wparams, reps, tau=None):
    """Schedules ``reps`` copies of the base batch in one call (so that the batch exceeds one wave of CTAs and the
    warp-per-matrix kernel runs) and compares every copy with the oracle's plan of the base matrix."""
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    D = torch.as_tensor(base, dtype=torch.int64)
    nb = D.shape[0]
    big = D.repeat(reps, 1, 1).contiguous()
    tau_t = None if tau is None else torch.as_tensor(np.tile(tau, reps), dtype=torch.int64).cuda()
    p = _params(vp, wparams)
    info = vp.schedule_launch_info(dc, big.shape[0], p)
    assert info["kernel"] == "warp per matrix", info
    got = vp.schedule_batch(dc, p, big.cuda(), tau_t).cpu()
    want = oc.schedule_batch(D.numpy(), wparams, tau_in=None if tau is None else np.asarray(tau), threads=8)
    for r in range(reps):
        for key in KEYS:
            g = got[key][r * nb:(r + 1) * nb]
            if not np.array_equal(g, want[key]):
                bad = np.argwhere(np.asarray(g) != np.asarray(want[key]))
                raise AssertionError(f"copy {r}: {key} differs at {bad[:5].tolist()} ({len(bad)} entries)")
    return got, want


@pytest.mark.parametrize("name", ["node8", "node8_64_50", "two_nodes", "two_nodes_64_50"])
def test_warp_kernel_random_demands(vp, oracle_lib, name):
    """Batches beyond one wave take the one-warp-per-matrix kernel: same plans, bit for bit (32-bit granule units
    and 64-bit byte values, uniform and mixed rates, empty matrices, several parameter sets)."""
    cat = TOPOS[name]()
    N = cat.topology.N
    rng = np.random.default_rng(sum(map(ord, name)) + 1)
    for u, hi, density, lam, extra in [(256, 3, 1.0, 8000, {}), (1, 100000, 0.5, 0, {}), (4096, 50, 0.15, 123, {"n_start": 1, "i_aa": 1}),
                                       (64, 1, 0.05, 8000, {"n_start": 7, "i_aa": 2, "k_target": 5}),
                                       (512, 300, 0.8, 8000, {"n_start": 2, "i_aa": 5, "k_target": 48})]:
        D = _random_batch(rng, 100, N, u, hi, density)
        D[5] = 0
        w = WParams(lambda_ns=lam, granule_bytes=u, **extra).resolved(N)
        tau = rng.integers(0, 3, size=100) * rng.integers(1, 5000, size=100) if extra else None
        _tiled_case(vp, oracle_lib, cat, D, w, reps=26, tau=tau)


def test_warp_kernel_status_codes_and_extremes(vp, oracle_lib):
    cat = complete_catalog(tree_topology(1))
    good = uniform_demand(8, 6400).numpy()
    D = np.stack([good] * 8)
    D[1, 2, 2] = 64
    D[2, 1, 3] = -64
    D[3, 1, 3] = 65
    D[4, 1, 3] = 1 << 40
    D[5, 0, 0] = -1; D[5, 4, 5] = 3
    tau = np.zeros(8, np.int64); tau[6] = (1 << 40) + 1
    got, want = _tiled_case(vp, oracle_lib, cat, D, WParams(granule_bytes=64).resolved(8), reps=330, tau=tau)
    assert got["status"][:8].tolist() == [0, vp.ST_DIAG_NONZERO, vp.ST_NEGATIVE, vp.ST_NOT_GRANULE, vp.ST_OVERFLOW_RISK,
                                          vp.ST_NEGATIVE | vp.ST_NOT_GRANULE, vp.ST_BAD_TAU, 0]
    got, want = _tiled_case(vp, oracle_lib, cat, D[:1], WParams(granule_bytes=64, k_max=5).resolved(8), reps=2600)
    assert got["status"][0] == vp.ST_STEP_LIMIT and got["n_steps"][-1] == 5
    only_pix = Catalog(cat.topology, [cat.shapes[-1]], [cat.buckets[-1]])
    got, want = _tiled_case(vp, oracle_lib, only_pix, D[:1], WParams(granule_bytes=64).resolved(8), reps=2600)
    assert got["status"][-1] == vp.ST_UNCOVERED
    # entries, lambda and tau at their limits with mixed rates: the 64-bit path and the 128-bit utility compare
    cat2 = complete_catalog(tree_topology(2, pcie_bw=64, nic_bw=50))
    rng = np.random.default_rng(17)
    big = (1 << 40) - 1
    E = np.zeros((6, 16, 16), np.int64)
    E[0] = rng.integers(big - 1000, big + 1, size=(16, 16))
    E[1] = rng.integers(0, 2, size=(16, 16)) * big
    E[2] = rng.integers(0, big + 1, size=(16, 16))
    E[3, 0, 9] = big
    E[4] = rng.integers(0, 3, size=(16, 16))
    E[5] = rng.integers(big // 2, big, size=(16, 16)) * (rng.random((16, 16)) < 0.2)
    for b in range(6):
        np.fill_diagonal(E[b], 0)
    tau = np.array([0, 0, 1 << 40, 1, 0, 12345], np.int64)
    w = WParams(lambda_ns=(1 << 40) - 1, granule_bytes=1, k_target=7, k_max=400).resolved(16)
    _tiled_case(vp, oracle_lib, cat2, E, w, reps=420, tau=tau)
    E2 = (E // 4096) * 4096
    _tiled_case(vp, oracle_lib, cat2, E2, WParams(lambda_ns=0, granule_bytes=4096, k_target=48, k_max=400).resolved(16), reps=420)


def test_warp_kernel_config2_tiled(vp, oracle_lib):
    c = build_config(2)
    _tiled_case(vp, oracle_lib, c["catalog"], c["demand"].numpy(), c["params"], reps=4)


@pytest.mark.parametrize("nodes", [12, 16, 24])
def test_mid_size_template_catalogs(vp, oracle_lib, nodes):
    """N = 96, 128, 192 with node-template catalogs of 575 .. 2,303 shapes: incremental scores with one warp per task
    (G <= 32) and with two warps per task (G > 32), 32-bit granule units and 64-bit byte values, mixed rates."""
    cat = node_template_catalog(tree_topology(nodes, pcie_bw=64, nic_bw=50 if nodes == 16 else 64))
    N = cat.topology.N
    rng = np.random.default_rng(nodes)
    for u, hi, density, extra in [(4096, 40, 0.3, {}), (1, 3_000_000, 0.05, {"n_start": 2, "i_aa": 2}), (256, 2, 1.0, {"k_target": 40})]:
        D = _random_batch(rng, 5, N, u, hi, density)
        D[3] = 0
        w = WParams(granule_bytes=u, k_max=16 * N, **extra).resolved(N)
        got, want, *_ = _both(vp, oracle_lib, cat, D, w)
        _assert_same(got, want)


@pytest.mark.parametrize("nodes", [9, 32])
def test_large_capacities_and_hot_columns(vp, oracle_lib, nodes):
    """Node-symmetric catalogs of more than sixteen groups with lane capacities of 2^16 granules and more: a few columns
    (popular destinations) hold cells far above 65,535 granules and are kept exactly beside the 16-bit credits; with
    too many such columns, or capacities of 2^22 granules and more, the general kernel takes the matrix.  Mixed in one
    batch with ordinary matrices, uniform and mixed rates."""
    cat = node_template_catalog(tree_topology(nodes, pcie_bw=64, nic_bw=50 if nodes == 9 else 64))
    N = cat.topology.N
    rng = np.random.default_rng(100 + nodes)
    u = 256
    B = 7
    D = (rng.integers(0, 3000, size=(B, N, N)) * (rng.random((B, N, N)) < 0.5)).astype(np.int64)
    hot = rng.choice(N, size=5, replace=False)
    D[0][:, hot] = rng.integers(60_000, 3_000_000, size=(N, 5))          # five hot columns, capacity well above 2^16
    D[1][:, hot[:2]] = rng.integers(65_535, 65_540, size=(N, 2))         # cells right at the 16-bit boundary
    D[2][:, rng.choice(N, size=40, replace=False)] = 200_000             # more hot columns than are kept: general kernel
    D[3][:, hot[:1]] = rng.integers(1 << 27, 1 << 28, size=(N, 1))       # capacity of 2^22 granules and more: general kernel
    D[4][hot[:3], :] = rng.integers(60_000, 900_000, size=(3, N))        # hot rows instead: every column is hot or none
    D[5] = 0
    D *= u
    for b in range(B):
        np.fill_diagonal(D[b], 0)
    for extra in ({}, {"n_start": 2, "i_aa": 5, "lambda_ns": 0}):
        w = WParams(granule_bytes=u, k_max=12 * N, **extra).resolved(N)
        got, want, *_ = _both(vp, oracle_lib, cat, D, w)
        _assert_same(got, want)
    tau = np.array([0, 70_000 * u // 50, 0, 0, 0, 1, 0], np.int64)       # a given quantum that puts matrix 1 in hot mode
    got, want, *_ = _both(vp, oracle_lib, cat, D, WParams(granule_bytes=u, k_max=12 * N).resolved(N), tau=tau)
    _assert_same(got, want)


@pytest.mark.parametrize("nodes", [9, 32])
def test_big_cells_beside_16_bit_credits(vp, oracle_lib, nodes):
    """Capacities below 2^16 granules with cells far above: such cells are kept exactly in a side list (16 N entries, at
    most 4,096) and the matrix holds their indices.  Cells right at the boundary value, a sparse block-diagonal matrix
    whose every cell is big, cells that shrink below the boundary while the matrix is decomposed, and more big cells
    than the list holds (the general kernel takes that matrix)."""
    cat = node_template_catalog(tree_topology(nodes, pcie_bw=64, nic_bw=50 if nodes == 9 else 64))
    N = cat.topology.N
    side = min(16 * N, 4096)
    floor = 65536 - side
    rng = np.random.default_rng(300 + nodes)
    u = 256
    B = 6
    D = (rng.integers(0, 3000, size=(B, N, N)) * (rng.random((B, N, N)) < 0.3)).astype(np.int64)
    D[0] = 0
    for i in range(N):                                                    # eight partners per rank, every cell big
        D[0][i, [(i // 8) * 8 + m for m in range(8)]] = rng.integers(70_000, 200_000)
    mask = rng.random((N, N)) < 0.02
    D[1][mask] = rng.integers(floor - 2, floor + 3, size=int(mask.sum()))   # right at the boundary
    over = rng.random((N, N)) < 1.3 * side / (N * N)                      # more big cells than the list holds
    D[2][over] = rng.integers(66_000, 90_000, size=int(over.sum()))
    assert int(over.sum()) - N > side
    D[3][rng.random((N, N)) < min(0.9 * side / (N * N), 0.5)] = 1_000_000  # just within the list, far above the boundary
    D[4][: N // 2] = rng.integers(floor - 500, floor + 500, size=(N // 2, N))
    D *= u
    for b in range(B):
        np.fill_diagonal(D[b], 0)
    for extra in ({}, {"k_target": 64}, {"n_start": 2, "i_aa": 5, "lambda_ns": 0}):
        w = WParams(granule_bytes=u, k_max=40 * N, **extra).resolved(N)
        got, want, *_ = _both(vp, oracle_lib, cat, D, w)
        _assert_same(got, want)
        if "n_start" not in extra:                     # (fewer starts than ranks per group can end in "no progress")
            assert int(np.asarray(want["n_steps"]).min()) > 0 and (np.asarray(want["status"]) == 0).all()


@pytest.mark.parametrize("granule", [256, 768])
def test_status_codes_on_large_catalogs(vp, oracle_lib, granule):
    """Invalid entries in matrices that take the kernel for large node-symmetric catalogs, with a power-of-two granule
    and with another one: the same status words as the oracle, in any combination, and untouched neighbours."""
    cat = node_template_catalog(tree_topology(9, pcie_bw=64, nic_bw=50))
    N = cat.topology.N
    rng = np.random.default_rng(granule)
    D = (rng.integers(0, 500, size=(9, N, N)) * (rng.random((9, N, N)) < 0.4)).astype(np.int64) * granule
    for b in range(9):
        np.fill_diagonal(D[b], 0)
    D[1, 5, 5] = granule                       # diagonal
    D[2, 70, 3] = -granule                     # negative
    D[3, 33, 64] += 1                          # not a granule multiple
    D[4, 71, 0] = 1 << 40                      # overflow risk
    D[5, 0, 0] = -1; D[5, 40, 41] = 3; D[5, 8, 9] = (1 << 40) + 5; D[5, 7, 7] = granule
    D[6, 2, 2] = (1 << 40) + 1                 # on the diagonal and over the limit: only the limit is reported
    D[7, 3, 3] = -3                            # negative on the diagonal: only "negative"
    w = WParams(granule_bytes=granule, k_max=12 * N).resolved(N)
    got, want, _, dc = _both(vp, oracle_lib, cat, D, w)
    _assert_same(got, want)
    p = _params(vp, w)
    assert vp.schedule_launch_info(dc, 9, p)["kernel"] == "CTA per matrix, 16-bit credits"
    assert got["status"].tolist() == [0, vp.ST_DIAG_NONZERO, vp.ST_NEGATIVE, vp.ST_NOT_GRANULE, vp.ST_OVERFLOW_RISK,
                                      vp.ST_NEGATIVE | vp.ST_NOT_GRANULE | vp.ST_OVERFLOW_RISK | vp.ST_DIAG_NONZERO,
                                      vp.ST_OVERFLOW_RISK, vp.ST_NEGATIVE, 0]


@pytest.mark.parametrize("nodes,nic_bw", [(24, 64), (20, 50)])
def test_class_wise_argmax_on_other_catalogs(vp, oracle_lib, nodes, nic_bw):
    """Two-rail node-template catalogs of more than 1,024 shapes take Step 1 class by class (2,303 shapes at 24 nodes,
    1,599 at 20 nodes with two path rates).  Matrices whose shape scores tie massively (every cell equal; equal cells
    inside the switches only; equal cells between the two switches of a node only) check that the first maximum is
    the same shape as in the oracle's scan; the others are random sparse, dense and flat, and a single cell."""
    cat = node_template_catalog(tree_topology(nodes, pcie_bw=64, nic_bw=nic_bw))
    N = cat.topology.N
    assert cat.n_shapes >= 1024
    rng = np.random.default_rng(nodes)
    u = 256
    B = 7
    D = (rng.integers(0, 2000, size=(B, N, N)) * (rng.random((B, N, N)) < 0.4)).astype(np.int64)
    D[1] = 1000                                              # every shape with the same lane count ties
    D[2] = 0
    D[3] = 0
    for n in range(nodes):
        lo = n * 8
        for g0 in (lo, lo + 4):
            D[2][g0:g0 + 4, g0:g0 + 4] = 700                 # inside the switches only
        D[3][lo:lo + 4, lo + 4:lo + 8] = 500                 # between the two switches of a node only
        D[3][lo + 4:lo + 8, lo:lo + 4] = 500
    D[4] = rng.integers(0, 300, size=(N, N))                 # dense and flat
    D[5] = 0
    D[5][5, 9] = 77                                          # a single cell
    D *= u
    for b in range(B):
        np.fill_diagonal(D[b], 0)
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    for extra in ({}, {"lambda_ns": 0, "k_target": N}):
        w = WParams(granule_bytes=u, k_max=10 * N, **extra).resolved(N)
        p = _params(vp, w)
        plan = vp.schedule_batch(dc, p, torch.from_numpy(D).cuda())
        torch.cuda.synchronize()
        want = oc.schedule_batch(D, w, threads=B)
        _assert_same(plan.cpu(), want)
        assert (np.asarray(want["status"]) == 0).all()
    assert vp.schedule_launch_info(dc, B, p)["kernel"] == "CTA per matrix, 16-bit credits"


def test_plan_arrays_at_odd_addresses(vp, oracle_lib):
    """Plan arrays that are aligned to their element size only (2, 8 bytes), not to 16: the kernel for large catalogs
    then writes emit rows and idle rows with plain stores instead of staged 16-byte copies and bulk copies.  Also the
    demand at an address that is 8 bytes off a 16-byte boundary."""
    cat = node_template_catalog(tree_topology(32))
    N = cat.topology.N
    rng = np.random.default_rng(77)
    B = 5
    D = (rng.integers(0, 4000, size=(B, N, N)) * (rng.random((B, N, N)) < 0.3)).astype(np.int64) * 256
    for b in range(B):
        np.fill_diagonal(D[b], 0)
    w = WParams(granule_bytes=256, k_max=6 * N).resolved(N)
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    want = oc.schedule_batch(D, w, threads=B)
    p = _params(vp, w)
    K = p.k_max

    def off(shape, dtype, elems):            # a contiguous tensor whose first element sits `elems` elements into an allocation
        n = int(np.prod(shape))
        return torch.empty(n + elems, dtype=dtype, device="cuda")[elems:].view(shape)

    plan = vp.Plan(n_steps=torch.empty(B, dtype=torch.int32, device="cuda"), chan_id=off((B, K), torch.int32, 1),
                   lane_dst=off((B, K, N), torch.int16, 1), lane_inst=off((B, K, N), torch.uint16, 3),
                   lane_bytes=off((B, K, N), torch.int64, 1), send_off=off((B, K + 1, N), torch.int64, 1),
                   recv_off=off((B, K + 1, N), torch.int64, 1), tau_ns=torch.empty(B, dtype=torch.int64, device="cuda"),
                   status=torch.empty(B, dtype=torch.int32, device="cuda"), k_max=K)
    assert plan.lane_dst.data_ptr() % 16 == 2 and plan.lane_bytes.data_ptr() % 16 == 8
    demand = off((B, N, N), torch.int64, 1)
    demand.copy_(torch.from_numpy(D))
    assert demand.data_ptr() % 16 == 8
    vp.schedule_batch(dc, p, demand, plan=plan)
    torch.cuda.synchronize()
    _assert_same(plan.cpu(), want)
    assert vp.schedule_launch_info(dc, B, p)["kernel"] == "CTA per matrix, 16-bit credits"


def test_batches_around_one_wave(vp, oracle_lib):
    """Batch sizes just below and above the number of resident CTAs: the launch changes (a warp or a CTA per matrix, one
    to four warps per CTA), the plans do not.  With the configuration's own granule every batch takes the warp kernel;
    with a granule below 256 bytes the small batches take a CTA per matrix."""
    c = build_config(2)
    cat, w0 = c["catalog"], c["params"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    base = c["demand"][:37]
    for granule, expect in ((w0.granule_bytes, {"warp per matrix"}), (64, {"CTA per matrix", "warp per matrix"})):
        w = WParams(granule_bytes=granule, k_max=w0.k_max).resolved(cat.topology.N)
        want = oc.schedule_batch(base.numpy(), w, threads=8)
        p = _params(vp, w)
        kernels, threads = set(), set()
        for B in (147, 591, 592, 593, 1187, 1190):
            D = base.repeat((B + 36) // 37, 1, 1)[:B].contiguous()
            info = vp.schedule_launch_info(dc, B, p)
            kernels.add(info["kernel"])
            threads.add(info["threads"])
            got = vp.schedule_batch(dc, p, D.cuda()).cpu()
            for key in KEYS:
                for r0 in range(0, B, 37):
                    n = min(37, B - r0)
                    assert np.array_equal(got[key][r0:r0 + n], want[key][:n]), (granule, B, key, r0)
        assert kernels == expect
        if granule >= 256:
            assert threads == {32, 64, 128}            # one, two and four warps per CTA


def test_launches_of_different_sizes_interleaved(vp, oracle_lib):
    """A large batch, a single matrix and the large batch again, on two catalogs that share a kernel: launches are
    replayed from a memo with different amounts of dynamic shared memory, and a later, smaller plan must not shrink
    what an earlier one needs."""
    c2, c1 = build_config(2), build_config(1)
    oc = oracle_lib.OracleCatalog(c2["catalog"].topology.blob(), c2["catalog"].blob())
    dc2 = vp.load_catalog(c2["catalog"].topology.blob(), c2["catalog"].blob())
    dc1 = vp.load_catalog(c1["catalog"].topology.blob(), c1["catalog"].blob())
    p2, p1 = _params(vp, c2["params"]), _params(vp, c1["params"])
    base = c2["demand"][:16]
    want = oc.schedule_batch(base.numpy(), c2["params"], threads=8)
    big = base.repeat(80, 1, 1).contiguous().cuda()            # 1280 matrices: four warps per CTA, the most shared memory
    for B in (1280, 1, 1280, 300, 1280):
        if B == 300:
            vp.schedule_batch(dc1, p1, c1["demand"][:8].cuda())    # another catalog plans the same kernel with less
        got = vp.schedule_batch(dc2, p2, big[:B].contiguous()).cpu()
        torch.cuda.synchronize()
        for key in KEYS:
            for r0 in range(0, B, 16):
                n = min(16, B - r0)
                assert np.array_equal(got[key][r0:r0 + n], want[key][:n]), (B, key, r0)


def test_randomised_topologies_and_parameters(vp, oracle_lib):
    """A seeded sweep over group sizes 1..4, complete and node-template catalogs, mixed rates, granules, densities,
    AA parameters, tau overrides and batch sizes on both sides of one wave: every plan equals the oracle's."""
    rng = np.random.default_rng(2024)
    cats = {}
    choices = [("complete", 1, 4), ("complete", 2, 4), ("complete", 1, 3), ("complete", 2, 2), ("complete", 2, 1),
               ("template", 3, 4), ("template", 4, 4), ("template", 6, 4), ("template", 8, 4), ("template", 3, 3), ("template", 12, 4)]
    for case in range(120):
        kind, nodes, g = choices[rng.integers(len(choices))]
        pb, nb = [(64, 64), (64, 50), (32, 64), (50, 25)][rng.integers(4)]
        key = (kind, nodes, g, pb, nb)
        if key not in cats:
            topo = tree_topology(nodes, g=g, pcie_bw=pb, nic_bw=nb)
            cats[key] = complete_catalog(topo) if kind == "complete" else node_template_catalog(topo)
        cat = cats[key]
        N = cat.topology.N
        u = int([1, 64, 256, 4096, 14336][rng.integers(5)])
        hi = int([1, 3, 50, 1000, 100000][rng.integers(5)])
        density = float([0.03, 0.2, 0.6, 1.0][rng.integers(4)])
        B = int([1, 7, 40][rng.integers(3)]) if N > 16 else int([1, 33, 700][rng.integers(3)])
        base = _random_batch(rng, min(B, 40), N, u, hi, density)
        nb0 = base.shape[0]
        reps = (B + nb0 - 1) // nb0
        D = np.tile(base, (reps, 1, 1))[:B]
        w = WParams(lambda_ns=int([0, 123, 8000][rng.integers(3)]), granule_bytes=u, n_start=int(rng.integers(0, 6)),
                    i_aa=int(rng.integers(0, 5)), k_target=int([0, 5, 48][rng.integers(3)]), k_max=int(min(16 * N, 2048))).resolved(N)
        tau = None
        if rng.random() < 0.3:
            tau = np.tile((rng.integers(0, 3, size=nb0) * rng.integers(1, 5000, size=nb0)).astype(np.int64), reps)[:B]
        oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
        dc = vp.load_catalog(cat.topology.blob(), cat.blob())
        got = vp.schedule_batch(dc, _params(vp, w), torch.from_numpy(D).cuda().contiguous(),
                                None if tau is None else torch.from_numpy(tau).cuda()).cpu()
        want = oc.schedule_batch(base, w, tau_in=None if tau is None else tau[:nb0], threads=8)
        for k in KEYS:
            for r0 in range(0, B, nb0):
                m = min(nb0, B - r0)
                assert np.array_equal(got[k][r0:r0 + m], want[k][:m]), (case, key, u, hi, density, B, k, r0)
