"""GPU parity of the two kernels around the scheduler: demand from routing, and Eq. (2) plan time."""
import os

import numpy as np
import pytest
import torch

from workloads import SchedParams as WParams, complete_catalog, node_template_catalog, tree_topology
from workloads.configs import build_config
from workloads.demand import moe_routing

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def vp():
    import paper_2609_34340_b200 as vp
    assert torch.cuda.is_available(), "these tests need a GPU"
    assert os.path.exists(vp.library_path()), "libvariopath.so has not been built"
    return vp


@pytest.mark.parametrize("N,E,T,topk", [(16, 256, 8192, 8), (8, 32, 777, 4), (256, 256, 300, 8), (3, 9, 50, 2)])
def test_demand_from_routing_matches_oracle(vp, oracle_lib, N, E, T, topk):
    idx = moe_routing(N * T, E, topk, 1.1, seed=N + T, device="cuda").reshape(N, T, topk).contiguous()
    idx[:, ::7, 0] = -1                                     # some dropped copies
    rb = 14336
    got, st = vp.demand_from_routing(idx, E // N, N, rb)
    want, bad = oracle_lib.demand_from_routing(idx.cpu().numpy(), E // N, N, rb)
    assert int(st.item()) == bad == 0
    assert np.array_equal(got.cpu().numpy(), want)
    assert (np.diag(want) == 0).all()
    # a slice of source ranks written into the middle of a matrix, and an out-of-range index
    D = torch.full((N, N), -1, dtype=torch.int64, device="cuda")
    lo = N // 3
    part = idx[lo:lo + 2].contiguous()
    part[0, 0, 1] = E
    got2, st2 = vp.demand_from_routing(part, E // N, N, rb, src0=lo, out=D[lo:lo + part.shape[0]])
    want2, bad2 = oracle_lib.demand_from_routing(part.cpu().numpy(), E // N, N, rb, src0=lo)
    assert int(st2.item()) == bad2 == 1
    assert np.array_equal(D[lo:lo + part.shape[0]].cpu().numpy(), want2)
    assert (D[:lo] == -1).all() and (D[lo + part.shape[0]:] == -1).all()


@pytest.mark.parametrize("cfg,batch,lam", [(1, 16, 8000), (2, 40, 0), (3, 24, 8000)])
def test_plan_time_matches_eq2_oracle(vp, oracle_lib, cfg, batch, lam):
    c = build_config(cfg, device="cuda", batch=batch, token_scale=0.25)
    cat, w = c["catalog"], c["params"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    p = vp.SchedParams(lambda_ns=w.lambda_ns, granule_bytes=w.granule_bytes, k_target=w.k_target,
                       n_start=w.n_start, i_aa=w.i_aa, k_max=w.k_max)
    plan = vp.schedule_batch(dc, p, c["demand"].cuda())
    got = vp.plan_time(dc, plan, lam).cpu().numpy()
    host = plan.cpu()
    for b in range(batch):
        one = {k: (v[b] if isinstance(v, np.ndarray) else v) for k, v in host.items()}
        assert int(got[b]) == oc.modeled_time_xw(one, lam)


def test_plan_time_with_mixed_rates(vp, oracle_lib):
    cat = complete_catalog(tree_topology(2, pcie_bw=64, nic_bw=50))
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    rng = np.random.default_rng(8)
    D = rng.integers(0, 500, size=(9, 16, 16)) * 64
    for b in range(9):
        np.fill_diagonal(D[b], 0)
    D[4] = 0
    plan = vp.schedule_batch(dc, vp.SchedParams(lambda_ns=123, granule_bytes=64, k_max=128), torch.from_numpy(D).cuda())
    got = vp.plan_time(dc, plan, 123).cpu().numpy()
    host = plan.cpu()
    assert dc.rate_lcm == 1600
    for b in range(9):
        one = {k: (v[b] if isinstance(v, np.ndarray) else v) for k, v in host.items()}
        assert int(got[b]) == oc.modeled_time_xw(one, 123)
    assert got[4] == 0


def test_sweep_plan_time_matches_oracle(vp, oracle_lib):
    """vp_sweep_plan_time over a grid of (lambda, K_target): rate_lcm x T(S) and the activation counts of every grid
    point equal the oracle's, integer for integer; every value is at least the link-load lower bound at lambda = 0."""
    from workloads.configs import build_config
    c = build_config(2, device="cuda", batch=6, token_scale=0.25)
    cat, w = c["catalog"], c["params"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    p = vp.SchedParams(lambda_ns=w.lambda_ns, granule_bytes=w.granule_bytes, k_target=w.k_target, n_start=w.n_start,
                       i_aa=w.i_aa, k_max=w.k_max)
    lambdas, k_targets = [0, 8000], [16, 32, 48]
    T, K, st = vp.sweep_plan_time(dc, p, c["demand"].cuda().contiguous(), lambdas, k_targets)
    torch.cuda.synchronize()
    wantT, wantK = oc.sweep_plan_time(c["demand"].numpy(), w, lambdas, k_targets, threads=4)
    assert (st.cpu().numpy() == 0).all()
    assert np.array_equal(K.cpu().numpy(), wantK)
    assert np.array_equal(T.cpu().numpy(), wantT)
    for b in range(6):
        lb = oc.lower_bound(c["demand"][b].numpy())
        assert all(int(T[0, j, b]) >= lb * oc.W for j in range(len(k_targets)))
