"""Pins for the oracle's Algorithm 2 (no GPU).

What the paper and mathematics fix: schedule validity (Section 3), AA never
lowering F (Section 4.2, Step 2), progress in every iteration (Step 3), Eq. (9)
volumes, Eq. (10) selection in exact rationals, the closed form for uniform
demand on a crossbar, the reduction of the one-group case to a textbook linear
assignment, and exhaustive search on four ranks against the link-load bound.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch
from scipy.optimize import linear_sum_assignment

from workloads import (SchedParams, complete_catalog, crossbar_catalog, crossbar_topology,
                       moe_demand, node_template_catalog, tree_topology, uniform_demand)
from workloads.configs import build_config
from tests.bruteforce import optimal_time


def _oc(oracle_lib, cat):
    return oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())


def _random_demand(rng, N, u, hi, density):
    D = rng.integers(0, hi + 1, size=(N, N)) * (rng.random((N, N)) < density) * u
    np.fill_diagonal(D, 0)
    return D.astype(np.int64)


def _caps(oc, tau, u):
    return np.array([max(u, (tau * i[3]) // u * u) for i in oc.instances()], dtype=np.int64)


def _replay(oc, D, plan, tau, u):
    """Walk the plan step by step in numpy, asserting the per-step facts; returns the remainder."""
    N = oc.N
    inst = oc.instances()
    cap = _caps(oc, tau, u)
    rem = D.copy()
    for k in range(int(plan["n_steps"])):
        dst, pid, x = plan["lane_dst"][k], plan["lane_inst"][k], plan["lane_bytes"][k]
        assert oc.lanes_feasible(dst, pid) == 0                     # Eq. (1)
        act = dst >= 0
        assert act.any() and (x[act] > 0).all() and (x[~act] == 0).all()
        assert len(set(dst[act].tolist())) == act.sum()             # partial permutation
        for i in np.nonzero(act)[0]:
            assert x[i] == min(cap[pid[i]], rem[i, dst[i]])         # Eq. (9)
            assert inst[pid[i]][0] == i // oc.g and inst[pid[i]][1] == dst[i] // oc.g
            rem[i, dst[i]] -= x[i]
        assert (rem >= 0).all()
    return rem


TOPOS = {
    "node8": lambda: complete_catalog(tree_topology(1)),
    "node8_64_50": lambda: complete_catalog(tree_topology(1, pcie_bw=64, nic_bw=50)),
    "fig1_g3": lambda: complete_catalog(tree_topology(1, g=3, pcie_bw=64, nic_bw=50)),
    "g2_two_nodes": lambda: complete_catalog(tree_topology(2, g=2)),
    "two_nodes": lambda: complete_catalog(tree_topology(2)),
    "template_4_nodes": lambda: node_template_catalog(tree_topology(4)),
    "crossbar6": lambda: crossbar_catalog(crossbar_topology(6)),
}


@pytest.mark.parametrize("name", sorted(TOPOS))
@pytest.mark.parametrize("lam", [0, 8000])
def test_plans_are_valid_schedules(oracle_lib, name, lam):
    cat = TOPOS[name]()
    oc = _oc(oracle_lib, cat)
    rng = np.random.default_rng(sum(map(ord, name)) + lam)
    u = 256
    for trial in range(6):
        D = _random_demand(rng, oc.N, u, hi=[3, 40, 4000][trial % 3], density=[1.0, 0.5, 0.15][trial // 2])
        p = SchedParams(lambda_ns=lam, granule_bytes=u, n_start=0).resolved(oc.N)
        plan = oc.schedule(D, p, trace_cap=200000)
        assert plan["status"] == 0
        tau = int(plan["tau_ns"])
        rem = _replay(oc, D, plan, tau, u)
        assert not rem.any()                                        # sum_k X(E_k) = D
        assert oc.check_plan(D, plan, tau, u) == 0                  # the C checker agrees
        # offsets: exclusive prefix sums; totals are the row / column sums of D
        K = int(plan["n_steps"])
        assert (plan["send_off"][0] == 0).all() and (plan["recv_off"][0] == 0).all()
        assert (np.diff(plan["send_off"], axis=0) == plan["lane_bytes"]).all()
        assert (plan["send_off"][K] == D.sum(1)).all() and (plan["recv_off"][K] == D.sum(0)).all()
        assert (np.diff(plan["recv_off"], axis=0) >= 0).all()
        for k in range(K):
            arr = np.zeros(oc.N, np.int64)
            act = plan["lane_dst"][k] >= 0
            arr[plan["lane_dst"][k][act]] = plan["lane_bytes"][k][act]
            assert (plan["recv_off"][k + 1] - plan["recv_off"][k] == arr).all()
        assert (plan["chan_id"][K:] == -1).all() and (plan["lane_dst"][K:] == -1).all()
        # AA: F never decreases from sweep to sweep inside a run (Step 2)
        tr = plan["trace"]
        aa = tr[tr[:, 2] >= 0]
        same_run = (aa[1:, :3] == aa[:-1, :3]).all(axis=1)
        assert (aa[1:, 4][same_run] >= aa[:-1, 4][same_run]).all()
        # Eq. (10): the emitted family is the first maximiser of sum x / duration, in exact rationals
        ev = tr[tr[:, 2] == -1]
        W = oc.W
        for k in range(K):
            rows = ev[ev[:, 0] == k]
            util = [Fraction(int(r[3]), int(r[4])) if r[3] else Fraction(0) for r in rows]
            best = max(util)
            first = int(rows[[i for i, v in enumerate(util) if v == best][0], 1])
            assert first == plan["chan_id"][k]
            r = rows[rows[:, 1] == first][0]
            act = plan["lane_dst"][k] >= 0
            inst = oc.instances()
            tmax = max(Fraction(int(plan["lane_bytes"][k][i]), inst[plan["lane_inst"][k][i]][3])
                       for i in np.nonzero(act)[0])
            assert int(r[3]) == plan["lane_bytes"][k].sum()
            assert Fraction(int(r[4]), W) == lam + tmax
        # Eq. (2) against the link-load lower bound
        if lam == 0:
            assert oc.modeled_time(plan, 0) >= oc.lower_bound(D)


def test_shape_choice_is_first_argmax_of_eq6(oracle_lib):
    cat = complete_catalog(tree_topology(2))
    oc = _oc(oracle_lib, cat)
    rng = np.random.default_rng(5)
    fam_shape = np.repeat(np.arange(cat.n_shapes), np.diff(cat.bucket_ptr))
    for _ in range(5):
        D = _random_demand(rng, 16, 64, 50, 0.6)
        plan = oc.schedule(D, SchedParams(granule_bytes=64).resolved(16))
        rem = D.copy()
        for k in range(int(plan["n_steps"])):
            Dhat = rem.reshape(4, 4, 4, 4).sum(axis=(1, 3))                      # Eq. (5)
            scores = [sum(int(Dhat[a, d]) * c for a, d, c in s) for s in cat.shapes]  # Eq. (6)
            assert fam_shape[plan["chan_id"][k]] == int(np.argmax(scores))
            act = plan["lane_dst"][k] >= 0
            rem[np.nonzero(act)[0], plan["lane_dst"][k][act]] -= plan["lane_bytes"][k][act]


@pytest.mark.parametrize("n", [3, 5, 8])
def test_uniform_demand_on_a_crossbar_closed_form(oracle_lib, n):
    """One group: each iteration is an exact assignment, regular demand always has a perfect
    matching of full lanes, so K = (N-1)*ceil(c/cap) and T = K*(lambda + lane time)."""
    oc = _oc(oracle_lib, crossbar_catalog(crossbar_topology(n, bw=64)))
    lam, u, tau = 500, 64, 10          # cap = 640 bytes
    for c, m, lane in [(640 * 3, 3, 640), (640, 1, 640), (320, 1, 320), (64, 1, 64)]:
        plan = oc.schedule(uniform_demand(n, c).numpy(), SchedParams(lambda_ns=lam, granule_bytes=u).resolved(n),
                           tau_in=tau)
        assert plan["status"] == 0
        assert plan["n_steps"] == (n - 1) * m
        assert oc.modeled_time(plan, lam) == (n - 1) * m * (lam + Fraction(lane, 64))
        assert (plan["lane_bytes"][: plan["n_steps"]] == lane).all()


def test_uniform_demand_on_the_tree_first_step(oracle_lib):
    """Off-diagonal group pairs carry g*g*c, diagonal ones g*(g-1)*c, so Eq. (6) picks the shape of
    smallest trace; the first activation fills all N lanes with min(c, cap)."""
    cat = complete_catalog(tree_topology(1))
    oc = _oc(oracle_lib, cat)
    fam_shape = np.repeat(np.arange(cat.n_shapes), np.diff(cat.bucket_ptr))
    traces = [sum(c for a, d, c in s if a == d) for s in cat.shapes]
    for c, tau in [(1 << 20, 1000), (4096, 1000)]:
        plan = oc.schedule(uniform_demand(8, c).numpy(), SchedParams(granule_bytes=64).resolved(8), tau_in=tau)
        assert traces[fam_shape[plan["chan_id"][0]]] == min(traces)
        assert plan["lane_bytes"][0].sum() == 8 * min(c, 64 * tau)
        assert plan["n_steps"] >= 8      # 32 cross-switch pairs, at most 4 cross lanes per step


@pytest.mark.parametrize("n", [4, 6, 8])
def test_single_group_step_equals_linear_assignment_optimum(oracle_lib, n):
    """G = 1: the source half of the first sweep is one exact N x N assignment on
    min(D_rem, cap); its value must equal the Hungarian optimum at every step."""
    oc = _oc(oracle_lib, crossbar_catalog(crossbar_topology(n, bw=32)))
    rng = np.random.default_rng(n)
    u, tau = 16, 5                     # cap = 160
    for _ in range(4):
        D = _random_demand(rng, n, u, 40, 0.8)
        plan = oc.schedule(D, SchedParams(lambda_ns=0, granule_bytes=u).resolved(n), tau_in=tau)
        rem = D.copy()
        for k in range(int(plan["n_steps"])):
            credit = np.minimum(rem, 160)
            r, c = linear_sum_assignment(credit, maximize=True)
            assert plan["lane_bytes"][k].sum() == credit[r, c].sum()
            act = plan["lane_dst"][k] >= 0
            rem[np.nonzero(act)[0], plan["lane_dst"][k][act]] -= plan["lane_bytes"][k][act]
        assert not rem.any()


@pytest.mark.parametrize("topo", ["g2x2", "crossbar4", "g2x2_64_50"])
def test_greedy_against_exhaustive_search_on_four_ranks(oracle_lib, topo):
    """LB <= T_opt <= T_greedy with T_opt from enumeration of all channel sequences."""
    if topo == "crossbar4":
        cat = crossbar_catalog(crossbar_topology(4, bw=64))
    elif topo == "g2x2":
        cat = complete_catalog(tree_topology(1, g=2))
    else:
        cat = complete_catalog(tree_topology(1, g=2, pcie_bw=64, nic_bw=50))
    oc = _oc(oracle_lib, cat)
    rng = np.random.default_rng(11)
    u, tau = 64, 2                    # cap = 128 at 64 B/ns, 64 at 50 B/ns
    cap = _caps(oc, tau, u).tolist()
    ratios = []
    for lam in (0, 3):
        for _ in range(4):
            D = _random_demand(rng, 4, u, 3, 0.7)
            if not D.any():
                continue
            plan = oc.schedule(D, SchedParams(lambda_ns=lam, granule_bytes=u, n_start=0).resolved(4), tau_in=tau)
            assert plan["status"] == 0 and oc.check_plan(D, plan, tau, u) == 0
            t_greedy = oc.modeled_time(plan, lam)
            t_opt = optimal_time(4, oc.g, oc.instances(), D.tolist(), cap, lam)
            assert t_opt <= t_greedy
            if lam == 0:
                assert oc.lower_bound(D) <= t_opt
            ratios.append(float(t_opt / t_greedy))
    assert min(ratios) > 0.5          # context: the paper reports >= 91.92 % of a MILP optimum


def test_quantum_rule_worked_example(oracle_lib):
    """tau = ceil(est / K_target): one node, only rank 0 -> rank 4 carries 64*1000 bytes; every path
    runs at 64 B/ns, the pair has two disjoint paths (PXB, NIC) so nothing is forced: est = 1000 ns."""
    oc = _oc(oracle_lib, complete_catalog(tree_topology(1)))
    D = np.zeros((8, 8), np.int64)
    D[0, 4] = 64000
    plan = oc.schedule(D, SchedParams(k_target=10, granule_bytes=64).resolved(8))
    assert plan["tau_ns"] == 100 and plan["n_steps"] == 10
    assert (plan["lane_bytes"][:10, 0] == 6400).all()
    # two nodes: rank 0 -> rank 8 can only use NIC(0 -> 2): forced through its transmit side
    oc2 = _oc(oracle_lib, complete_catalog(tree_topology(2, nic_bw=50)))
    D = np.zeros((16, 16), np.int64)
    D[0, 8] = D[1, 9] = 50 * 640
    plan = oc2.schedule(D, SchedParams(k_target=4, granule_bytes=1).resolved(16))
    assert plan["tau_ns"] == (2 * 640) // 4      # both flows share NICtx(0): est = 1280 ns
    assert plan["n_steps"] == 4                  # one NIC lane of 50*320 bytes per step = K_target rounds


def test_status_codes(oracle_lib):
    oracle = oracle_lib
    cat = complete_catalog(tree_topology(1))
    oc = _oc(oracle, cat)
    p = SchedParams(granule_bytes=64).resolved(8)
    D = uniform_demand(8, 640).numpy()
    bad = D.copy(); bad[2, 2] = 64
    assert oc.schedule(bad, p)["status"] == oracle.ST_DIAG
    bad = D.copy(); bad[1, 2] = -64
    assert oc.schedule(bad, p)["status"] == oracle.ST_NEGATIVE
    bad = D.copy(); bad[1, 2] = 65
    assert oc.schedule(bad, p)["status"] == oracle.ST_GRANULE
    bad = D.copy(); bad[1, 2] = 1 << 40
    out = oc.schedule(bad, p)
    assert out["status"] == oracle.ST_OVERFLOW and out["n_steps"] == 0 and not out["lane_bytes"].any()
    assert oc.schedule(D, p, tau_in=(1 << 40) + 1)["status"] == oracle.ST_BAD_TAU
    # step limit: the steps written are valid and the remainder is what is left unserved
    short = SchedParams(granule_bytes=64, k_max=3).resolved(8)
    out = oc.schedule(D, short)
    assert out["status"] == oracle.ST_STEP_LIMIT and out["n_steps"] == 3
    rem = _replay(oc, D, out, int(out["tau_ns"]), 64)
    assert rem.sum() == D.sum() - out["lane_bytes"].sum() and rem.any()
    # a catalog without any cross-switch shape cannot serve cross-switch demand
    from workloads.topology import Catalog
    only_pix = Catalog(cat.topology, [cat.shapes[-1]], [cat.buckets[-1]])
    oc2 = _oc(oracle, only_pix)
    assert not oc2.covers()
    out = oc2.schedule(D, p)
    assert out["status"] == oracle.ST_UNCOVERED
    assert _replay(oc2, D, out, int(out["tau_ns"]), 64)[:4, 4:].sum() == D[:4, 4:].sum()
    # zero demand: nothing to do
    out = oc.schedule(np.zeros((8, 8), np.int64), p)
    assert out["status"] == 0 and out["n_steps"] == 0 and out["tau_ns"] == 1


def test_round_counts_on_the_configs(oracle_lib):
    """Section 5 expects roughly K_target rounds; the scaled-down configs stay within a small factor."""
    for idx, scale in [(1, 0.25), (2, 0.125)]:
        c = build_config(idx, batch=3, token_scale=scale)
        oc = _oc(oracle_lib, c["catalog"])
        out = oc.schedule_batch(c["demand"].numpy(), c["params"], threads=2)
        assert (out["status"] == 0).all()
        assert (out["n_steps"] >= oc.N).all() and (out["n_steps"] <= 5 * oc.N).all()
        single = oc.schedule_batch(c["demand"].numpy(), c["params"], threads=1)
        for k in ("n_steps", "chan_id", "lane_dst", "lane_inst", "lane_bytes", "send_off", "recv_off"):
            assert (out[k] == single[k]).all()


def _aa_cases():
    """(catalog, demand, params, tau) where the starts of MultiStartAA really differ: two or more groups and
    sparse demand in a handful of small values, so that runs end at different sweeps, with different F and,
    among equal F, with different bindings."""
    rng = np.random.default_rng(77)
    u = 64
    for name, i_aa in [("node8", 1), ("node8", 5), ("two_nodes", 3), ("two_nodes", 5), ("g2_two_nodes", 5),
                       ("node8_64_50", 2), ("template_4_nodes", 4)]:
        cat = TOPOS[name]()
        N = cat.topology.N
        for density, hi in [(0.25, 2), (0.4, 5), (0.15, 9)]:
            D = _random_demand(rng, N, u, hi, density)
            if D.any():
                yield cat, D, SchedParams(lambda_ns=100, granule_bytes=u, n_start=4, i_aa=i_aa).resolved(N), 2


def test_multistart_aa_stop_rule_and_best_start(oracle_lib):
    """Section 4.2, Step 2: a run of the Alternating Algorithm ends after I_AA sweeps or after the first
    complete sweep that does not raise F_B, and MultiStartAA returns its highest-scoring run (lowest start
    among equals, this build's convention).  Checked from the trace: every run's sweep records end exactly
    where the rule says; the binding a run ends with scores the F of its last sweep on the residual demand
    (recomputed here in numpy); each candidate's volume is the largest such F; and the emitted activation is
    the binding of the lowest start that reaches it."""
    seen = dict(early=0, limit=0, later_start=0, tie_other_binding=0, runs=0)
    for cat, D, p, tau in _aa_cases():
        oc = _oc(oracle_lib, cat)
        N, u = oc.N, p.granule_bytes
        plan = oc.schedule(D, p, tau_in=tau, trace_cap=2_000_000)
        assert plan["status"] == 0 and len(plan["trace"]) < 2_000_000
        cap = _caps(oc, tau, u)
        fam = oc.families()
        tr = plan["trace"]
        rem = D.copy()
        for k in range(int(plan["n_steps"])):
            rows = tr[tr[:, 0] == k]
            cands = rows[rows[:, 2] == -1]
            assert len(cands) >= 1
            for f, vol in zip(cands[:, 1].tolist(), cands[:, 3].tolist()):
                fr = rows[rows[:, 1] == f]
                last_f, binds = [], []
                for t in range(p.n_start):
                    F = fr[fr[:, 2] == t]
                    assert F[:, 3].tolist() == list(range(len(F))) and 1 <= len(F) <= p.i_aa
                    Fv = [-1] + F[:, 4].tolist()
                    m = len(F)
                    assert all(Fv[s + 1] > Fv[s] for s in range(m - 1))       # it went on only after an improvement
                    assert m == p.i_aa or Fv[m] <= Fv[m - 1]                  # it ended at the limit or at no gain
                    seen["early" if m < p.i_aa else "limit"] += 1
                    b = fr[fr[:, 2] == -2 - t]
                    assert b[:, 3].tolist() == list(range(N))
                    src, dst = b[:, 4] // 65536, b[:, 4] % 65536
                    assert sorted(src.tolist()) == list(range(N)) and sorted(dst.tolist()) == list(range(N))
                    credit = np.minimum(rem[src, dst], cap[fam[f]])           # Eq. (7) x tau, Eq. (8)
                    assert credit.sum() == Fv[m]                              # the binding as it stands scores the last F
                    last_f.append(Fv[m]); binds.append((src, dst, credit))
                    seen["runs"] += 1
                assert vol == max(last_f)                                     # returns the highest-scoring run
                if f == plan["chan_id"][k]:
                    t_star = last_f.index(max(last_f))
                    seen["later_start"] += t_star > 0
                    src, dst, x = binds[t_star]
                    exp_dst = np.full(N, -1, np.int64); exp_x = np.zeros(N, np.int64); exp_i = np.full(N, 0xFFFF, np.int64)
                    busy = x > 0
                    exp_dst[src[busy]] = dst[busy]; exp_x[src[busy]] = x[busy]; exp_i[src[busy]] = fam[f][busy]
                    assert (plan["lane_dst"][k] == exp_dst).all() and (plan["lane_bytes"][k] == exp_x).all()
                    assert (plan["lane_inst"][k] == exp_i).all()
                    for t in range(t_star + 1, p.n_start):                    # an equal run that would emit something else
                        if last_f[t] == last_f[t_star]:
                            s2, d2, x2 = binds[t]
                            o_dst = np.full(N, -1, np.int64); o_dst[s2[x2 > 0]] = d2[x2 > 0]
                            seen["tie_other_binding"] += int((o_dst != exp_dst).any())
            act = plan["lane_dst"][k] >= 0
            rem[np.nonzero(act)[0], plan["lane_dst"][k][act]] -= plan["lane_bytes"][k][act]
        assert not rem.any()
    # the cases exercise every branch of the rule
    assert seen["early"] > 100 and seen["limit"] > 100 and seen["later_start"] > 10 and seen["tie_other_binding"] > 10


@pytest.mark.parametrize("n", [4, 7])
def test_sweep_of_lambda_and_k_target_against_the_crossbar_closed_form(oracle_lib, n):
    """Eq. (2) over a grid of (lambda, K_target) (Section 5: K_target sets the quantum).  Uniform demand c on a crossbar:
    est = (N-1) c / bw, tau = ceil(est / K_target), cap = max(u, floor(tau bw / u) u), then (N-1) ceil(c / cap) rounds of
    full lanes, the last round of each pair carrying the remainder -- a closed form for every grid point."""
    bw, u, c = 64, 64, 64 * 1000
    oc = _oc(oracle_lib, crossbar_catalog(crossbar_topology(n, bw=bw)))
    D = uniform_demand(n, c).numpy()[None]
    lambdas, k_targets = [0, 500, 8000], [1, 3, n, 2 * n, 5 * n, 1000 * n]
    T, K = oc.sweep_plan_time(D, SchedParams(granule_bytes=u, k_max=1200 * n).resolved(n), lambdas, k_targets)
    for i, lam in enumerate(lambdas):
        for j, kt in enumerate(k_targets):
            est = -(-(n - 1) * c // bw)
            tau = max(1, -(-est // kt))
            cap = max(u, tau * bw // u * u)
            full, rest = divmod(c, cap)
            rounds = full + (1 if rest else 0)
            want = (n - 1) * (full * (lam + Fraction(cap, bw)) + (1 if rest else 0) * (lam + Fraction(rest, bw)))
            assert K[i, j, 0] == (n - 1) * rounds
            assert Fraction(int(T[i, j, 0]), oc.W) == want
    # more rounds cost more overhead and never less transfer time: T grows with lambda at every K_target
    assert (np.diff(T[:, :, 0], axis=0) >= 0).all()
