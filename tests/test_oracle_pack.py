"""Pins for the oracle's pack (no GPU): a slow per-row search in pure Python on tiny inputs, and
the properties that hold at any size."""
import numpy as np
import pytest

from workloads import SchedParams, complete_catalog, tree_topology
from workloads.demand import demand_from_routing, moe_routing

import torch


def _case(oracle_lib, T, topk, E, hidden, seed, rank, drop=False):
    cat = complete_catalog(tree_topology(1))
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    N = oc.N
    row_bytes = hidden * 2
    idx = moe_routing(T * N, E, topk, 1.2, seed)
    src = torch.repeat_interleave(torch.arange(N), T)
    D = demand_from_routing(idx, src, N, E, row_bytes).numpy()
    mine = idx[rank * T:(rank + 1) * T].numpy().copy()
    if drop:                                   # dropped copies (negative ids) are not part of the demand
        mine[::3, 0] = -1
        D[rank] = 0
        for t in range(T):
            for s in range(topk):
                if mine[t, s] >= 0 and mine[t, s] // (E // N) != rank:
                    D[rank, mine[t, s] // (E // N)] += row_bytes
    plan = oc.schedule(D, SchedParams(granule_bytes=row_bytes).resolved(N))
    assert plan["status"] == 0
    rows = np.random.default_rng(seed).integers(0, 65536, size=(T, hidden), dtype=np.uint16)
    return oc, plan, mine, rows, D, row_bytes, E // N


@pytest.mark.parametrize("rank,drop", [(0, False), (5, False), (3, True)])
def test_pack_matches_per_row_search(oracle_lib, rank, drop):
    oc, plan, idx, rows, D, row_bytes, epr = _case(oracle_lib, T=37, topk=4, E=32, hidden=24, seed=7,
                                                   rank=rank, drop=drop)
    R = int(D[rank].sum() // row_bytes)
    staged, src_map, st = oc.pack(plan, rank, idx, epr, rows, R)
    assert st == 0
    T, topk = idx.shape
    # slow definition: staged row r belongs to the step whose [send_off[k], send_off[k+1]) holds it;
    # it is the p-th row of that step, i.e. the (rows sent to that destination in earlier steps + p)-th
    # copy, in ascending (token, slot), among the copies routed to the step's destination.
    for r in range(R):
        k = max(kk for kk in range(int(plan["n_steps"])) if plan["send_off"][kk][rank] <= r * row_bytes
                and plan["lane_dst"][kk][rank] >= 0 and plan["send_off"][kk][rank] < plan["send_off"][kk + 1][rank])
        j = int(plan["lane_dst"][k][rank])
        earlier = sum(int(plan["lane_bytes"][kk][rank]) // row_bytes for kk in range(k)
                      if plan["lane_dst"][kk][rank] == j)
        p = r - int(plan["send_off"][k][rank]) // row_bytes
        copies = [(t, s) for t in range(T) for s in range(topk)
                  if idx[t, s] >= 0 and idx[t, s] // epr == j]
        t, s = copies[earlier + p]
        assert src_map[r] == t * topk + s
        assert (staged[r].view(np.uint16) == rows[t]).all()


def test_pack_properties(oracle_lib):
    oc, plan, idx, rows, D, row_bytes, epr = _case(oracle_lib, T=400, topk=8, E=64, hidden=16, seed=3, rank=2)
    rank = 2
    R = int(D[rank].sum() // row_bytes)
    staged, src_map, st = oc.pack(plan, rank, idx, epr, rows, R + 5)
    assert st == 0
    topk = idx.shape[1]
    remote = sorted(e for e in range(idx.size) if idx.flat[e] // epr != rank)
    assert sorted(src_map[:R].tolist()) == remote            # a permutation of the remote copies
    assert (src_map[R:] == -1).all() and not staged[R:].any()  # nothing beyond the plan's bytes
    for k in range(int(plan["n_steps"])):
        lo, hi = (int(plan["send_off"][k + x][rank]) // row_bytes for x in (0, 1))
        chunk = src_map[lo:hi]
        assert (np.diff(chunk) > 0).all()                     # ascending (token, slot) inside a step
        if hi > lo:
            assert (idx.flat[chunk] // epr == plan["lane_dst"][k][rank]).all()
    assert (staged[:R].view(np.uint16) == rows[src_map[:R] // topk]).all()


def test_pack_error_statuses(oracle_lib):
    oracle = oracle_lib
    oc, plan, idx, rows, D, row_bytes, epr = _case(oracle_lib, T=50, topk=4, E=32, hidden=8, seed=9, rank=1)
    R = int(D[1].sum() // row_bytes)
    assert oc.pack(plan, 1, idx, epr, rows, R - 1)[2] == oracle.ST_PACK_CAPACITY
    other = idx.copy()
    other[0, 0] = (other[0, 0] + epr) % 32                    # routing no longer matches the plan
    assert oc.pack(plan, 1, other, epr, rows, R)[2] & oracle.ST_PACK_MISMATCH
    assert oc.pack(plan, 1, idx, epr, rows, R)[2] == 0


def test_demand_from_routing_equals_a_library_histogram(oracle_lib):
    """The demand rows are a 2-D histogram of (source, destination rank) pairs: numpy's bincount is the pin."""
    rng = np.random.default_rng(4)
    n_src, T, topk, epr, N, rb = 5, 300, 6, 4, 8, 1024
    idx = rng.integers(-1, N * epr, size=(n_src, T, topk)).astype(np.int32)      # -1 = dropped copy
    rows, bad = oracle_lib.demand_from_routing(idx, epr, N, rb, src0=2)
    assert bad == 0
    want = np.zeros((n_src, N), np.int64)
    for s in range(n_src):
        d = idx[s][idx[s] >= 0] // epr
        want[s] = np.bincount(d, minlength=N) * rb
        want[s, 2 + s] = 0
    assert np.array_equal(rows, want)
    idx[0, 0, 0] = N * epr                                                         # a rank that does not exist
    assert oracle_lib.demand_from_routing(idx, epr, N, rb, src0=2)[1] == 1


def test_pack_exchange_unpack_round_trip(oracle_lib):
    """End to end on one node: every rank packs, the chunks travel as the plan says, rank j unpacks.  The result
    must be what the routing says directly: for each local expert, the rows of all (source, token, slot) copies
    routed to it, in (source, token, slot) order -- a definition that involves neither plan nor offsets."""
    from tests.exchange import deliver
    from workloads import complete_catalog, tree_topology, SchedParams
    from workloads.demand import demand_from_routing, moe_routing
    import torch
    cat = complete_catalog(tree_topology(1))
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    N, T, topk, E, hidden = 8, 60, 4, 32, 8
    epr, rb = E // N, hidden * 2
    idx = moe_routing(N * T, E, topk, 1.0, seed=77).reshape(N, T, topk).numpy()
    D = demand_from_routing(torch.from_numpy(idx.reshape(N * T, topk)), torch.repeat_interleave(torch.arange(N), T), N, E, rb).numpy()
    plan = oc.schedule(D, SchedParams(granule_bytes=rb).resolved(N))
    assert plan["status"] == 0
    rng = np.random.default_rng(1)
    rows = rng.integers(0, 65536, size=(N, T, hidden), dtype=np.uint16)
    staged, meta = {}, {}
    for i in range(N):
        R = int(D[i].sum() // rb)
        s, m, st = oc.pack(plan, i, idx[i], epr, rows[i], R)
        assert st == 0
        staged[i], meta[i] = s, idx[i].reshape(-1)[m] % epr          # local expert id travels with each row
    # the oracle's exchange (sender side, rank by rank) delivers the payload; the metadata travels by the numpy helper.
    # Both must give the receiver the same rows, and every rank must receive exactly its demand column.
    bufs, arrived, xst = oc.exchange(plan, staged)
    assert xst == 0 and arrived.tolist() == D.sum(0).tolist()
    for j in (0, 5):
        recv, recv_expert = deliver(plan, j, staged, rb, meta)
        assert np.array_equal(bufs[j].reshape(-1, rb), recv)
        recv = bufs[j].reshape(-1, rb)
        out, expert_off, out_src, out_map, st = oc.unpack(plan, j, recv, recv_expert, epr)
        assert st == 0
        want_rows, want_src, want_off = [], [], [0]
        for e in range(epr):
            for i in range(N):
                if i == j:
                    continue
                for t in range(T):
                    for s in range(topk):
                        if idx[i, t, s] == j * epr + e:
                            want_rows.append(rows[i, t]); want_src.append(i)
            want_off.append(len(want_rows))
        assert expert_off.tolist() == want_off
        assert out_src.tolist() == want_src
        assert np.array_equal(out.view(np.uint16), np.array(want_rows, dtype=np.uint16))
        assert sorted(out_map.tolist()) == list(range(len(want_rows)))


def test_dispatch_and_return_round_trip(oracle_lib):
    """Dispatch and return on one node, every stage by the oracle: pack -> exchange -> unpack (expert-major) -> each
    expert tags its rows -> return pack (plan of D^T, destination = the row's source) -> exchange -> unpack into the
    token layout.  Every remote copy (t, slot) of every rank must come back as its own token row tagged by the
    expert it was routed to: a statement about routing only."""
    from tests.exchange import deliver
    from workloads import complete_catalog, tree_topology, SchedParams
    from workloads.demand import demand_from_routing, moe_routing
    import torch
    cat = complete_catalog(tree_topology(1))
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    N, T, topk, E, hidden = 8, 40, 3, 24, 8
    epr, rb = E // N, hidden * 2
    idx = moe_routing(N * T, E, topk, 0.8, seed=91).reshape(N, T, topk).numpy().astype(np.int32)
    src_of = torch.repeat_interleave(torch.arange(N), T)
    D = demand_from_routing(torch.from_numpy(idx.reshape(N * T, topk)), src_of, N, E, rb).numpy()
    w = SchedParams(granule_bytes=rb).resolved(N)
    plan = oc.schedule(D, w)
    back = oc.schedule(np.ascontiguousarray(D.T), w)                       # the return call has its own plan
    assert plan["status"] == 0 and back["status"] == 0
    rows = np.random.default_rng(4).integers(0, 65536, size=(N, T, hidden), dtype=np.uint16)
    staged, meta = {}, {}
    for i in range(N):
        s, m, st = oc.pack(plan, i, idx[i], epr, rows[i], int(D[i].sum() // rb))
        assert st == 0
        staged[i], meta[i] = s, idx[i].reshape(-1)[m] % epr
    ret_staged = {}
    for j in range(N):
        recv, recv_expert = deliver(plan, j, staged, rb, meta)
        out, expert_off, out_src, out_map, st = oc.unpack(plan, j, recv, recv_expert, epr)
        assert st == 0
        y = out.view(np.uint16).copy()
        for e in range(epr):                                               # expert e of rank j tags what it processed
            y[expert_off[e]:expert_off[e + 1]] ^= np.uint16(j * epr + e + 1)
        s, m, st = oc.pack(back, j, out_src.reshape(-1, 1), 1, y, int(D[:, j].sum() // rb))
        assert st == 0
        ret_staged[j] = s
    for i in range(N):
        ret_recv, _ = deliver(back, i, ret_staged, rb)
        out = np.zeros((T * topk, rb), np.uint8)
        out, out_map, st = oc.unpack_tokens(back, i, idx[i], epr, ret_recv, out)
        assert st == 0
        got = out.view(np.uint16).reshape(T, topk, hidden)
        for t in range(T):
            for s in range(topk):
                e = idx[i, t, s]
                if e < 0 or e // epr == i:
                    assert out_map[t * topk + s] == -1 and not got[t, s].any()
                else:
                    assert np.array_equal(got[t, s], rows[i, t] ^ np.uint16(e + 1)), (i, t, s)
