"""GPU parity: vp_unpack (through the C ABI) against the CPU oracle, byte for byte, and the whole
pack -> exchange -> unpack chain against the routing definition of the expert-major layout."""
import os

import numpy as np
import pytest
import torch

from workloads import SchedParams as WParams, complete_catalog, tree_topology
from workloads.configs import build_pack_case

pytestmark = pytest.mark.gpu
GUARD = 64


@pytest.fixture(scope="module")
def vp():
    import paper_2609_34340_b200 as vp
    assert torch.cuda.is_available(), "these tests need a GPU"
    assert os.path.exists(vp.library_path()), "libvariopath.so has not been built"
    return vp


def _params(vp, w):
    return vp.SchedParams(lambda_ns=w.lambda_ns, granule_bytes=w.granule_bytes, k_target=w.k_target,
                          n_start=w.n_start, i_aa=w.i_aa, k_max=w.k_max)


def _plans(vp, oracle_lib, cat, demand, w):
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    plan = vp.schedule_batch(dc, _params(vp, w), demand.cuda())
    want = oc.schedule_batch(demand.numpy(), w)
    one = {k: (v[0] if isinstance(v, np.ndarray) else v) for k, v in want.items()}
    return oc, plan, one


def _receive_case(case, rank, epr, seed, dtype=torch.int16, extra_rows=0):
    """A synthetic receive buffer for ``rank``: as many random rows as the demand column says, each with a
    local expert id drawn with a skew (some experts get most rows, some none)."""
    rb = case["row_bytes"]
    R = int(case["demand"][0, :, rank].sum().item() // rb)
    rng = np.random.default_rng(seed)
    width = rb // (2 if dtype == torch.int16 else 1)
    recv = torch.from_numpy(rng.integers(0, 256, size=(R + extra_rows, rb), dtype=np.uint8)).view(dtype).reshape(R + extra_rows, width)
    p = rng.dirichlet(np.full(epr, 0.3))
    expert = rng.choice(epr, size=R + extra_rows, p=p).astype(np.int32)
    return R, recv, expert


def _run(vp, oc, plan, one, rank, recv, expert, epr):
    cap = recv.shape[0]
    out = torch.zeros((cap + GUARD, recv.shape[1]), dtype=recv.dtype, device="cuda")
    out[cap:] = 0x55 if recv.dtype == torch.uint8 else 0x5555
    out_src = torch.full((cap + GUARD,), -7, dtype=torch.int32, device="cuda")
    out_map = torch.full((cap + GUARD,), -7, dtype=torch.int32, device="cuda")
    off, st = vp.unpack(plan, 0, rank, recv.cuda().contiguous(), torch.from_numpy(expert).cuda(), epr, out[:cap],
                        out_src=out_src, out_map=out_map)
    torch.cuda.synchronize()
    want = oc.unpack(one, rank, recv.numpy(), expert, epr)
    return (out.cpu().numpy(), off.cpu().numpy(), out_src.cpu().numpy(), out_map.cpu().numpy(), int(st.item())), want, cap


def _assert_unpack(got, want, cap):
    out, off, src, mp, st = got
    w_out, w_off, w_src, w_map, w_st = want
    assert st == w_st
    assert off.tolist() == w_off.tolist()
    n = int(w_off[-1])
    assert np.array_equal(src[:n], w_src[:n]) and np.array_equal(mp[:n], w_map[:n])
    assert np.array_equal(out[:n].view(np.uint8).reshape(n, -1), w_out[:n].reshape(n, -1)) if n else True
    assert (src[n:] == -7).all() and (mp[n:] == -7).all()               # nothing written past the received rows
    assert (out[cap:].view(np.uint8) == 0x55).all()


@pytest.mark.parametrize("tokens,hidden,rank,extra", [(300, 1024, 0, 0), (300, 1024, 9, 100), (1000, 7168, 3, 0), (257, 8200, 15, 3)])
def test_unpack_matches_oracle_bulk_path(vp, oracle_lib, tokens, hidden, rank, extra):
    case = build_pack_case(device="cpu", tokens=tokens, hidden=hidden, rank=rank, seed=21)
    oc, plan, one = _plans(vp, oracle_lib, case["catalog"], case["demand"], case["params"])
    R, recv, expert = _receive_case(case, rank, case["experts_per_rank"], seed=rank, extra_rows=extra)
    got, want, cap = _run(vp, oc, plan, one, rank, recv, expert, case["experts_per_rank"])
    assert got[4] == 0 and int(got[1][-1]) == R
    _assert_unpack(got, want, cap)


@pytest.mark.parametrize("hidden,dtype", [(64, torch.int16), (1000, torch.int16), (333, torch.uint8), (6, torch.int16)])
def test_unpack_matches_oracle_plain_path(vp, oracle_lib, hidden, dtype):
    case = build_pack_case(device="cpu", tokens=500, hidden=hidden, rank=2, seed=22)
    if dtype == torch.uint8:
        case["demand"] = case["demand"] // case["row_bytes"] * hidden
        case["row_bytes"] = hidden
        case["params"] = WParams(granule_bytes=hidden).resolved(16)
    oc, plan, one = _plans(vp, oracle_lib, case["catalog"], case["demand"], case["params"])
    R, recv, expert = _receive_case(case, 2, case["experts_per_rank"], seed=5, dtype=dtype)
    got, want, cap = _run(vp, oc, plan, one, 2, recv, expert, case["experts_per_rank"])
    assert got[4] == 0 and int(got[1][-1]) == R
    _assert_unpack(got, want, cap)


def test_unpack_error_statuses(vp, oracle_lib):
    case = build_pack_case(device="cpu", tokens=200, hidden=1024, rank=4, seed=23)
    epr = case["experts_per_rank"]
    oc, plan, one = _plans(vp, oracle_lib, case["catalog"], case["demand"], case["params"])
    R, recv, expert = _receive_case(case, 4, epr, seed=1)
    # an expert id out of range: that row is left out, the rest is placed
    bad = expert.copy()
    bad[R // 2] = epr
    bad[3] = -1
    got, want, cap = _run(vp, oc, plan, one, 4, recv, bad, epr)
    assert got[4] == vp.ST_PACK_MISMATCH and int(got[1][-1]) == R - 2
    _assert_unpack(got, want, cap)
    # a receive buffer that is too small: nothing is copied
    got, want, cap = _run(vp, oc, plan, one, 4, recv[:R - 1], expert[:R - 1], epr)
    assert got[4] == vp.ST_PACK_CAPACITY and got[1].tolist() == [0] * (epr + 1)
    _assert_unpack(got, want, cap)
    assert (got[0][:cap] == 0).all()
    # a rank that receives nothing
    empty = case["demand"].clone()
    empty[0, :, 4] = 0
    oc, plan, one = _plans(vp, oracle_lib, case["catalog"], empty, case["params"])
    got, want, cap = _run(vp, oc, plan, one, 4, recv[:10], expert[:10], epr)
    assert got[4] == 0 and got[1].tolist() == [0] * (epr + 1)
    _assert_unpack(got, want, cap)
    # sizes outside the limits are refused before any launch
    with pytest.raises(vp.VpError) as e:
        vp.unpack(plan, 0, 4, recv[:10].cuda(), torch.zeros(10, dtype=torch.int32, device="cuda"), 100,
                  torch.zeros_like(recv[:10]).cuda())
    assert e.value.code == vp.E_UNSUPPORTED


def test_pack_exchange_unpack_round_trip(vp, oracle_lib):
    """Every rank of one node packs on the GPU, the chunks travel as the plan says (numpy), rank j unpacks on the
    GPU; the result is what the routing says directly: per local expert the rows of all (source, token, slot)
    copies routed to it, in that order."""
    from tests.exchange import deliver
    from workloads.demand import demand_from_routing, moe_routing
    cat = complete_catalog(tree_topology(1))
    N, T, topk, E, hidden = 8, 700, 4, 32, 1024
    epr, rb = E // N, hidden * 2
    idx = moe_routing(N * T, E, topk, 1.0, seed=78).reshape(N, T, topk)
    D = demand_from_routing(idx.reshape(N * T, topk), torch.repeat_interleave(torch.arange(N), T), N, E, rb)
    w = WParams(granule_bytes=rb).resolved(N)
    oc, plan, one = _plans(vp, oracle_lib, cat, D.unsqueeze(0), w)
    rows = torch.randint(-32768, 32768, (N, T, hidden), dtype=torch.int16, generator=torch.Generator().manual_seed(3))
    staged, meta = {}, {}
    for i in range(N):
        R = int(D[i].sum().item() // rb)
        s = torch.zeros((R, hidden), dtype=torch.int16, device="cuda")
        m = torch.full((R,), -1, dtype=torch.int32, device="cuda")
        st = vp.pack(plan, 0, i, idx[i].to(torch.int32).cuda().contiguous(), epr, rows[i].cuda().contiguous(), s, m)
        assert int(st.item()) == 0
        staged[i] = s.cpu().numpy().view(np.uint8).reshape(R, rb)
        meta[i] = idx[i].reshape(-1).numpy()[m.cpu().numpy()] % epr
    idx_np, rows_np = idx.numpy(), rows.numpy()
    for j in (0, 6):
        recv, recv_expert = deliver(one, j, staged, rb, meta)
        got, want, cap = _run(vp, oc, plan, one, j, torch.from_numpy(recv).view(torch.int16), recv_expert.astype(np.int32), epr)
        assert got[4] == 0
        _assert_unpack(got, want, cap)
        want_rows, want_src, want_off = [], [], [0]
        for e in range(epr):
            for i in range(N):
                if i == j:
                    continue
                t_sel, _ = np.nonzero(idx_np[i] == j * epr + e)
                want_rows.append(rows_np[i, t_sel]); want_src += [i] * len(t_sel)
            want_off.append(len(want_src))
        assert got[1].tolist() == want_off
        assert got[2][:len(want_src)].tolist() == want_src
        assert np.array_equal(got[0][:len(want_src)], np.concatenate(want_rows))


def test_unpack_config5_size(vp, oracle_lib):
    """Receive side at the size of the packed-buffer configuration (16,384 tokens x top-8 per rank, 14,336-byte
    rows): the full output is compared with the oracle."""
    case = build_pack_case(device="cpu", rank=8)
    epr = case["experts_per_rank"]
    oc, plan, one = _plans(vp, oracle_lib, case["catalog"], case["demand"], case["params"])
    R, recv, expert = _receive_case(case, 8, epr, seed=8)
    got, want, cap = _run(vp, oc, plan, one, 8, recv, expert, epr)
    assert got[4] == 0 and int(got[1][-1]) == R
    _assert_unpack(got, want, cap)


# ---- return direction ---------------------------------------------------------------------------------

def _return_case(vp, oracle_lib, case, rank, seed, extra_rows=0):
    """The return call of a packed-buffer case: plan of D^T, rank's routing, a synthetic return receive buffer."""
    Dt = case["demand"].transpose(1, 2).contiguous()
    oc, plan, one = _plans(vp, oracle_lib, case["catalog"], Dt, case["params"])
    rb = case["row_bytes"]
    R = int(Dt[0, :, rank].sum().item() // rb)             # what rank receives back = what it sent
    rng = np.random.default_rng(seed)
    recv = torch.from_numpy(rng.integers(0, 256, size=(R + extra_rows, rb), dtype=np.uint8)).view(torch.int16)
    return oc, plan, one, R, recv


def _run_tokens(vp, oc, plan, one, rank, idx, epr, recv):
    T, topk = idx.shape
    out = torch.full((T * topk + GUARD, recv.shape[1]), 0x1111, dtype=recv.dtype, device="cuda")
    out_map = torch.full((T * topk + GUARD,), -7, dtype=torch.int32, device="cuda")
    st = vp.unpack_tokens(plan, 0, rank, idx.cuda().contiguous(), epr, recv.cuda().contiguous(), out[:T * topk], out_map)
    torch.cuda.synchronize()
    base = np.full((T * topk, recv.shape[1]), 0x1111, dtype=np.int16).view(np.uint8)
    w_out, w_map, w_st = oc.unpack_tokens(one, rank, idx.numpy(), epr, recv.numpy(), base)
    got_out, got_map = out.cpu().numpy(), out_map.cpu().numpy()
    assert int(st.item()) == w_st
    assert np.array_equal(got_map[:T * topk], w_map)
    assert np.array_equal(got_out[:T * topk].view(np.uint8), w_out)
    assert (got_map[T * topk:] == -7).all() and (got_out[T * topk:] == 0x1111).all()
    return w_st, w_map


@pytest.mark.parametrize("tokens,hidden,rank,extra", [(300, 1024, 0, 0), (1000, 7168, 3, 5), (257, 8200, 15, 0), (500, 64, 2, 0)])
def test_unpack_tokens_matches_oracle(vp, oracle_lib, tokens, hidden, rank, extra):
    case = build_pack_case(device="cpu", tokens=tokens, hidden=hidden, rank=rank, seed=31)
    oc, plan, one, R, recv = _return_case(vp, oracle_lib, case, rank, seed=rank, extra_rows=extra)
    st, w_map = _run_tokens(vp, oc, plan, one, rank, case["expert_idx"], case["experts_per_rank"], recv)
    assert st == 0 and int((w_map >= 0).sum()) == R


def test_unpack_tokens_statuses(vp, oracle_lib):
    case = build_pack_case(device="cpu", tokens=200, hidden=1024, rank=4, seed=33)
    epr = case["experts_per_rank"]
    oc, plan, one, R, recv = _return_case(vp, oracle_lib, case, 4, seed=2)
    idx = case["expert_idx"].clone()
    idx[7, 2] = -1                                           # the routing lost a copy the plan still delivers
    st, _ = _run_tokens(vp, oc, plan, one, 4, idx, epr, recv)
    assert st == vp.ST_PACK_MISMATCH
    st, w_map = _run_tokens(vp, oc, plan, one, 4, case["expert_idx"], epr, recv[:R - 1])
    assert st == vp.ST_PACK_CAPACITY and (w_map == -1).all()


def test_dispatch_and_return_round_trip_on_gpu(vp, oracle_lib):
    """The oracle-level round trip with every pack / unpack on the GPU: dispatch pack -> exchange -> vp_unpack ->
    experts tag their rows -> return vp_pack (topk = 1, destination = source rank) -> exchange -> vp_unpack_tokens."""
    from tests.exchange import deliver
    from workloads.demand import demand_from_routing, moe_routing
    cat = complete_catalog(tree_topology(1))
    N, T, topk, E, hidden = 8, 300, 4, 32, 1024
    epr, rb = E // N, hidden * 2
    idx = moe_routing(N * T, E, topk, 0.9, seed=92).reshape(N, T, topk).to(torch.int32)
    D = demand_from_routing(idx.reshape(N * T, topk), torch.repeat_interleave(torch.arange(N), T), N, E, rb)
    w = WParams(granule_bytes=rb).resolved(N)
    oc, plan, one = _plans(vp, oracle_lib, cat, D.unsqueeze(0), w)
    _, back, back_one = _plans(vp, oracle_lib, cat, D.t().contiguous().unsqueeze(0), w)
    rows = torch.randint(0, 32768, (N, T, hidden), dtype=torch.int16, generator=torch.Generator().manual_seed(5))
    staged, meta = {}, {}
    for i in range(N):
        R = int(D[i].sum().item() // rb)
        s = torch.zeros((R, hidden), dtype=torch.int16, device="cuda")
        m = torch.full((R,), -1, dtype=torch.int32, device="cuda")
        assert int(vp.pack(plan, 0, i, idx[i].cuda().contiguous(), epr, rows[i].cuda().contiguous(), s, m).item()) == 0
        staged[i] = s.cpu().numpy().view(np.uint8).reshape(R, rb)
        meta[i] = idx[i].reshape(-1).numpy()[m.cpu().numpy()] % epr
    ret_staged = {}
    for j in range(N):
        recv, recv_expert = deliver(one, j, staged, rb, meta)
        R = recv.shape[0]
        out = torch.zeros((R, hidden), dtype=torch.int16, device="cuda")
        out_src = torch.full((R,), -1, dtype=torch.int32, device="cuda")
        off, st = vp.unpack(plan, 0, j, torch.from_numpy(recv).view(torch.int16).cuda(), torch.from_numpy(recv_expert.astype(np.int32)).cuda(),
                            epr, out, out_src=out_src)
        assert int(st.item()) == 0
        off = off.cpu().tolist()
        for e in range(epr):
            out[off[e]:off[e + 1]] ^= (j * epr + e + 1)
        s = torch.zeros((R, hidden), dtype=torch.int16, device="cuda")
        assert int(vp.pack(back, 0, j, out_src.reshape(R, 1).contiguous(), 1, out, s).item()) == 0
        ret_staged[j] = s.cpu().numpy().view(np.uint8).reshape(R, rb)
    for i in range(N):
        ret_recv, _ = deliver(back_one, i, ret_staged, rb)
        out = torch.zeros((T * topk, hidden), dtype=torch.int16, device="cuda")
        st = vp.unpack_tokens(back, 0, i, idx[i].cuda().contiguous(), epr, torch.from_numpy(ret_recv).view(torch.int16).cuda(), out)
        assert int(st.item()) == 0
        got = out.cpu().reshape(T, topk, hidden)
        e = idx[i].to(torch.int16)
        remote = (idx[i] // epr != i)
        want = (rows[i].unsqueeze(1) ^ (e + 1).unsqueeze(2)) * remote.unsqueeze(2)
        assert torch.equal(got, want.to(torch.int16))
