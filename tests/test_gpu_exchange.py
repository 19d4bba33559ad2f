"""GPU parity of the exchange step (vp_exchange_put / vp_exchange_wait) against the CPU oracle: every rank's chunks land
where the plan says, the arrival counters end at the receive totals, the bounded wait returns, and a wait that cannot
be satisfied gives up with a status bit instead of hanging."""
import os

import numpy as np
import pytest
import torch

from workloads import SchedParams as WParams, complete_catalog, tree_topology
from workloads.demand import demand_from_routing, moe_routing

pytestmark = pytest.mark.gpu
GUARD = 256


@pytest.fixture(scope="module")
def vp():
    import paper_2609_34340_b200 as vp
    assert torch.cuda.is_available(), "these tests need a GPU"
    assert os.path.exists(vp.library_path()), "libvariopath.so has not been built"
    return vp


def _case(vp, oracle_lib, nodes, T, topk, E, row_bytes, seed):
    """Routing -> demand -> plan (GPU and oracle) -> every rank's staged buffer packed on the GPU."""
    cat = complete_catalog(tree_topology(nodes))
    N = cat.topology.N
    epr = E // N
    idx = moe_routing(N * T, E, topk, 1.0, seed=seed).reshape(N, T, topk).to(torch.int32)
    D = demand_from_routing(idx.reshape(N * T, topk), torch.repeat_interleave(torch.arange(N), T), N, E, row_bytes)
    w = WParams(granule_bytes=row_bytes).resolved(N)
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    p = vp.SchedParams(lambda_ns=w.lambda_ns, granule_bytes=w.granule_bytes, k_target=w.k_target, n_start=w.n_start, i_aa=w.i_aa,
                       k_max=w.k_max)
    plan = vp.schedule_batch(dc, p, D.unsqueeze(0).cuda().contiguous())
    want = oc.schedule_batch(D.unsqueeze(0).numpy(), w)
    one = {k: (v[0] if isinstance(v, np.ndarray) else v) for k, v in want.items()}
    rows = torch.randint(0, 256, (N, T, row_bytes), dtype=torch.uint8, generator=torch.Generator().manual_seed(seed + 1))
    staged = []
    for i in range(N):
        R = int(D[i].sum().item() // row_bytes)
        s = torch.zeros((max(R, 1), row_bytes), dtype=torch.uint8, device="cuda")
        st = vp.pack(plan, 0, i, idx[i].cuda().contiguous(), epr, rows[i].cuda().contiguous(), s[:R])
        assert int(st.item()) == 0
        staged.append(s[:R])
    return dict(N=N, D=D, oc=oc, plan=plan, one=one, staged=staged, keep=dc)


def _buffers(c, shrink_rank=None):
    N, D = c["N"], c["D"]
    cap = D.sum(0).tolist()
    if shrink_rank is not None:
        cap[shrink_rank] = max(0, cap[shrink_rank] - 16)
    bufs = [torch.full((int(cap[j]) + GUARD,), 0xAB, dtype=torch.uint8, device="cuda") for j in range(N)]
    counters = torch.zeros(N, dtype=torch.int64, device="cuda")
    ptrs = torch.tensor([b.data_ptr() for b in bufs], dtype=torch.int64, device="cuda")
    cptrs = torch.tensor([counters[j:].data_ptr() for j in range(N)], dtype=torch.int64, device="cuda")
    caps = torch.tensor(cap, dtype=torch.int64, device="cuda")
    return bufs, counters, ptrs, cptrs, caps, cap


@pytest.mark.parametrize("nodes,T,topk,E,row_bytes", [(2, 300, 8, 256, 2048), (1, 77, 4, 32, 6), (2, 40, 2, 64, 4096 + 16)])
def test_exchange_put_matches_oracle(vp, oracle_lib, nodes, T, topk, E, row_bytes):
    c = _case(vp, oracle_lib, nodes, T, topk, E, row_bytes, seed=nodes * 100 + T)
    N = c["N"]
    bufs, counters, ptrs, cptrs, caps, cap = _buffers(c)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for i in range(N):                                    # every sender first ...
        vp.exchange_put(c["plan"], 0, i, c["staged"][i], ptrs, caps, cptrs, status)
    for j in range(N):                                    # ... then every receiver's bounded wait, on the same stream
        vp.exchange_wait(c["plan"], 0, j, counters[j:], 0, 1000, status)
    torch.cuda.synchronize()
    want_bufs, want_arrived, want_st = c["oc"].exchange(c["one"], {i: c["staged"][i].cpu().numpy() for i in range(N)})
    assert int(status.item()) == want_st == 0
    assert counters.cpu().tolist() == [int(x) for x in want_arrived] == cap
    for j in range(N):
        got = bufs[j].cpu().numpy()
        assert np.array_equal(got[:cap[j]], want_bufs[j]), j
        assert (got[cap[j]:] == 0xAB).all(), j            # nothing past the receive total


def test_exchange_refuses_to_overrun_a_receive_buffer(vp, oracle_lib):
    c = _case(vp, oracle_lib, 1, 50, 4, 32, 64, seed=9)
    N = c["N"]
    bufs, counters, ptrs, cptrs, caps, cap = _buffers(c, shrink_rank=3)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for i in range(N):
        vp.exchange_put(c["plan"], 0, i, c["staged"][i], ptrs, caps, cptrs, status)
    torch.cuda.synchronize()
    assert int(status.item()) == vp.ST_PACK_CAPACITY
    assert (bufs[3].cpu().numpy()[cap[3]:] == 0xAB).all()  # the chunk that did not fit was not written at all
    assert int(counters[3].item()) < int(c["D"].sum(0)[3])


def test_exchange_wait_gives_up_with_a_status_bit(vp, oracle_lib):
    """A counter that nothing advances: the wait runs out of polls, reports it, and the context stays usable."""
    c = _case(vp, oracle_lib, 1, 20, 2, 16, 32, seed=4)
    counter = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rank = int(np.argmax(c["D"].sum(0).numpy()))
    vp.exchange_wait(c["plan"], 0, rank, counter, 0, 2000, status)
    torch.cuda.synchronize()
    assert int(status.item()) == vp.ST_EXCHANGE_TIMEOUT
    # with the counter already at the total (as after the senders' puts) the same wait returns at its first poll
    counter.fill_(int(c["D"].sum(0)[rank]))
    status.zero_()
    vp.exchange_wait(c["plan"], 0, rank, counter, 0, 2000, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert int((torch.arange(10, device="cuda") * 2).sum().item()) == 90      # the context still runs kernels
