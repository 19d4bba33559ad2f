"""GPU parity: vp_pack (through the C ABI) against the CPU oracle, byte for byte."""
import os

import numpy as np
import pytest
import torch

from workloads import SchedParams as WParams, complete_catalog, tree_topology
from workloads.configs import build_pack_case

pytestmark = pytest.mark.gpu
GUARD = 64    # guard rows after the staged buffer: must stay untouched


@pytest.fixture(scope="module")
def vp():
    import paper_2609_34340_b200 as vp
    assert torch.cuda.is_available(), "these tests need a GPU"
    assert os.path.exists(vp.library_path()), "libvariopath.so has not been built"
    return vp


def _params(vp, w):
    return vp.SchedParams(lambda_ns=w.lambda_ns, granule_bytes=w.granule_bytes, k_target=w.k_target,
                          n_start=w.n_start, i_aa=w.i_aa, k_max=w.k_max)


def _run_case(vp, oracle_lib, case, capacity_rows=None, rows_override=None):
    cat = case["catalog"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    w = case["params"]
    plan = vp.schedule_batch(dc, _params(vp, w), case["demand"].cuda())
    want_plan = oc.schedule_batch(case["demand"].numpy(), w)
    one = {k: (v[0] if isinstance(v, np.ndarray) else v) for k, v in want_plan.items()}
    rank = case["rank"]
    rows = case["rows"] if rows_override is None else rows_override
    idx = case["expert_idx"].cuda().contiguous()
    row_bytes = rows.shape[1] * rows.element_size()
    R = int(case["demand"][0, rank].sum().item() // row_bytes) if capacity_rows is None else capacity_rows
    staged = torch.zeros((R + GUARD, rows.shape[1]), dtype=rows.dtype, device="cuda")
    staged[R:] = 0x55 if rows.dtype == torch.uint8 else 0x5555
    src_map = torch.full((R + GUARD,), -1, dtype=torch.int32, device="cuda")
    status = vp.pack(plan, 0, rank, idx, case["experts_per_rank"], rows.cuda().contiguous(), staged[:R], src_map)
    torch.cuda.synchronize()
    want_staged, want_map, want_st = oc.pack(one, rank, idx.cpu().numpy(), case["experts_per_rank"],
                                             rows.cpu().numpy(), R)
    return (staged.cpu().numpy(), src_map.cpu().numpy(), int(status.item()),
            want_staged, want_map, want_st, R)


def _assert_pack(res):
    staged, src_map, st, want_staged, want_map, want_st, R = res
    assert st == want_st
    assert np.array_equal(src_map[:R], want_map)
    assert np.array_equal(staged[:R].view(np.uint8).reshape(R, -1), want_staged)
    guard = staged[R:].view(np.uint8)
    assert (guard == 0x55).all() and (src_map[R:] == -1).all()       # nothing written past the buffer


@pytest.mark.parametrize("tokens,hidden,rank", [(300, 1024, 0), (300, 1024, 9), (1000, 7168, 3), (257, 8200, 15)])
def test_pack_matches_oracle_bulk_path(vp, oracle_lib, tokens, hidden, rank):
    case = build_pack_case(device="cuda", tokens=tokens, hidden=hidden, rank=rank, seed=11)
    res = _run_case(vp, oracle_lib, case)
    assert res[2] == 0
    _assert_pack(res)


@pytest.mark.parametrize("hidden,dtype", [(64, torch.int16), (1000, torch.int16), (333, torch.uint8), (6, torch.int16)])
def test_pack_matches_oracle_plain_path(vp, oracle_lib, hidden, dtype):
    """Short rows and rows whose size is not a multiple of 16 bytes take the plain-load kernel."""
    case = build_pack_case(device="cuda", tokens=500, hidden=hidden, rank=2, seed=12)
    rows = case["rows"]
    if dtype == torch.uint8:
        rows = (rows & 0xFF).to(torch.uint8)
        rb = hidden
        case["demand"] = case["demand"] // case["row_bytes"] * rb
        case["params"] = WParams(granule_bytes=rb).resolved(16)
    res = _run_case(vp, oracle_lib, case, rows_override=rows)
    assert res[2] == 0
    _assert_pack(res)


def test_pack_with_dropped_copies_and_other_topk(vp, oracle_lib):
    case = build_pack_case(device="cuda", tokens=400, hidden=2048, rank=1, seed=13, topk=4, experts=64)
    idx = case["expert_idx"].clone()
    idx[::5, 1] = -1
    # the demand row of this rank must describe the routing that is packed
    epr, rb = case["experts_per_rank"], case["row_bytes"]
    dest = (idx.cpu().numpy() // epr)
    counts = np.bincount(dest[idx.cpu().numpy() >= 0], minlength=16)
    counts[1] = 0
    case["demand"][0, 1] = torch.from_numpy(counts * rb)
    case["expert_idx"] = idx
    res = _run_case(vp, oracle_lib, case)
    assert res[2] == 0
    _assert_pack(res)


def test_pack_error_statuses(vp, oracle_lib):
    case = build_pack_case(device="cuda", tokens=200, hidden=1024, rank=0, seed=14)
    R = int(case["demand"][0, 0].sum().item() // case["row_bytes"])
    res = _run_case(vp, oracle_lib, case, capacity_rows=R - 1)
    assert res[2] == vp.ST_PACK_CAPACITY == res[5]
    assert not res[0][:R - 1].any()                                  # nothing copied
    other = dict(case)
    idx = case["expert_idx"].clone()
    idx[0, 0] = (idx[0, 0] + case["experts_per_rank"]) % 256
    other["expert_idx"] = idx
    res = _run_case(vp, oracle_lib, other)
    assert res[2] & vp.ST_PACK_MISMATCH and res[5] & vp.ST_PACK_MISMATCH


def test_pack_host_variant(vp, oracle_lib):
    case = build_pack_case(device="cuda", tokens=300, hidden=2048, rank=4, seed=15)
    cat = case["catalog"]
    oc = oracle_lib.OracleCatalog(cat.topology.blob(), cat.blob())
    dc = vp.load_catalog(cat.topology.blob(), cat.blob())
    plan = vp.schedule_batch_host(dc, _params(vp, case["params"]), case["demand"].pin_memory())
    R = int(case["demand"][0, 4].sum().item() // case["row_bytes"])
    rows = case["rows"].cpu().pin_memory()
    idx = case["expert_idx"].cpu().pin_memory()
    staged = torch.zeros((R, rows.shape[1]), dtype=rows.dtype).pin_memory()
    src_map = torch.full((R,), -1, dtype=torch.int32).pin_memory()
    st = vp.pack_host(plan, 0, 4, idx, case["experts_per_rank"], rows, staged, src_map)
    one = {k: (v[0] if isinstance(v, np.ndarray) else v) for k, v in plan.cpu().items()}
    want_staged, want_map, want_st = oc.pack(one, 4, idx.numpy(), case["experts_per_rank"], rows.numpy(), R)
    assert int(st.item()) == want_st == 0
    assert np.array_equal(src_map.numpy(), want_map)
    assert np.array_equal(staged.numpy().view(np.uint8).reshape(R, -1), want_staged)


def test_config5_full_size(vp, oracle_lib):
    """16384 tokens x top-8, 7168 bf16 per row (about 1.9 GB staged): byte-exact against the oracle."""
    case = build_pack_case(device="cuda")
    res = _run_case(vp, oracle_lib, case)
    assert res[2] == 0
    _assert_pack(res)
    assert res[6] * case["row_bytes"] > 1.7e9


@pytest.mark.parametrize("hidden", [1024, 64])
def test_pack_with_more_than_32_copies_per_token(vp, oracle_lib, hidden):
    """top-40 routing: the copy handles the destinations of a token 32 slots at a time."""
    case = build_pack_case(device="cuda", tokens=150, hidden=hidden, rank=5, seed=14, topk=40, experts=256)
    res = _run_case(vp, oracle_lib, case)
    assert res[2] == 0
    _assert_pack(res)
