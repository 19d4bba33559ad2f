"""The benchmark's multi-rank plumbing on CPU: two gloo ranks, no GPU."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(code_or_args, world, extra_env=None, script=None):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PYTHONPATH=ROOT)
        env.update(extra_env or {})
        cmd = [sys.executable] + ([script] + code_or_args if script else ["-c", code_or_args])
        procs.append(subprocess.Popen(cmd, env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    return [(p.returncode, o, e) for p, (o, e) in zip(procs, outs)]


def test_max_reduction_and_aggregation_over_two_gloo_ranks():
    code = (
        "import os, torch.distributed as dist, bench\n"
        "dist.init_process_group('gloo')\n"
        "r = dist.get_rank()\n"
        "ms = bench.reduce_max(1.0 + r, dist.get_world_size())\n"
        "print(ms, bench.aggregate_value(256, dist.get_world_size(), ms / 1e3))\n"
        "dist.destroy_process_group()\n")
    res = _spawn(code, 2)
    for rc, out, err in res:
        assert rc == 0, err
        ms, value = (float(x) for x in out.split())
        assert ms == 2.0                      # the slowest rank defines the step
        assert value == 256 * 2 / 2e-3        # whole-job units / slowest time


def test_reference_arm_runs_on_rank0_only():
    args = ["--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--sched-config", "1",
            "--batch", "3", "--token-scale", "0.02", "--pack-tokens", "128"]
    res = _spawn(args, 2, script=os.path.join(ROOT, "bench.py"))
    (rc0, out0, err0), (rc1, out1, err1) = res
    assert rc0 == 0, err0
    assert rc1 == 0 and out1.strip() == ""    # other ranks exit 0 without work
    line = json.loads(out0.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    for key in ("metric", "unit", "steps", "warmup", "ms_per_step", "higher_is_better", "config"):
        assert key in line


def test_exchange_tables_over_two_gloo_ranks():
    """Host side of a multi-rank exchange: every rank learns every rank's receive-buffer address, counter address and
    capacity, indexed by rank (two gloo ranks on CPU; the addresses are stand-ins)."""
    code = (
        "import torch.distributed as dist\n"
        "import paper_2609_34340_b200 as vp\n"
        "dist.init_process_group('gloo')\n"
        "r = dist.get_rank()\n"
        "bufs, ctrs, caps = vp.gather_exchange_tables(0x1000 * (r + 1), 0x2000 * (r + 1) + 8, 4096 * (r + 3))\n"
        "import json; print(json.dumps([bufs.tolist(), ctrs.tolist(), caps.tolist()]))\n"
        "dist.destroy_process_group()\n")
    res = _spawn(code, 2)
    for rc, out, err in res:
        assert rc == 0, err
        assert json.loads(out.strip().splitlines()[-1]) == [[0x1000, 0x2000], [0x2008, 0x4008], [4096 * 3, 4096 * 4]]
