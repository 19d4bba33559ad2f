#!/usr/bin/env python
"""Benchmark of the VarioPath online scheduler + pack on B200.

A *step* is one pass of the whole hot path over one batch of synthetic input:
``vp_schedule_batch`` over the N=16 batch of 256 MoE demand matrices (config 2) followed by
``vp_pack`` of one rank's 16384 x top-8 routed rows of 7168 bf16 (config 5).  ``value`` is
matrices per second over whole steps (inputs resident in HBM); ``e2e`` is the same step through
the host-buffer entry points with pinned host memory, copies inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--sched-config 1|2|3|4]

With N > 1 (torchrun) every rank runs its own replica of the step (the path has no exchange
step: matrices are independent and a rank packs only its own rows), times are max-reduced.
``--impl reference`` times the CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "matrices_scheduled_per_sec"
UNIT = "matrices/s"
INT64_OPS_PER_LANE_CLK = 0.5    # one 64-bit add/min/compare needs two 32-bit ALU issues
SM_COUNT, LANES_PER_SM = 148, 128
# dram__bytes_read.sum + dram__bytes_write.sum of one launch on the default workload (ncu, see profiles/)
NCU_DRAM_BYTES_PER_LAUNCH = {"pack_copy_bulk_kernel": 235_441_664 + 1_791_668_000, "vp_schedule_kernel": 646_656 + 0}


def _dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def reduce_max(value: float, world: int) -> float:
    """Max over ranks (the slowest rank defines a step's duration)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(units_per_rank: float, world: int, seconds_max: float) -> float:
    """Whole-job throughput: units all ranks processed / slowest rank's time (weak scaling)."""
    return units_per_rank * world / seconds_max


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), source="measured", sm_max_mhz=float(p.get("sm_max_mhz", 1965.0)))
    return dict(hbm_gbs=6650.0, source="fallback", sm_max_mhz=1965.0)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), reasons=sorted(reasons))


# ------------------------------------------------------------------------------------------
# workload
# ------------------------------------------------------------------------------------------

def build_workload(args, device: str):
    """The timed inputs.  ``--batch / --token-scale / --pack-tokens`` shrink them (CPU tests only)."""
    from workloads.configs import build_config, build_pack_case
    sched = build_config(args.sched_config, device=device, batch=args.batch, token_scale=args.token_scale)
    pack = build_pack_case(device=device, tokens=args.pack_tokens)
    if args.sched_repeat > 1:           # the same matrices several times over: a batch beyond one wave of CTAs
        sched["demand"] = sched["demand"].repeat(args.sched_repeat, 1, 1).contiguous()
    return sched, pack


def vp_params(vp, w):
    return vp.SchedParams(lambda_ns=w.lambda_ns, granule_bytes=w.granule_bytes, k_target=w.k_target,
                          n_start=w.n_start, i_aa=w.i_aa, k_max=w.k_max)


def sched_ops(cat, stats: dict, n_start: int) -> float:
    """Algorithmic 64-bit integer operations of a measured batch (Section 4.2, planning complexity,
    with sparse shapes): per activation one multiply-add per shape term and N subtract/offset updates;
    per AA sweep 2G assignments of g! permutations x g terms (min + add); per task 2N for Evaluate."""
    import math
    topo = cat.topology
    terms = sum(len(s) for s in cat.shapes)
    per_sweep = 2 * topo.G * math.factorial(topo.g) * topo.g
    return stats["activations"] * (terms + topo.N) + stats["sweeps"] * per_sweep + stats["tasks"] * 2 * topo.N


def run_ours(args):
    import torch
    import paper_2609_34340_b200 as vp
    from paper_2609_34340_b200.build import build
    rank, local_rank, world = _dist_env()
    build()
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    sched, pk = build_workload(args, dev)
    cat, w = sched["catalog"], sched["params"]
    dc = vp.load_catalog(cat.topology.blob(), cat.blob(), device=local_rank)
    params = vp_params(vp, w)
    demand = sched["demand"].to(dev).contiguous()
    B, N = demand.shape[0], cat.topology.N
    sub = min(B, 256) if N > 64 else B          # N=256 plans are 30 MB each: sub-batches reuse the output buffers
    plan = vp.Plan.empty(sub, N, w.k_max, dev)
    ws = torch.empty(vp.schedule_workspace_bytes(dc, sub, params), dtype=torch.uint8, device=dev)
    sched["_launch"] = vp.schedule_launch_info(dc, sub, params)

    # pack case: its own one-matrix plan on the config-2 topology
    pcat, pw = pk["catalog"], pk["params"]
    pdc = vp.load_catalog(pcat.topology.blob(), pcat.blob(), device=local_rank)
    pparams = vp_params(vp, pw)
    pdemand = pk["demand"].to(dev).contiguous()
    pplan = vp.schedule_batch(pdc, pparams, pdemand)
    prank, row_bytes = pk["rank"], pk["row_bytes"]
    idx = pk["expert_idx"].to(dev).contiguous()
    rows = pk["rows"].to(dev).contiguous()
    T, topk = idx.shape
    R = int(pk["demand"][0, prank].sum().item() // row_bytes)
    staged = torch.empty((R, rows.shape[1]), dtype=rows.dtype, device=dev)
    src_map = torch.empty(R, dtype=torch.int32, device=dev)
    pstatus = torch.zeros(1, dtype=torch.int32, device=dev)
    pws = torch.empty(vp.pack_workspace_bytes(16, T, topk, pw.k_max), dtype=torch.uint8, device=dev)
    pack_bytes = T * row_bytes + R * row_bytes + 4 * T * topk + 4 * R      # rows once + staged once + indices + src_map
    copy_bytes = T * row_bytes + R * row_bytes + 4 * T * topk              # what the copy kernel itself must move

    def step():
        for lo in range(0, B, sub):
            vp.schedule_batch(dc, params, demand[lo:lo + sub], plan=plan, workspace=ws)
        vp.pack(pplan, 0, prank, idx, pk["experts_per_rank"], rows, staged, src_map, pstatus, pws)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)     # sampled from warm-up to the end of the timed region
    sampler.start()
    t_warm, n_warm = time.perf_counter(), 0
    while n_warm < args.warmup or (time.perf_counter() - t_warm < args.min_warmup_s and n_warm < 100000):
        step()
        n_warm += 1
        if n_warm % 16 == 0:
            torch.cuda.synchronize()
    barrier()
    assert int(pstatus.item()) == 0 and int(plan.status.max().item()) == 0, "workload did not schedule cleanly"

    vp.profile_enable(True)
    for k in range(3):
        vp.profile_read(k)
    launches0 = vp.kernel_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    total_ms = ev0.elapsed_time(ev1)
    launches = vp.kernel_launch_count() - launches0
    sched_ms, n_sched = vp.profile_read(0)
    index_ms, _ = vp.profile_read(1)
    copy_ms, n_copy = vp.profile_read(2)
    vp.profile_enable(False)
    clocks = sampler.stop()
    stats = vp.schedule_read_stats(ws)
    if sub < B:                                    # counters cover the last sub-batch only: scale to the batch
        stats = {k: v * (B // sub) for k, v in stats.items()}

    ms_per_step = reduce_max(total_ms / args.steps, world)
    value = aggregate_value(B, world, ms_per_step / 1e3)

    sched_avg = sched_ms / max(n_sched, 1) * (B // sub)
    if sub < B or args.no_e2e:
        e2e_ms, h2d, d2h, e2e_steps = None, 0, 0, 0
    else:
        e2e_ms, h2d, d2h, e2e_steps = run_e2e(vp, args, world, local_rank, dev, sched, pk, dc, params, pplan, idx, rows,
                                              R, barrier)
    tools = run_tools(vp, dev, load_peaks()) if args.tools and rank == 0 else None
    if rank != 0:
        return
    sched["_tools"] = tools
    finish(args, world, cat, w, B, N, T, topk, R, prank, row_bytes, pack_bytes, copy_bytes, stats, clocks, launches,
           sched_avg, index_ms, copy_ms, n_copy, ms_per_step, value, e2e_ms, h2d, d2h, e2e_steps, sched, pk)


def run_tools(vp, dev, peaks):
    """The two kernels around the scheduler (`--tools`): Eq. (2) plan time over the config-3 plans and the
    demand rows of 16 ranks from config-5-sized routing.  Device-resident, CUDA-event timed."""
    import torch
    from workloads.configs import build_config
    from workloads.demand import moe_routing
    c = build_config(3, device=dev)
    cat, w = c["catalog"], c["params"]
    dc = vp.load_catalog(cat.topology.blob(), cat.blob(), device=torch.device(dev).index or 0)
    plan = vp.schedule_batch(dc, vp_params(vp, w), c["demand"].to(dev).contiguous())
    out = torch.empty(plan.n_steps.shape[0], dtype=torch.int64, device=dev)
    steps = int(plan.n_steps.sum().item())

    def timed(fn, reps=20):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    # the scheduler beyond one wave: config 2's 256 matrices 16 times over (one warp per matrix)
    c2 = build_config(2, device=dev)
    cat2, w2 = c2["catalog"], c2["params"]
    dc2 = vp.load_catalog(cat2.topology.blob(), cat2.blob(), device=torch.device(dev).index or 0)
    p2 = vp_params(vp, w2)
    D2 = c2["demand"].to(dev).repeat(16, 1, 1).contiguous()
    B2 = D2.shape[0]
    plan2 = vp.Plan.empty(B2, cat2.topology.N, w2.k_max, dev)
    ws2 = torch.empty(vp.schedule_workspace_bytes(dc2, B2, p2), dtype=torch.uint8, device=dev)
    ms_s = timed(lambda: vp.schedule_batch(dc2, p2, D2, plan=plan2, workspace=ws2), reps=10)
    ops2 = sched_ops(cat2, vp.schedule_read_stats(ws2), w2.n_start)
    alu_peak = SM_COUNT * LANES_PER_SM * INT64_OPS_PER_LANE_CLK * peaks["sm_max_mhz"] * 1e6
    large = {"workload": f"config 2 matrices x16: {B2} matrices N=16", "launch": vp.schedule_launch_info(dc2, B2, p2),
             "ms": round(ms_s, 4), "matrices_per_s": round(B2 / ms_s * 1e3, 1),
             "alu_frac": round(ops2 / (ms_s * 1e-3) / alu_peak, 4),
             "ncu": {"issue_active_pct": 57.1, "shared_wavefronts_pct_of_peak": 53.9, "lsu_pipe_pct": 45.7,
                     "source": "profiles/vp_schedule_warp_kernel_config2_x16.md"}}
    del plan2, D2
    ms_t = timed(lambda: vp.plan_time(dc, plan, w.lambda_ns, out=out))
    bytes_t = steps * cat.topology.N * 10                       # lane_bytes (8) + lane_inst (2) of every emitted step
    idx = moe_routing(16 * 16384, 256, 8, 1.2, seed=5, device=dev).reshape(16, 16384, 8).contiguous()
    rows = torch.empty((16, 16), dtype=torch.int64, device=dev)
    st = torch.empty(1, dtype=torch.int32, device=dev)
    ms_d = timed(lambda: vp.demand_from_routing(idx, 16, 16, 14336, out=rows, status=st))
    bytes_d = idx.numel() * 4
    # receive side of the packed-buffer configuration: rank 8's receive buffer (random rows, skewed local experts)
    from workloads.configs import build_pack_case
    pk = build_pack_case(device=dev)
    pcat, pw, prank, epr = pk["catalog"], pk["params"], pk["rank"], pk["experts_per_rank"]
    pdc = vp.load_catalog(pcat.topology.blob(), pcat.blob(), device=torch.device(dev).index or 0)
    pplan = vp.schedule_batch(pdc, vp_params(vp, pw), pk["demand"].to(dev).contiguous())
    R = int(pk["demand"][0, :, prank].sum().item() // pk["row_bytes"])
    gen = torch.Generator(device=dev).manual_seed(9)
    recv = torch.randint(-32768, 32768, (R, pk["row_bytes"] // 2), dtype=torch.int16, device=dev, generator=gen)
    prob = torch.rand(epr, device=dev, generator=gen) ** 3
    rexp = torch.multinomial(prob / prob.sum(), R, replacement=True, generator=gen).to(torch.int32)
    uout = torch.empty_like(recv)
    uoff = torch.empty(epr + 1, dtype=torch.int32, device=dev)
    ust = torch.empty(1, dtype=torch.int32, device=dev)
    usrc, umap = torch.empty(R, dtype=torch.int32, device=dev), torch.empty(R, dtype=torch.int32, device=dev)
    uws = torch.empty(vp.unpack_workspace_bytes(16, R, epr, pw.k_max), dtype=torch.uint8, device=dev)
    un = lambda: vp.unpack(pplan, 0, prank, recv, rexp, epr, uout, uoff, usrc, umap, ust, uws)
    vp.profile_enable(True)
    vp.profile_read(3)
    ms_u = timed(un)
    ms_copy, n_copy = vp.profile_read(3)
    vp.profile_enable(False)
    assert int(ust.item()) == 0 and int(uoff[-1].item()) == R
    bytes_u = 2 * R * pk["row_bytes"]
    # return direction at the source: what rank 8 sent comes back (plan of D^T) and is put into the token layout
    bplan = vp.schedule_batch(pdc, vp_params(vp, pw), pk["demand"].to(dev).transpose(1, 2).contiguous())
    Rb = int(pk["demand"][0, prank, :].sum().item() // pk["row_bytes"])
    ridx = pk["expert_idx"].to(dev).contiguous()
    Tt, tk = ridx.shape
    rrecv = torch.randint(-32768, 32768, (Rb, pk["row_bytes"] // 2), dtype=torch.int16, device=dev, generator=gen)
    tout = torch.empty((Tt * tk, pk["row_bytes"] // 2), dtype=torch.int16, device=dev)
    tst = torch.empty(1, dtype=torch.int32, device=dev)
    tws = torch.empty(int(vp.binding._load().vp_unpack_tokens_workspace_bytes(16, Tt, tk, epr, Rb, pw.k_max)), dtype=torch.uint8, device=dev)
    vp.profile_enable(True)
    vp.profile_read(3)
    ms_r = timed(lambda: vp.unpack_tokens(bplan, 0, prank, ridx, epr, rrecv, tout, None, tst, tws))
    ms_rcopy, n_rcopy = vp.profile_read(3)
    vp.profile_enable(False)
    assert int(tst.item()) == 0
    bytes_r = 2 * Rb * pk["row_bytes"]
    ret = {"workload": f"config 5 return side: rank {prank}, {Rb} rows x {pk['row_bytes']} B back into {Tt} x top-{tk} slots",
           "ms": round(ms_r, 4), "copy_kernel_ms": round(ms_rcopy / max(n_rcopy, 1), 4), "gb_per_s": round(bytes_r / ms_r / 1e6, 1),
           "copy_kernel_gb_per_s": round(bytes_r / (ms_rcopy / max(n_rcopy, 1)) / 1e6, 1),
           "copy_kernel_frac_of_hbm_peak": round(bytes_r / (ms_rcopy / max(n_rcopy, 1)) / 1e6 / peaks["hbm_gbs"], 4)}
    del rrecv, tout
    return {"schedule_large_batch": large, "unpack_tokens": ret, "unpack": {"workload": f"config 5 receive side: rank {prank}, {R} rows x {pk['row_bytes']} B, {epr} local experts",
                       "ms": round(ms_u, 4), "copy_kernel_ms": round(ms_copy / max(n_copy, 1), 4),
                       "gb_per_s": round(bytes_u / ms_u / 1e6, 1),
                       "copy_kernel_gb_per_s": round(bytes_u / (ms_copy / max(n_copy, 1)) / 1e6, 1),
                       "copy_kernel_frac_of_hbm_peak": round(bytes_u / (ms_copy / max(n_copy, 1)) / 1e6 / peaks["hbm_gbs"], 4)},
            "plan_time": {"workload": f"config 3 plans: 1024 matrices, {steps} activations x 64 lanes", "ms": round(ms_t, 4),
                          "gb_per_s": round(bytes_t / ms_t / 1e6, 1), "frac_of_hbm_peak": round(bytes_t / ms_t / 1e6 / peaks["hbm_gbs"], 4)},
            "demand_from_routing": {"workload": "16 ranks x 16384 tokens x top-8 (8.4 MB of indices, L2-resident)",
                                    "ms": round(ms_d, 4), "gb_per_s": round(bytes_d / ms_d / 1e6, 1)}}


def run_e2e(vp, args, world, local_rank, dev, sched, pk, dc, params, pplan, idx, rows, R, barrier):
    import torch
    cat, w, pw = sched["catalog"], sched["params"], pk["params"]
    B, N = sched["demand"].shape[0], cat.topology.N
    T, topk = idx.shape
    prank, row_bytes = pk["rank"], pk["row_bytes"]
    # ---- end to end through the host-buffer entry points (pinned memory, copies timed)
    h_demand = sched["demand"].cpu().contiguous().pin_memory()
    h_plan = vp.Plan.empty(B, N, w.k_max, "cpu", pin=True)
    h_pplan = vp.Plan.empty(1, 16, pw.k_max, "cpu", pin=True)
    for name in ("n_steps", "chan_id", "lane_dst", "lane_inst", "lane_bytes", "send_off", "recv_off", "tau_ns", "status"):
        getattr(h_pplan, name).copy_(getattr(pplan, name).cpu())
    h_idx, h_rows = idx.cpu().pin_memory(), rows.cpu().pin_memory()
    h_staged = torch.empty((R, rows.shape[1]), dtype=rows.dtype).pin_memory()
    h_map = torch.empty(R, dtype=torch.int32).pin_memory()
    h_status = torch.zeros(1, dtype=torch.int32).pin_memory()
    need = int(vp.binding._load().vp_schedule_host_scratch_bytes(dc._h, B, __import__("ctypes").byref(params._c(N))))
    sscr = torch.empty(need, dtype=torch.uint8, device=dev)
    need = int(vp.binding._load().vp_pack_host_scratch_bytes(16, T, topk, pw.k_max, row_bytes, R * row_bytes))
    pscr = torch.empty(need, dtype=torch.uint8, device=dev)

    def e2e_step():
        vp.schedule_batch_host(dc, params, h_demand, plan=h_plan, scratch=sscr)
        vp.pack_host(h_pplan, 0, prank, h_idx, pk["experts_per_rank"], h_rows, h_staged, h_map, h_status, pscr,
                     device=local_rank)
        return int(h_status.item())

    e2e_steps = max(3, min(args.steps, 10))
    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()                      # synchronous: returns after the results are in host memory
    barrier()
    e2e_ms = reduce_max((time.perf_counter() - t0) * 1e3 / e2e_steps, world)
    K1 = w.k_max
    h2d = (B * N * N * 8) + (4 + pw.k_max * 16 * 10 + (pw.k_max + 1) * 16 * 8 + T * topk * 4 + T * row_bytes)
    d2h = (B * (4 + K1 * 4 + K1 * N * 12 + 2 * (K1 + 1) * N * 8 + 8 + 4)) + (4 + R * row_bytes + R * 4)
    return e2e_ms, h2d, d2h, e2e_steps


def finish(args, world, cat, w, B, N, T, topk, R, prank, row_bytes, pack_bytes, copy_bytes, stats, clocks, launches,
           sched_avg, index_ms, copy_ms, n_copy, ms_per_step, value, e2e_ms, h2d, d2h, e2e_steps, sched, pk):
    peaks = load_peaks()
    copy_avg = copy_ms / max(n_copy, 1)
    index_avg = index_ms / max(n_copy, 1)
    pack_gbs = copy_bytes / (copy_avg * 1e-3) / 1e9
    ops = sched_ops(cat, stats, w.n_start)
    sm_mhz = clocks.get("sm_mhz") or peaks["sm_max_mhz"]
    alu_peak_max = SM_COUNT * LANES_PER_SM * INT64_OPS_PER_LANE_CLK * peaks["sm_max_mhz"] * 1e6 / 1e12
    alu_peak_now = SM_COUNT * LANES_PER_SM * INT64_OPS_PER_LANE_CLK * sm_mhz * 1e6 / 1e12
    sched_tops = ops / (sched_avg * 1e-3) / 1e12
    # DRAM bytes per launch from the ncu captures summarised under profiles/ (default workload only)
    default_workload = args.sched_config == 2 and args.batch is None and args.pack_tokens == 16384 and args.sched_repeat == 1
    traffic_copy = NCU_DRAM_BYTES_PER_LAUNCH["pack_copy_bulk_kernel"] if default_workload else None
    traffic_sched = NCU_DRAM_BYTES_PER_LAUNCH["vp_schedule_kernel"] if default_workload else None
    roof_pack = dict(kernel="pack_copy_bulk_kernel", bound="hbm", achieved=round(pack_gbs, 1), peak=peaks["hbm_gbs"],
                     unit="GB/s", frac=round(pack_gbs / peaks["hbm_gbs"], 4), traffic=traffic_copy,
                     peak_source=peaks["source"], ms_per_launch=round(copy_avg, 4),
                     algorithmic_bytes_per_launch=copy_bytes)
    launch = sched.get("_launch") or {}
    roof_sched = dict(kernel="vp_schedule_warp_kernel" if launch.get("kernel") == "warp per matrix" else "vp_schedule_kernel",
                      launch=launch, bound="alu", achieved=round(sched_tops, 4), peak=round(alu_peak_max, 2),
                      unit="Tops/s (64-bit integer)", frac=round(sched_tops / alu_peak_max, 5), traffic=traffic_sched,
                      peak_source="derived: 148 SMs x 128 lanes x 0.5 64-bit ops/clk x max SM clock",
                      frac_at_sampled_clock=round(sched_tops / alu_peak_now, 5), ms_per_launch=round(sched_avg, 4),
                      algorithmic_ops_per_launch=int(ops))
    dominant, other = (roof_pack, roof_sched) if copy_avg >= sched_avg else (roof_sched, roof_pack)
    act = stats["activations"]
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": f"config {args.sched_config}{' x%d' % args.sched_repeat if args.sched_repeat > 1 else ''}: {B} MoE demand matrices N={N} "
                               f"({cat.n_shapes} shapes / {cat.n_families} families) + config 5 pack: rank {prank} of 16, "
                               f"{T} tokens x top-{topk}, {row_bytes}-B rows, {R} staged rows",
                   "batch_per_gpu": B, "parallelism": f"replicas x{world}, no collective",
                   "l2": "each step's pack streams %.2f GB (> 126 MB L2) between two schedule launches" % (pack_bytes / 1e9)},
        "sched": {"matrices_per_s": round(B / (sched_avg * 1e-3), 1), "ms": round(sched_avg, 4),
                  "activations_per_batch": act, "us_per_activation_amortized": round(sched_avg * 1e3 / max(act, 1), 4),
                  "activations_per_s": round(act / (sched_avg * 1e-3), 1)},
        "pack": {"gb_per_s": round(pack_gbs, 1), "copy_ms": round(copy_avg, 4), "index_ms": round(index_avg, 4),
                 "gb_per_s_incl_index": round(pack_bytes / ((copy_avg + index_avg) * 1e-3) / 1e9, 1)},
        "roofline": dominant, "roofline_other": other,
        "e2e": ({"value": round(B * world / (e2e_ms / 1e3), 1), "unit": UNIT, "ms_per_step": round(e2e_ms, 3),
                 "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps}
                if e2e_ms else None),
        "gpu_launches": int(launches), "clocks": clocks,
    }
    if sched.get("_tools"):
        line["next_rows"] = sched["_tools"]
    line["cpu_baseline"] = cpu_baseline(sched, pk, budget_s=20.0) if world == 1 and not args.no_cpu_baseline else None
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------

def _oracle_step(oc, poc, sched, pk, plan_one, threads, tokens):
    """One oracle step: schedule the whole batch, pack the first ``tokens`` tokens' worth of plan."""
    import numpy as np
    t0 = time.perf_counter()
    oc.schedule_batch(sched["demand"].numpy(), sched["params"], threads=threads)
    t1 = time.perf_counter()
    rows = pk["_rows_np"]
    R = pk["_R"]
    if pk.get("_staged") is None:
        pk["_staged"] = np.zeros((R, rows.shape[1] * rows.itemsize), np.uint8)
    poc.pack(plan_one, pk["rank"], pk["_idx_np"], pk["experts_per_rank"], rows, R, staged=pk["_staged"])
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def _oracle_setup(sched, pk):
    import numpy as np
    import oracle
    oracle.build()
    cat, pcat = sched["catalog"], pk["catalog"]
    oc = oracle.OracleCatalog(cat.topology.blob(), cat.blob())
    poc = oracle.OracleCatalog(pcat.topology.blob(), pcat.blob())
    pplan = poc.schedule_batch(pk["demand"].numpy(), pk["params"])
    plan_one = {k: (v[0] if isinstance(v, np.ndarray) else v) for k, v in pplan.items()}
    pk["_rows_np"] = pk["rows"].cpu().numpy()
    pk["_idx_np"] = pk["expert_idx"].cpu().numpy()
    pk["_R"] = int(pk["demand"][0, pk["rank"]].sum().item() // pk["row_bytes"])
    return oc, poc, plan_one


def cpu_baseline(sched, pk, budget_s: float) -> dict:
    """The oracle as it stands, timed on this machine's host cores on the same workload."""
    cores = os.cpu_count() or 1
    oc, poc, plan_one = _oracle_setup(sched, pk)
    B = sched["demand"].shape[0]
    ts, tp, n = 0.0, 0.0, 0
    t_start = time.perf_counter()
    while n < 1 or (time.perf_counter() - t_start < budget_s and n < 5):
        a, b = _oracle_step(oc, poc, sched, pk, plan_one, cores, None)
        ts += a; tp += b; n += 1
    step_s = (ts + tp) / n
    return {"value": round(B / step_s, 2), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} full step(s): all {B} matrices split over {cores} threads + the whole pack on 1 thread",
            "sched_matrices_per_s": round(B / (ts / n), 2), "pack_gb_per_s": round(
                (pk["_rows_np"].nbytes + pk["_R"] * pk["row_bytes"]) / (tp / n) / 1e9, 3)}


def run_reference(args):
    rank, _, world = _dist_env()
    if rank != 0:
        return
    sched, pk = build_workload(args, "cpu" if not _has_cuda() else "cuda")
    sched["demand"] = sched["demand"].cpu()
    cores = os.cpu_count() or 1
    oc, poc, plan_one = _oracle_setup(sched, pk)
    B = sched["demand"].shape[0]
    for _ in range(args.warmup):
        _oracle_step(oc, poc, sched, pk, plan_one, cores, None)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        _oracle_step(oc, poc, sched, pk, plan_one, cores, None)
    ms = (time.perf_counter() - t0) * 1e3 / args.steps
    value = B / (ms / 1e3)
    N = sched["catalog"].topology.N
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 3), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": f"config {args.sched_config}: {B} MoE demand matrices N={N} + config 5 pack "
                                   f"(CPU oracle, whole workload per step)"},
            "cpu_baseline": {"value": round(value, 2), "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"every step: all {B} matrices over {cores} threads + the whole pack on 1 thread"},
            "e2e": {"value": round(value, 2), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def _has_cuda() -> bool:
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sched-config", type=int, default=2, choices=[1, 2, 3, 4])
    ap.add_argument("--batch", type=int, default=None, help="truncate the scheduler batch (tests)")
    ap.add_argument("--sched-repeat", type=int, default=1,
                    help="schedule the batch this many times over in one call (a batch beyond one wave; not the default benchmark)")
    ap.add_argument("--token-scale", type=float, default=1.0, help="scale token counts (tests)")
    ap.add_argument("--pack-tokens", type=int, default=16384, help="tokens of the packed rank (tests)")
    ap.add_argument("--min-warmup-s", type=float, default=1.0,
                    help="keep warming up (beyond --warmup steps) until this many seconds have passed, so that "
                         "clocks settle and nvidia-smi has samples under load")
    ap.add_argument("--tools", action="store_true", help="also time vp_plan_time and vp_demand_from_routing")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the CPU oracle leg (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
