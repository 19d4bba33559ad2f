#!/usr/bin/env python
"""Benchmark of the VarioPath online scheduler + pack on B200.

A *step* is one pass of the whole hot path over one batch of synthetic input: ``vp_schedule_batch`` over the
N=256 batch of 4096 demand matrices (config 4, in sub-batches that reuse the plan buffers) followed by ``vp_pack``
of one rank's 16384 x top-8 routed rows of 7168 bf16 (config 5).  ``value`` is matrices per second over whole
steps with inputs resident in HBM; ``e2e`` is the same step through the host-buffer entry points with pinned host
memory, copies inside the timed region.  Beside the headline the line carries

* ``sched_configs``: the scheduler alone on configs 1, 2 and 3 (L2 flushed between launches),
* ``peaks``: integer-issue, shared-memory and write-only rates measured in this run by the library's probes,
* ``roofline`` (scheduler, the dominant kernel) and ``roofline_other`` (pack copy kernel),
* ``cpu_baseline``: the CPU oracle on a bounded sample of the same workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--sched-config 1|2|3|4]

With N > 1 (torchrun) every rank runs its own replica of the step (the path has no exchange step: matrices are
independent and a rank packs only its own rows); times are max-reduced.  ``--impl reference`` times the CPU oracle
on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import math
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
SM_COUNT, SCHEDULERS_PER_SM = 148, 4
COUNTERS_JSON = os.path.join(ROOT, "profiles", "ncu_counters.json")


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


def load_counters() -> dict:
    """Per-kernel ncu counters of earlier captures (warp instructions and shared-memory wavefronts per activation,
    DRAM bytes per launch), kept under profiles/ with the commit they were captured at."""
    try:
        with open(COUNTERS_JSON) as f:
            return json.load(f)
    except (OSError, ValueError):
        return {}


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


def workload_string(args, sched, pk) -> str:
    """Names the step's workload; both arms build it from the same inputs, so the strings are identical."""
    cat = sched["catalog"]
    B, N = sched["demand"].shape[0], cat.topology.N
    T, topk = pk["expert_idx"].shape
    R = int(pk["demand"][0, pk["rank"]].sum().item() // pk["row_bytes"])
    kind = {1: "MoE", 2: "MoE", 3: "MoE", 4: "MoE + sequence-parallel"}[args.sched_config]
    rep = " x%d" % args.sched_repeat if args.sched_repeat > 1 else ""
    return (f"config {args.sched_config}{rep}: {B} {kind} demand matrices N={N} ({cat.n_shapes} shapes / "
            f"{cat.n_families} families) + config 5 pack: rank {pk['rank']} of 16, {T} tokens x top-{topk}, "
            f"{pk['row_bytes']}-B rows, {R} staged rows")


def vp_params(vp, w):
    return vp.SchedParams(lambda_ns=w.lambda_ns, granule_bytes=w.granule_bytes, k_target=w.k_target,
                          n_start=w.n_start, i_aa=w.i_aa, k_max=w.k_max)


def sched_ops(cat, stats: dict, n_start: int) -> float:
    """Algorithmic integer operations of a measured batch (Section 4.2, planning complexity, with sparse
    shapes): per activation one multiply-add per shape term and N subtract/offset updates; per AA sweep 2G
    assignments of g! permutations x g terms (min + add); per task 2N for Evaluate."""
    topo = cat.topology
    terms = sum(len(s) for s in cat.shapes)
    per_sweep = 2 * topo.G * math.factorial(topo.g) * topo.g
    return stats["activations"] * (terms + topo.N) + stats["sweeps"] * per_sweep + stats["tasks"] * 2 * topo.N


class SchedRun:
    """One scheduler workload on the device: the batch goes through ``vp_schedule_batch`` in sub-batches that
    reuse one set of plan buffers (a config-4 plan is 29 MB per matrix)."""

    def __init__(self, vp, torch, sched, dev, local_rank, sub_batch):
        self.vp, self.torch = vp, torch
        cat, w = sched["catalog"], sched["params"]
        self.cat, self.w = cat, w
        self.dc = vp.load_catalog(cat.topology.blob(), cat.blob(), device=local_rank)
        self.params = vp_params(vp, w)
        self.demand = sched["demand"].to(dev).contiguous()
        self.B, self.N = self.demand.shape[0], cat.topology.N
        per_matrix = w.k_max * self.N * 12 + 2 * (w.k_max + 1) * self.N * 8
        fit = max(1, int(64e9 // per_matrix))                    # at most ~64 GB of plan buffers
        self.sub = min(self.B, sub_batch or self.B, fit)
        self.plan = vp.Plan.empty(self.sub, self.N, w.k_max, dev)
        self.ws = torch.empty(vp.schedule_workspace_bytes(self.dc, self.sub, self.params), dtype=torch.uint8, device=dev)
        self.launch = vp.schedule_launch_info(self.dc, self.sub, self.params)
        self.calls = (self.B + self.sub - 1) // self.sub

    def run(self):
        for lo in range(0, self.B, self.sub):
            self.vp.schedule_batch(self.dc, self.params, self.demand[lo:lo + self.sub], plan=self.plan, workspace=self.ws)

    def stats_whole_batch(self) -> dict:
        """Work counters of the whole batch: the workspace holds those of the last call, so one extra pass reads
        them call by call (outside any timed region)."""
        total = dict(activations=0, tasks=0, sweeps=0)
        for lo in range(0, self.B, self.sub):
            self.vp.schedule_batch(self.dc, self.params, self.demand[lo:lo + self.sub], plan=self.plan, workspace=self.ws)
            st = self.vp.schedule_read_stats(self.ws)
            assert int(self.plan.status[: min(self.sub, self.B - lo)].max().item()) == 0, "workload did not schedule cleanly"
            for k in total:
                total[k] += st[k]
        # bytes of the plan rows in use (what vp_schedule_batch_host_used brings back): per activation N lanes of
        # 2 + 2 + 8 bytes, a chan_id and two offset rows, plus one more offset row pair per matrix
        self.used_rows_bytes = total["activations"] * (self.N * 12 + 4 + 2 * self.N * 8) + self.B * 2 * self.N * 8
        return total


def event_pair(torch):
    return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)


def measure_peaks(vp, torch, dev, staged) -> dict:
    """Integer-issue and shared-memory rates from the library's probes, and the write-only rate of a
    ``cudaMemsetAsync`` over the staged buffer.  Best of five launches each, CUDA events."""
    sink = torch.zeros(1, dtype=torch.int64, device=dev)
    out = {}
    for name, kind, iters, scale, unit in (("int32_add_min_tops", 0, 400, 1e12, "Tops/s"), ("int64_add_min_tops", 1, 200, 1e12, "Tops/s"),
                                           ("smem_load32_tbs", 2, 400, 1e12, "TB/s"), ("smem_load64_tbs", 3, 400, 1e12, "TB/s")):
        best = 0.0
        vp.microbench(kind, iters, sink)
        for _ in range(5):
            e0, e1 = event_pair(torch)
            e0.record()
            units = vp.microbench(kind, iters, sink)
            e1.record()
            torch.cuda.synchronize()
            best = max(best, units / (e0.elapsed_time(e1) * 1e-3) / scale)
        out[name] = round(best, 3)
    best = 0.0
    for _ in range(6):
        e0, e1 = event_pair(torch)
        e0.record()
        n = vp.memset_probe(staged)
        e1.record()
        torch.cuda.synchronize()
        best = max(best, n / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    out["write_only_gbs"] = round(best, 1)
    out["how"] = ("vp_microbench kinds 0-3 (every warp slot of every SM busy, eight independent chains per thread) and "
                  "cudaMemsetAsync over the staged buffer; best of 5, CUDA events, at the clock sampled in this run")
    return out


def time_sched_config(vp, torch, idx, dev, local_rank, flush, peaks_now, counters, reps=20) -> dict:
    """The scheduler alone on config ``idx``: L2 flushed (a 256 MB fill) before every timed launch."""
    from workloads.configs import build_config
    sched = build_config(idx, device=dev)
    run = SchedRun(vp, torch, sched, dev, local_rank, None)
    for _ in range(3):
        run.run()
    torch.cuda.synchronize()
    times = []
    for _ in range(reps):
        flush.zero_()
        e0, e1 = event_pair(torch)
        e0.record()
        run.run()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    stats = run.stats_whole_batch()
    ms = statistics.median(times)
    act = stats["activations"]
    ops = sched_ops(run.cat, stats, run.w.n_start)
    out = {"workload": f"config {idx}: {run.B} matrices N={run.N} ({run.cat.n_shapes} shapes / {run.cat.n_families} families)",
           "launch": run.launch, "ms": round(ms, 4), "ms_best": round(min(times), 4),
           "matrices_per_s": round(run.B / ms * 1e3, 1), "activations": act,
           "activations_per_s": round(act / ms * 1e3, 1), "us_per_activation": round(ms * 1e3 / max(act, 1), 4),
           "algorithmic_int_ops": int(ops),
           "alu_frac_of_measured_int32_peak": round(ops / (ms * 1e-3) / 1e12 / peaks_now["int32_add_min_tops"], 5)}
    out.update(issue_fraction(counters, f"config{idx}", act, ms, peaks_now.get("sm_mhz")))
    return out


def issue_fraction(counters: dict, key: str, activations: int, ms: float, sm_mhz) -> dict:
    """Issue-slot and shared-memory-pipe use from the warp instructions / wavefronts per activation that an ncu
    capture of the same kernel and config recorded (profiles/ncu_counters.json), over this run's time and clock."""
    c = (counters.get("scheduler") or {}).get(key)
    if not c or not sm_mhz:
        return {"issue_slot_frac": None, "shared_wavefront_frac": None}
    cycles = ms * 1e-3 * sm_mhz * 1e6
    inst = c["warp_inst_per_activation"] * activations
    wave = c["shared_wavefronts_per_activation"] * activations
    return {"issue_slot_frac": round(inst / (cycles * SM_COUNT * SCHEDULERS_PER_SM), 4),
            "shared_wavefront_frac": round(wave / (cycles * SM_COUNT), 4),
            "counters_from": f"profiles/ncu_counters.json ({c.get('source', '?')}, commit {c.get('commit', counters.get('commit', '?'))})",
            "ncu_issue_active_pct": c.get("issue_active_pct"), "ncu_shared_wavefront_pct": c.get("shared_wavefront_pct")}


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
    run = SchedRun(vp, torch, sched, dev, local_rank, args.sub_batch)
    cat, w, B, N = run.cat, run.w, run.B, run.N

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
        run.run()
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
    assert int(pstatus.item()) == 0 and int(run.plan.status.max().item()) == 0, "workload did not schedule cleanly"

    vp.profile_enable(True)
    for k in range(3):
        vp.profile_read(k)
    launches0 = vp.kernel_launch_count()
    ev0, ev1 = event_pair(torch)
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
    stats = run.stats_whole_batch()

    ms_per_step = reduce_max(total_ms / args.steps, world)
    value = aggregate_value(B, world, ms_per_step / 1e3)
    sched_per_step = sched_ms / max(args.steps, 1)               # all scheduler launches of one step
    sched_per_launch = sched_ms / max(n_sched, 1)

    extras = {}
    if rank == 0 and world == 1 and not args.no_extras:
        sampler2 = ClockSampler(local_rank)
        sampler2.start()
        peaks_now = measure_peaks(vp, torch, dev, staged)
        peaks_now["sm_mhz"] = clocks.get("sm_mhz") or load_peaks()["sm_max_mhz"]
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        counters = load_counters()
        extras["peaks"] = peaks_now
        extras["sched_configs"] = {}
        for idx_cfg in (1, 2, 3):
            if idx_cfg != args.sched_config:
                extras["sched_configs"][f"config{idx_cfg}"] = time_sched_config(vp, torch, idx_cfg, dev, local_rank, flush, peaks_now, counters)
        extras["clocks_extras"] = sampler2.stop()
        del flush
    if args.no_e2e:
        e2e = None
    else:
        e2e = run_e2e(vp, args, world, local_rank, dev, run, pk, pplan, idx, rows, R, barrier)
    tools = run_tools(vp, dev, load_peaks()) if args.tools and rank == 0 else None
    if rank != 0:
        return
    finish(args, world, run, sched, pk, T, topk, R, pack_bytes, copy_bytes, stats, clocks, launches, sched_per_step,
           sched_per_launch, n_sched, index_ms, copy_ms, n_copy, ms_per_step, value, e2e, extras, tools)


def run_tools(vp, dev, peaks):
    """The kernels around the scheduler (`--tools`): Eq. (2) plan time over the config-3 plans, the demand rows of
    16 ranks from config-5-sized routing, both unpack directions, and the warp-per-matrix kernel beyond one wave.
    Device-resident, CUDA-event timed."""
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
    large = {"workload": f"config 2 matrices x16: {B2} matrices N=16", "launch": vp.schedule_launch_info(dc2, B2, p2),
             "ms": round(ms_s, 4), "matrices_per_s": round(B2 / ms_s * 1e3, 1)}
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
    # plan execution, sender side: rank 8 puts its staged buffer (1.85 GB) into the 15 receivers' buffers on this GPU
    Rs = int(pk["demand"][0, prank, :].sum().item() // pk["row_bytes"])
    xstaged = torch.randint(-32768, 32768, (Rs, pk["row_bytes"] // 2), dtype=torch.int16, device=dev, generator=gen)
    capv = [int(pk["demand"][0, :, j].sum().item()) for j in range(16)]
    xbufs = [torch.empty(max(cj, 16), dtype=torch.uint8, device=dev) for cj in capv]
    xcnt = torch.zeros(16, dtype=torch.int64, device=dev)
    xptr = torch.tensor([t_.data_ptr() for t_ in xbufs], dtype=torch.int64, device=dev)
    xcptr = torch.tensor([xcnt[j:].data_ptr() for j in range(16)], dtype=torch.int64, device=dev)
    xcap = torch.tensor(capv, dtype=torch.int64, device=dev)
    xst = torch.zeros(1, dtype=torch.int32, device=dev)
    ms_x = timed(lambda: vp.exchange_put(pplan, 0, prank, xstaged, xptr, xcap, xcptr, xst))
    assert int(xst.item()) == 0
    bytes_x = 2 * Rs * pk["row_bytes"]
    xput = {"workload": f"config 5 sender side: rank {prank} puts {Rs} rows x {pk['row_bytes']} B into 15 receive buffers on the same GPU",
            "ms": round(ms_x, 4), "gb_per_s": round(bytes_x / ms_x / 1e6, 1), "frac_of_hbm_peak": round(bytes_x / ms_x / 1e6 / peaks["hbm_gbs"], 4)}
    del xstaged, xbufs
    return {"schedule_large_batch": large, "exchange_put": xput, "unpack_tokens": ret, "unpack": {"workload": f"config 5 receive side: rank {prank}, {R} rows x {pk['row_bytes']} B, {epr} local experts",
                       "ms": round(ms_u, 4), "copy_kernel_ms": round(ms_copy / max(n_copy, 1), 4),
                       "gb_per_s": round(bytes_u / ms_u / 1e6, 1),
                       "copy_kernel_gb_per_s": round(bytes_u / (ms_copy / max(n_copy, 1)) / 1e6, 1),
                       "copy_kernel_frac_of_hbm_peak": round(bytes_u / (ms_copy / max(n_copy, 1)) / 1e6 / peaks["hbm_gbs"], 4)},
            "plan_time": {"workload": f"config 3 plans: 1024 matrices, {steps} activations x 64 lanes", "ms": round(ms_t, 4),
                          "gb_per_s": round(bytes_t / ms_t / 1e6, 1), "frac_of_hbm_peak": round(bytes_t / ms_t / 1e6 / peaks["hbm_gbs"], 4)},
            "demand_from_routing": {"workload": "16 ranks x 16384 tokens x top-8 (8.4 MB of indices, L2-resident)",
                                    "ms": round(ms_d, 4), "gb_per_s": round(bytes_d / ms_d / 1e6, 1)}}


def run_e2e(vp, args, world, local_rank, dev, run, pk, pplan, idx, rows, R, barrier):
    """The same step through the host-buffer entry points: demand, routing and rows start in pinned host memory,
    plans and the staged buffer end there; every copy is inside the timed region.  The scheduler batch goes
    through ``vp_schedule_batch_host`` in sub-batches that reuse one pinned plan buffer."""
    import ctypes
    import torch
    cat, w, pw = run.cat, run.w, pk["params"]
    B, N = run.B, run.N
    T, topk = idx.shape
    prank, row_bytes = pk["rank"], pk["row_bytes"]
    per_matrix = w.k_max * N * 12 + 2 * (w.k_max + 1) * N * 8
    # at most ~16 GB pinned at a time: the host-buffer call works through such a sub-batch in chunks of about one matrix per
    # SM, decomposing one chunk while the results of the chunk before it travel to the host
    sub = max(1, min(B, int(16e9 // per_matrix)))
    h_demand = run.demand.cpu().contiguous().pin_memory()
    h_plan = vp.Plan.empty(sub, N, w.k_max, "cpu", pin=True)
    h_pplan = vp.Plan.empty(1, 16, pw.k_max, "cpu", pin=True)
    for name in ("n_steps", "chan_id", "lane_dst", "lane_inst", "lane_bytes", "send_off", "recv_off", "tau_ns", "status"):
        getattr(h_pplan, name).copy_(getattr(pplan, name).cpu())
    h_idx, h_rows = idx.cpu().pin_memory(), rows.cpu().pin_memory()
    h_staged = torch.empty((R, rows.shape[1]), dtype=rows.dtype).pin_memory()
    h_map = torch.empty(R, dtype=torch.int32).pin_memory()
    h_status = torch.zeros(1, dtype=torch.int32).pin_memory()
    need = int(vp.binding._load().vp_schedule_host_scratch_bytes(run.dc._h, sub, ctypes.byref(run.params._c(N))))
    sscr = torch.empty(need, dtype=torch.uint8, device=dev)
    need = int(vp.binding._load().vp_pack_host_scratch_bytes(16, T, topk, pw.k_max, row_bytes, R * row_bytes))
    pscr = torch.empty(need, dtype=torch.uint8, device=dev)

    def e2e_step():
        bad = 0
        for lo in range(0, B, sub):
            n = min(sub, B - lo)
            vp.schedule_batch_host(run.dc, run.params, h_demand[lo:lo + n], plan=h_plan, scratch=sscr, used_only=used_only)
            bad |= int(h_plan.status[:n].max().item())           # the step's result is read on the host
        vp.pack_host(h_pplan, 0, prank, h_idx, pk["experts_per_rank"], h_rows, h_staged, h_map, h_status, pscr,
                     device=local_rank)
        return bad | int(h_status.item())

    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    K1 = w.k_max
    h2d = (B * N * N * 8) + (4 + pw.k_max * 16 * 10 + (pw.k_max + 1) * 16 * 8 + T * topk * 4 + T * row_bytes)
    pack_d2h = 4 + R * row_bytes + R * 4
    out = {}
    # the headline end-to-end figure brings back the rows the plans use (vp_schedule_batch_host_used: what a caller that
    # executes the plan needs); the whole-array variant (every idle row too) is timed beside it
    for used_only, key in ((True, None), (False, "whole_arrays")):
        assert e2e_step() == 0
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()                  # synchronous: returns after the results are in host memory
        barrier()
        e2e_ms = reduce_max((time.perf_counter() - t0) * 1e3 / e2e_steps, world)
        if used_only:
            used = run.used_rows_bytes if hasattr(run, "used_rows_bytes") else None
            d2h = (used if used is not None else 0) + B * 16 + pack_d2h
            out = {"value": round(B * world / (e2e_ms / 1e3), 1), "unit": UNIT, "ms_per_step": round(e2e_ms, 3),
                   "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps, "host_sub_batch": sub,
                   "api": "vp_schedule_batch_host_used + vp_pack_host (plan rows below n_steps only)"}
        else:
            d2h = (B * (4 + K1 * 4 + K1 * N * 12 + 2 * (K1 + 1) * N * 8 + 8 + 4)) + pack_d2h
            out[key] = {"value": round(B * world / (e2e_ms / 1e3), 1), "ms_per_step": round(e2e_ms, 3), "d2h_bytes_per_step": int(d2h),
                        "api": "vp_schedule_batch_host + vp_pack_host (every element of the plan arrays)"}
    return out


def finish(args, world, run, sched, pk, T, topk, R, pack_bytes, copy_bytes, stats, clocks, launches, sched_per_step,
           sched_per_launch, n_sched, index_ms, copy_ms, n_copy, ms_per_step, value, e2e, extras, tools):
    peaks = load_peaks()
    counters = load_counters()
    cat, w, B, N = run.cat, run.w, run.B, run.N
    copy_avg = copy_ms / max(n_copy, 1)
    index_avg = index_ms / max(n_copy, 1)
    pack_gbs = copy_bytes / (copy_avg * 1e-3) / 1e9
    ops = sched_ops(cat, stats, w.n_start)
    sm_mhz = clocks.get("sm_mhz") or peaks["sm_max_mhz"]
    p_now = extras.get("peaks") or {}
    int_peak = p_now.get("int32_add_min_tops")
    sched_tops = ops / (sched_per_step * 1e-3) / 1e12
    pack_counters = (counters.get("pack_copy_bulk_kernel") or {}) if args.pack_tokens == 16384 else {}
    roof_pack = dict(kernel="pack_copy_bulk_kernel", bound="hbm", achieved=round(pack_gbs, 1), peak=peaks["hbm_gbs"],
                     unit="GB/s", frac=round(pack_gbs / peaks["hbm_gbs"], 4), traffic=pack_counters.get("dram_bytes_per_launch"),
                     peak_source=peaks["source"] + " copy peak (MEASURED_PEAKS.json)", ms_per_launch=round(copy_avg, 4),
                     algorithmic_bytes_per_launch=copy_bytes,
                     frac_of_nominal_8tbs=round(pack_gbs / 8000.0, 4),
                     whole_call_gb_per_s=round(pack_bytes / ((copy_avg + index_avg) * 1e-3) / 1e9, 1),
                     whole_call_frac=round(pack_bytes / ((copy_avg + index_avg) * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                     write_only_peak_gbs=p_now.get("write_only_gbs"))
    key = f"config{args.sched_config}"
    sc = (counters.get("scheduler") or {}).get(key) or {}
    calls = run.calls
    roof_sched = dict(kernel={"warp per matrix": "vp_schedule_warp_kernel", "CTA per matrix": "vp_schedule_kernel"}.get(
                          run.launch.get("kernel"), "vp_schedule_big_kernel"),
                      launch=run.launch, bound="alu", achieved=round(sched_tops, 4), peak=int_peak,
                      unit="Tops/s (integer add/min, algorithmic)",
                      frac=round(sched_tops / int_peak, 5) if int_peak else None,
                      traffic=int(sc["dram_bytes_per_matrix"] * B / calls) if sc.get("dram_bytes_per_matrix") else None,
                      peak_source="measured in this run: vp_microbench kind 0 (32-bit add + min, all warp slots busy)",
                      ms_per_launch=round(sched_per_launch, 4), launches_per_step=calls,
                      algorithmic_ops_per_launch=int(ops / calls))
    roof_sched.update(issue_fraction(counters, key, stats["activations"], sched_per_step, sm_mhz))
    dominant, other = (roof_pack, roof_sched) if copy_avg >= sched_per_step else (roof_sched, roof_pack)
    act = stats["activations"]
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": workload_string(args, sched, pk),
                   "value_is": "matrices of the scheduler batch per second of whole step (all sub-batches + one pack)",
                   "batch_per_gpu": B, "sub_batch": run.sub, "parallelism": f"replicas x{world}, no collective",
                   "l2": "inputs larger than L2: %.2f GB of demand per step, and each step's pack streams %.2f GB"
                         % (B * N * N * 8 / 1e9, pack_bytes / 1e9)},
        "sched": {"matrices_per_s": round(B / (sched_per_step * 1e-3), 1), "ms": round(sched_per_step, 4),
                  "activations_per_batch": act, "us_per_activation_amortized": round(sched_per_step * 1e3 / max(act, 1), 4),
                  "activations_per_s": round(act / (sched_per_step * 1e-3), 1)},
        "pack": {"gb_per_s": round(pack_gbs, 1), "copy_ms": round(copy_avg, 4), "index_ms": round(index_avg, 4),
                 "gb_per_s_incl_index": round(pack_bytes / ((copy_avg + index_avg) * 1e-3) / 1e9, 1)},
        "roofline": dominant, "roofline_other": other,
        "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
    }
    line.update(extras)
    if tools:
        line["next_rows"] = tools
    line["cpu_baseline"] = cpu_baseline(args, sched, pk, budget_s=20.0) if world == 1 and not args.no_cpu_baseline else None
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------

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


def oracle_sample(sched, limit: int):
    """The bounded sample the oracle schedules per step: the whole batch when it is small, else ``limit`` matrices
    spread evenly over the seeded batch (so that every class of the recipe is in it).  Returns (matrices, note)."""
    import numpy as np
    D = sched["demand"].cpu().numpy()
    B = D.shape[0]
    if B <= limit:
        return D, B, f"all {B} matrices"
    pick = np.linspace(0, B - 1, limit).astype(np.int64)
    return np.ascontiguousarray(D[pick]), limit, f"{limit} of the {B} matrices (evenly spaced), scaled to {B}"


def _oracle_sched(oc, D, params, threads):
    """Schedules the sample on ``threads`` host threads (interleaved split: equal mixes of long and short matrices)."""
    import numpy as np
    n = D.shape[0]
    order = np.concatenate([np.arange(t, n, threads) for t in range(threads)]) if threads > 1 else np.arange(n)
    t0 = time.perf_counter()
    oc.schedule_batch(np.ascontiguousarray(D[order]), params, threads=threads)
    return time.perf_counter() - t0


def _oracle_pack(poc, pk, plan_one):
    import numpy as np
    rows, R = pk["_rows_np"], pk["_R"]
    if pk.get("_staged") is None:
        pk["_staged"] = np.zeros((R, rows.shape[1] * rows.itemsize), np.uint8)
    t0 = time.perf_counter()
    poc.pack(plan_one, pk["rank"], pk["_idx_np"], pk["experts_per_rank"], rows, R, staged=pk["_staged"])
    return time.perf_counter() - t0


def cpu_baseline(args, sched, pk, budget_s: float) -> dict:
    """The oracle as it stands, timed on this machine's host cores on a bounded sample of the same workload."""
    cores = os.cpu_count() or 1
    oc, poc, plan_one = _oracle_setup(sched, pk)
    B = sched["demand"].shape[0]
    D, n, note = oracle_sample(sched, args.oracle_sample)
    t_all = _oracle_sched(oc, D, sched["params"], cores)
    n1 = max(1, min(n, n // cores if t_all > 1.0 else n))        # the one-thread figure on a smaller slice
    t_one = _oracle_sched(oc, D[:n1], sched["params"], 1)
    t_pack = _oracle_pack(poc, pk, plan_one)
    sched_s = t_all * B / n
    step_s = sched_s + t_pack
    pack_bytes = pk["_rows_np"].nbytes + pk["_R"] * pk["row_bytes"]
    return {"value": round(B / step_s, 2), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"scheduler: {note}, over {cores} threads; pack: the whole pack on 1 thread",
            "sched_matrices_per_s": round(n / t_all, 2),
            "sched_matrices_per_s_one_thread": round(n1 / t_one, 3), "one_thread_sample": f"first {n1} matrices of the sample",
            "pack_gb_per_s_one_thread": round(pack_bytes / t_pack / 1e9, 3)}


def run_reference(args):
    rank, _, world = _dist_env()
    if rank != 0:
        return
    sched, pk = build_workload(args, "cpu" if not _has_cuda() else "cuda")
    sched["demand"] = sched["demand"].cpu()
    cores = os.cpu_count() or 1
    oc, poc, plan_one = _oracle_setup(sched, pk)
    B = sched["demand"].shape[0]
    D, n, note = oracle_sample(sched, args.oracle_sample)

    def step():
        return _oracle_sched(oc, D, sched["params"], cores), _oracle_pack(poc, pk, plan_one)

    for _ in range(args.warmup):
        step()
    ts = tp = 0.0
    for _ in range(args.steps):
        a, b = step()
        ts += a; tp += b
    sched_s = ts / args.steps * B / n                            # the sample's time scaled to the whole batch
    ms_scaled = (sched_s + tp / args.steps) * 1e3
    ms_measured = (ts + tp) / args.steps * 1e3                   # what one step of this run really took (the sample + the pack)
    value = B / (ms_scaled / 1e3)
    sample = f"every step: scheduler on {note}, over {cores} threads; the whole pack on 1 thread"
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_measured, 3),
            "ms_per_step_scaled_to_batch": round(ms_scaled, 3), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": workload_string(args, sched, pk)},
            "cpu_baseline": {"value": round(value, 2), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": round(value, 2), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_quality(args):
    """Plan-quality report (`--quality`): Eq. (2) over a grid of (lambda, K_target) on config 2's 256 matrices
    (vp_sweep_plan_time), the same with the two-node node-template catalog (15 shapes / 20 families) in place of
    the complete one (89 / 152), and the ratio to the link-load lower bound on a sample (the bound is oracle-side
    Python, test infrastructure, so the sample is small)."""
    import numpy as np
    import torch
    import oracle
    import paper_2609_34340_b200 as vp
    from paper_2609_34340_b200.build import build
    from workloads.configs import build_config
    from workloads.topology import node_template_catalog, tree_topology
    build()
    dev = "cuda:0"
    c = build_config(2, device=dev)
    w = c["params"]
    D = c["demand"].to(dev).contiguous()
    N = c["catalog"].topology.N
    lambdas, k_targets = [0, 2000, 8000, 32000], [N, 2 * N, 3 * N, 4 * N]
    cats = {"complete 89/152": c["catalog"], "node-template 15/20": node_template_catalog(tree_topology(2))}
    res = {}
    for name, cat in cats.items():
        dc = vp.load_catalog(cat.topology.blob(), cat.blob(), device=0)
        T, K, st = vp.sweep_plan_time(dc, vp_params(vp, w), D, lambdas, k_targets)
        torch.cuda.synchronize()
        assert int(st.max().item()) == 0
        res[name] = (T.cpu().numpy().astype(np.float64) / dc.rate_lcm, K.cpu().numpy())
    Tc, Kc = res["complete 89/152"]
    Tt, Kt = res["node-template 15/20"]
    oc = oracle.OracleCatalog(c["catalog"].topology.blob(), c["catalog"].blob())
    sample = list(range(0, D.shape[0], 8))
    lb = np.array([float(oc.lower_bound(c["demand"][b].numpy())) for b in sample])
    out = {"workload": "config 2: 256 MoE demand matrices N=16", "lambda_ns": lambdas, "k_target": k_targets,
           "mean_T_us_complete": np.round(Tc.mean(axis=2) / 1e3, 1).tolist(),
           "mean_activations_complete": np.round(Kc.mean(axis=2), 1).tolist(),
           "mean_T_us_template": np.round(Tt.mean(axis=2) / 1e3, 1).tolist(),
           "template_over_complete_mean_ratio": np.round((Tt / Tc).mean(axis=2), 4).tolist(),
           "template_over_complete_max_ratio": np.round((Tt / Tc).max(axis=2), 4).tolist(),
           "T_over_lower_bound_at_lambda0": {"sample": f"{len(sample)} matrices (every 8th)",
                                             "mean_per_k_target": np.round((Tc[0][:, sample] / lb).mean(axis=1), 4).tolist()}}
    print(json.dumps({"plan_quality": out}))


def _has_cuda() -> bool:
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sched-config", type=int, default=4, choices=[1, 2, 3, 4])
    ap.add_argument("--sub-batch", type=int, default=2048,
                    help="matrices per vp_schedule_batch call (the plan buffers are reused); the batch when smaller")
    ap.add_argument("--batch", type=int, default=None, help="truncate the scheduler batch (tests)")
    ap.add_argument("--sched-repeat", type=int, default=1,
                    help="schedule the batch this many times over in one call (a batch beyond one wave; not the default benchmark)")
    ap.add_argument("--token-scale", type=float, default=1.0, help="scale token counts (tests)")
    ap.add_argument("--pack-tokens", type=int, default=16384, help="tokens of the packed rank (tests)")
    ap.add_argument("--oracle-sample", type=int, default=64,
                    help="matrices the CPU oracle schedules per step when the batch is larger (reference arm, cpu_baseline)")
    ap.add_argument("--min-warmup-s", type=float, default=1.0,
                    help="keep warming up (beyond --warmup steps) until this many seconds have passed, so that "
                         "clocks settle and nvidia-smi has samples under load")
    ap.add_argument("--e2e-steps", type=int, default=2, help="steps of the host-buffer leg (each moves the whole plan over PCIe)")
    ap.add_argument("--quality", action="store_true", help="print the plan-quality report (Eq. 2 sweep, template vs complete catalog) and exit")
    ap.add_argument("--tools", action="store_true", help="also time the kernels around the scheduler (unpack, plan time, demand rows)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the CPU oracle leg (profiling runs)")
    ap.add_argument("--no-extras", action="store_true", help="skip the peak probes and the other scheduler configs (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.quality:
        run_quality(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
