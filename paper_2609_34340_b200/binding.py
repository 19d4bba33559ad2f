"""ctypes binding of ``libvariopath.so``; names follow the C ABI (``vp_*`` without the prefix).

PyTorch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libvariopath.so")

E_BAD_ARG, E_BAD_CATALOG, E_NOMEM, E_CUDA, E_WORKSPACE, E_UNSUPPORTED = -1, -2, -3, -4, -5, -6
ST_NEGATIVE, ST_OVERFLOW_RISK, ST_DIAG_NONZERO, ST_NOT_GRANULE = 1, 2, 4, 8
ST_BAD_TAU, ST_UNCOVERED, ST_NO_PROGRESS, ST_STEP_LIMIT = 16, 32, 64, 128
ST_PACK_MISMATCH, ST_PACK_CAPACITY = 256, 512
ST_EXCHANGE_TIMEOUT = 2048
ST_INTERNAL_TIMEOUT = 1 << 30    # a row-copy kernel gave up a bounded wait: the output buffer is incomplete


class VpError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {_strerror(code)} ({code})")


class _Info(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("N", "G", "g", "groups_per_node", "n_resources", "n_instances",
                                          "n_shapes", "n_families", "max_nnz", "max_bucket", "covered",
                                          "node_symmetric")] + [("rate_lcm", C.c_int64), ("row_patterns", C.c_int32),
                                                                ("argmax_classes", C.c_int32)]


class _Params(C.Structure):
    _fields_ = [("lambda_ns", C.c_int64), ("granule_bytes", C.c_int64), ("k_target", C.c_int32),
                ("n_start", C.c_int32), ("i_aa", C.c_int32), ("k_max", C.c_int32)]


@dataclass
class SchedParams:
    """Scheduler parameters (``vp_sched_params``); 0 selects the documented default."""
    lambda_ns: int = 8000
    granule_bytes: int = 1
    k_target: int = 0
    n_start: int = 0
    i_aa: int = 0
    k_max: int = 0

    def _c(self, N: int) -> _Params:
        return _Params(int(self.lambda_ns), int(self.granule_bytes), int(self.k_target), int(self.n_start),
                       int(self.i_aa), int(self.k_max) or 8 * N)


_lib = None


def library_path() -> str:
    return _LIB_PATH


def _load():
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_34340_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(_LIB_PATH)
    vp, i32, i64, sz, P = C.c_void_p, C.c_int, C.c_int64, C.c_size_t, C.c_void_p
    lib.vp_load_catalog.argtypes = [P, sz, P, sz, i32, C.POINTER(vp)]
    lib.vp_free_catalog.argtypes = [vp]
    lib.vp_free_catalog.restype = None
    lib.vp_catalog_info.argtypes = [vp, C.POINTER(_Info)]
    lib.vp_catalog_argmax_classes.argtypes = [vp, P, sz, C.POINTER(sz)]
    lib.vp_schedule_workspace_bytes.argtypes = [vp, i32, C.POINTER(_Params)]
    lib.vp_schedule_workspace_bytes.restype = sz
    sched_args = [vp, C.POINTER(_Params), P, P, i32] + [P] * 9
    lib.vp_schedule_batch.argtypes = sched_args + [P, sz, P]
    lib.vp_schedule_host_scratch_bytes.argtypes = [vp, i32, C.POINTER(_Params)]
    lib.vp_schedule_host_scratch_bytes.restype = sz
    lib.vp_schedule_batch_host.argtypes = sched_args + [P, sz, P]
    lib.vp_schedule_batch_host_used.argtypes = sched_args + [P, sz, P]
    lib.vp_pack_workspace_bytes.argtypes = [i32, i32, i32, i32]
    lib.vp_pack_workspace_bytes.restype = sz
    pack_args = [P, P, P, P, i32, i32, i32, P, i32, i32, i32, P, i64, P, i64, P, P]
    lib.vp_pack.argtypes = pack_args + [P, sz, P]
    lib.vp_pack_static.argtypes = pack_args + [P]
    lib.vp_pack_host_scratch_bytes.argtypes = [i32, i32, i32, i32, i64, i64]
    lib.vp_pack_host_scratch_bytes.restype = sz
    lib.vp_pack_host.argtypes = pack_args + [P, sz, P]
    lib.vp_unpack_workspace_bytes.argtypes = [i32, i64, i32, i32]
    lib.vp_unpack_workspace_bytes.restype = sz
    lib.vp_unpack.argtypes = [P, P, P, i32, i32, i32, P, i64, i64, P, i32, P, P, P, P, P, P, sz, P]
    lib.vp_unpack_tokens_workspace_bytes.argtypes = [i32, i32, i32, i32, i64, i32]
    lib.vp_unpack_tokens_workspace_bytes.restype = sz
    lib.vp_unpack_tokens.argtypes = [P, P, P, P, i32, i32, i32, P, i32, i32, i32, P, i64, i64, P, P, P, P, sz, P]
    lib.vp_kernel_launch_count.restype = i64
    lib.vp_build_catalog.argtypes = [P, sz, P, sz, C.POINTER(sz), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.vp_build_template_catalog.argtypes = [P, sz, P, sz, C.POINTER(sz), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.vp_prune_paths.argtypes = [P, sz, P, sz, C.POINTER(sz), C.POINTER(C.c_int32)]
    lib.vp_plan_time.argtypes = [vp, i32, i32, P, P, P, i64, P, P]
    lib.vp_demand_from_routing.argtypes = [P, i32, i32, i32, i32, i32, i32, i64, P, P, P]
    lib.vp_sweep_workspace_bytes.argtypes = [vp, i32, C.POINTER(_Params)]
    lib.vp_sweep_workspace_bytes.restype = sz
    lib.vp_sweep_plan_time.argtypes = [vp, C.POINTER(_Params), P, i32, P, i32, P, i32, P, P, P, P, sz, P]
    lib.vp_schedule_read_stats.argtypes = [P, P, P]
    lib.vp_schedule_launch_info.argtypes = [vp, i32, C.POINTER(_Params), P]
    lib.vp_microbench.argtypes = [i32, i32, P, C.POINTER(i64), P]
    lib.vp_exchange_put.argtypes = [P, P, P, P, i32, i32, i32, P, P, P, P, P, P]
    lib.vp_exchange_wait.argtypes = [P, P, i32, i32, i32, P, C.c_uint64, C.c_uint32, P, P]
    lib.vp_memset_probe.argtypes = [P, sz, P]
    lib.vp_profile_enable.argtypes = [i32]
    lib.vp_profile_read.argtypes = [i32, C.POINTER(C.c_double), C.POINTER(i64)]
    lib.vp_strerror.argtypes = [i32]
    lib.vp_strerror.restype = C.c_char_p
    _lib = lib
    return lib


def _strerror(code: int) -> str:
    return _load().vp_strerror(int(code)).decode()


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise VpError(rc, what)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def kernel_launch_count() -> int:
    return int(_load().vp_kernel_launch_count())


def schedule_launch_info(catalog: "Catalog", B: int, params: "SchedParams") -> dict:
    """``vp_schedule_launch_info``: which kernel and launch shape a batch of ``B`` matrices gets."""
    out = (C.c_int32 * 4)()
    p = params._c(catalog.N)
    _check(_load().vp_schedule_launch_info(catalog._h, int(B), C.byref(p), out), "vp_schedule_launch_info")
    kernel = {0: "CTA per matrix", 1: "warp per matrix", 2: "CTA per matrix, 16-bit credits"}[int(out[0])]
    return dict(kernel=kernel, ctas=int(out[1]), threads=int(out[2]), smem=int(out[3]))


def schedule_read_stats(workspace: torch.Tensor, stream=None) -> dict:
    """``vp_schedule_read_stats``: work counters of the last batch scheduled with ``workspace``."""
    out = (C.c_uint64 * 3)()
    _check(_load().vp_schedule_read_stats(_ptr(workspace), _stream(stream), out), "vp_schedule_read_stats")
    return dict(activations=int(out[0]), tasks=int(out[1]), sweeps=int(out[2]))


def exchange_put(plan: "Plan", b: int, rank: int, staged: torch.Tensor, recv_bufs: torch.Tensor, recv_capacity: torch.Tensor,
                 arrived: Optional[torch.Tensor], status: torch.Tensor, stream=None) -> None:
    """``vp_exchange_put`` for matrix ``b`` of a device plan: ``recv_bufs`` / ``arrived`` are int64 device tensors ``[N]`` holding
    device addresses (``tensor.data_ptr()`` of every rank's receive buffer / counter), ``recv_capacity`` int64 ``[N]`` bytes."""
    N = plan.lane_dst.shape[2]
    _check(_load().vp_exchange_put(_ptr(plan.n_steps[b:]), _ptr(plan.lane_dst[b]), _ptr(plan.send_off[b]), _ptr(plan.recv_off[b]),
                                   int(N), int(rank), int(plan.k_max), _ptr(staged), _ptr(recv_bufs), _ptr(recv_capacity),
                                   _ptr(arrived), _ptr(status), _stream(stream)), "vp_exchange_put")


def exchange_wait(plan: "Plan", b: int, rank: int, counter: torch.Tensor, base: int, max_polls: int, status: torch.Tensor,
                  stream=None) -> None:
    """``vp_exchange_wait``: bounded wait for rank ``rank``'s arrival counter (an int64/uint64 device tensor of one element)."""
    N = plan.lane_dst.shape[2]
    _check(_load().vp_exchange_wait(_ptr(plan.n_steps[b:]), _ptr(plan.recv_off[b]), int(N), int(rank), int(plan.k_max),
                                    _ptr(counter), int(base), int(max_polls), _ptr(status), _stream(stream)), "vp_exchange_wait")


def gather_exchange_tables(recv_ptr: int, counter_ptr: int, capacity_bytes: int, device=None):
    """The three tables ``vp_exchange_put`` takes, assembled over ``torch.distributed``: every rank contributes the address
    of its receive buffer and of its arrival counter (addresses that are valid on the other ranks' GPUs: peer-mapped or
    symmetric memory) and its buffer size; every rank gets all of them, indexed by rank.  Returns int64 tensors
    (recv_bufs ``[world]``, arrived ``[world]``, recv_capacity ``[world]``) on ``device`` (default: CPU, for gloo groups)."""
    import torch.distributed as dist
    world = dist.get_world_size()
    on = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")
    mine = torch.tensor([int(recv_ptr), int(counter_ptr), int(capacity_bytes)], dtype=torch.int64, device=on)
    every = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(every, mine)
    table = torch.stack(every).to(device if device is not None else "cpu")
    return table[:, 0].contiguous(), table[:, 1].contiguous(), table[:, 2].contiguous()


def microbench(kind: int, iters: int, sink: torch.Tensor, stream=None) -> int:
    """``vp_microbench``: launches peak-rate probe ``kind`` on the current stream; returns the units (integer
    operations or bytes) one launch performs.  ``sink`` is an 8-byte device tensor."""
    units = C.c_int64(0)
    _check(_load().vp_microbench(int(kind), int(iters), _ptr(sink), C.byref(units), _stream(stream)), "vp_microbench")
    return int(units.value)


def memset_probe(buf: torch.Tensor, stream=None) -> int:
    """``vp_memset_probe``: one ``cudaMemsetAsync`` over ``buf``; returns the bytes written."""
    n = buf.numel() * buf.element_size()
    _check(_load().vp_memset_probe(_ptr(buf), n, _stream(stream)), "vp_memset_probe")
    return n


def profile_enable(on: bool) -> None:
    _check(_load().vp_profile_enable(1 if on else 0), "vp_profile_enable")


def profile_read(kind: int):
    """``vp_profile_read``: (total device ms, launches) of kind 0 schedule / 1 pack index / 2 pack copy."""
    ms, n = C.c_double(0), C.c_int64(0)
    _check(_load().vp_profile_read(int(kind), C.byref(ms), C.byref(n)), "vp_profile_read")
    return float(ms.value), int(n.value)


class Catalog:
    """Handle of a catalog loaded on one device (``vp_catalog``)."""

    def __init__(self, handle: int, device: int):
        self._h = C.c_void_p(handle)
        self.device = device
        info = _Info()
        _check(_load().vp_catalog_info(self._h, C.byref(info)), "vp_catalog_info")
        for name, _ in _Info._fields_:
            setattr(self, name, int(getattr(info, name)))

    def free(self) -> None:
        if self._h:
            _load().vp_free_catalog(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def load_catalog(topology: bytes, channels: bytes, device: int = 0) -> Catalog:
    """``vp_load_catalog``: validate the blobs (Eq. 3, Eq. 4) and upload the device image."""
    h = C.c_void_p()
    topology, channels = bytes(topology), bytes(channels)
    _check(_load().vp_load_catalog(topology, len(topology), channels, len(channels), int(device), C.byref(h)),
           "vp_load_catalog")
    return Catalog(h.value, int(device))


def catalog_argmax_classes(catalog: Catalog):
    """``vp_catalog_argmax_classes``: the class decomposition of the arg-max as a numpy uint32 array (empty if none)."""
    import numpy as np
    need = C.c_size_t(0)
    _check(_load().vp_catalog_argmax_classes(catalog._h, None, 0, C.byref(need)), "vp_catalog_argmax_classes")
    out = np.zeros(need.value, dtype=np.uint32)
    if need.value:
        _check(_load().vp_catalog_argmax_classes(catalog._h, out.ctypes.data_as(C.c_void_p), need.value, C.byref(need)),
               "vp_catalog_argmax_classes")
    return out


def build_catalog(topology: bytes):
    """``vp_build_catalog`` (Algorithm 1, host code): returns (channels blob, n_shapes, n_families)."""
    topology = bytes(topology)
    need, ns, nf = C.c_size_t(0), C.c_int32(0), C.c_int32(0)
    _check(_load().vp_build_catalog(topology, len(topology), None, 0, C.byref(need), C.byref(ns), C.byref(nf)),
           "vp_build_catalog")
    buf = C.create_string_buffer(need.value)
    _check(_load().vp_build_catalog(topology, len(topology), buf, need.value, C.byref(need), C.byref(ns), C.byref(nf)),
           "vp_build_catalog")
    return buf.raw[:need.value], int(ns.value), int(nf.value)


def schedule_workspace_bytes(catalog: Catalog, B: int, params: SchedParams) -> int:
    p = params._c(catalog.N)
    return int(_load().vp_schedule_workspace_bytes(catalog._h, int(B), C.byref(p)))


@dataclass
class Plan:
    """Output arrays of ``vp_schedule_batch`` (device or host tensors, layouts as in the header)."""
    n_steps: torch.Tensor
    chan_id: torch.Tensor
    lane_dst: torch.Tensor
    lane_inst: torch.Tensor
    lane_bytes: torch.Tensor
    send_off: torch.Tensor
    recv_off: torch.Tensor
    tau_ns: torch.Tensor
    status: torch.Tensor
    k_max: int

    @staticmethod
    def empty(B: int, N: int, k_max: int, device, pin: bool = False) -> "Plan":
        kw = dict(device=device, pin_memory=pin) if pin else dict(device=device)
        return Plan(
            n_steps=torch.empty(B, dtype=torch.int32, **kw),
            chan_id=torch.empty((B, k_max), dtype=torch.int32, **kw),
            lane_dst=torch.empty((B, k_max, N), dtype=torch.int16, **kw),
            lane_inst=torch.empty((B, k_max, N), dtype=torch.uint16, **kw),
            lane_bytes=torch.empty((B, k_max, N), dtype=torch.int64, **kw),
            send_off=torch.empty((B, k_max + 1, N), dtype=torch.int64, **kw),
            recv_off=torch.empty((B, k_max + 1, N), dtype=torch.int64, **kw),
            tau_ns=torch.empty(B, dtype=torch.int64, **kw),
            status=torch.empty(B, dtype=torch.int32, **kw),
            k_max=k_max)

    def cpu(self) -> dict:
        """Numpy copies keyed like the oracle's output."""
        out = {k: getattr(self, k).cpu().numpy() for k in ("n_steps", "chan_id", "lane_dst", "lane_bytes",
                                                             "send_off", "recv_off", "tau_ns", "status")}
        out["lane_inst"] = self.lane_inst.cpu().view(torch.int16).numpy().view("uint16")
        out["k_max"] = self.k_max
        return out


def _sched_call(fn, catalog, p, demand, tau_ns_in, B, plan, scratch, stream):
    return fn(catalog._h, C.byref(p), _ptr(demand), _ptr(tau_ns_in), int(B), _ptr(plan.n_steps),
              _ptr(plan.chan_id), _ptr(plan.lane_dst), _ptr(plan.lane_inst), _ptr(plan.lane_bytes),
              _ptr(plan.send_off), _ptr(plan.recv_off), _ptr(plan.tau_ns), _ptr(plan.status),
              _ptr(scratch), scratch.numel(), _stream(stream))


def schedule_batch(catalog: Catalog, params: SchedParams, demand: torch.Tensor,
                   tau_ns_in: Optional[torch.Tensor] = None, plan: Optional[Plan] = None,
                   workspace: Optional[torch.Tensor] = None, stream=None) -> Plan:
    """``vp_schedule_batch`` on device tensors: ``demand`` is ``[B,N,N]`` int64 on the catalog's device."""
    assert demand.is_cuda and demand.dtype == torch.int64 and demand.is_contiguous()
    B, N = demand.shape[0], catalog.N
    assert demand.shape == (B, N, N)
    p = params._c(N)
    if plan is None:
        plan = Plan.empty(B, N, p.k_max, demand.device)
    if workspace is None:
        workspace = torch.empty(schedule_workspace_bytes(catalog, B, params), dtype=torch.uint8, device=demand.device)
    _check(_sched_call(_load().vp_schedule_batch, catalog, p, demand, tau_ns_in, B, plan, workspace, stream),
           "vp_schedule_batch")
    return plan


def schedule_batch_host(catalog: Catalog, params: SchedParams, demand: torch.Tensor,
                        tau_ns_in: Optional[torch.Tensor] = None, plan: Optional[Plan] = None,
                        scratch: Optional[torch.Tensor] = None, stream=None, used_only: bool = False) -> Plan:
    """``vp_schedule_batch_host``: host tensors in and out (pinned memory recommended).  ``used_only`` selects
    ``vp_schedule_batch_host_used``: only the rows below each matrix's ``n_steps`` come back."""
    assert not demand.is_cuda and demand.dtype == torch.int64 and demand.is_contiguous()
    B, N = demand.shape[0], catalog.N
    p = params._c(N)
    if plan is None:
        plan = Plan.empty(B, N, p.k_max, "cpu", pin=True)
    if scratch is None:
        need = int(_load().vp_schedule_host_scratch_bytes(catalog._h, B, C.byref(p)))
        scratch = torch.empty(need, dtype=torch.uint8, device=f"cuda:{catalog.device}")
    fn = _load().vp_schedule_batch_host_used if used_only else _load().vp_schedule_batch_host
    _check(_sched_call(fn, catalog, p, demand, tau_ns_in, B, plan, scratch, stream), "vp_schedule_batch_host")
    return plan


def plan_time(catalog: Catalog, plan: Plan, lambda_ns: int, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """``vp_plan_time``: ``rate_lcm x`` modeled completion time (Eq. 2) of every plan, int64 ``[B]`` on device."""
    B = plan.n_steps.shape[0]
    if out is None:
        out = torch.empty(B, dtype=torch.int64, device=plan.n_steps.device)
    _check(_load().vp_plan_time(catalog._h, int(B), int(plan.k_max), _ptr(plan.n_steps), _ptr(plan.lane_inst),
                                _ptr(plan.lane_bytes), int(lambda_ns), _ptr(out), _stream(stream)), "vp_plan_time")
    return out


def sweep_plan_time(catalog: Catalog, params: SchedParams, demand: torch.Tensor, lambdas, k_targets, stream=None):
    """``vp_sweep_plan_time``: returns (time_xw int64 ``[n_lambda, n_k, B]``, n_steps int32, status int32), all on device."""
    assert demand.is_cuda and demand.dtype == torch.int64 and demand.is_contiguous()
    B, N = demand.shape[0], catalog.N
    p = params._c(N)
    lam = (C.c_int64 * len(lambdas))(*[int(x) for x in lambdas])
    kt = (C.c_int32 * len(k_targets))(*[int(x) for x in k_targets])
    shape = (len(lambdas), len(k_targets), B)
    out = torch.empty(shape, dtype=torch.int64, device=demand.device)
    n_steps = torch.empty(shape, dtype=torch.int32, device=demand.device)
    status = torch.empty(shape, dtype=torch.int32, device=demand.device)
    need = int(_load().vp_sweep_workspace_bytes(catalog._h, B, C.byref(p)))
    ws = torch.empty(need, dtype=torch.uint8, device=demand.device)
    _check(_load().vp_sweep_plan_time(catalog._h, C.byref(p), _ptr(demand), B, lam, len(lambdas), kt, len(k_targets), _ptr(out),
                                      _ptr(n_steps), _ptr(status), _ptr(ws), need, _stream(stream)), "vp_sweep_plan_time")
    return out, n_steps, status


def demand_from_routing(expert_idx: torch.Tensor, experts_per_rank: int, N: int, row_bytes: int, src0: int = 0,
                        out: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None, stream=None):
    """``vp_demand_from_routing``: ``expert_idx`` is ``[n_src, T, topk]`` int32 on device; returns
    (``[n_src, N]`` int64 demand rows, status int32[1])."""
    assert expert_idx.is_cuda and expert_idx.dtype == torch.int32 and expert_idx.is_contiguous() and expert_idx.dim() == 3
    n_src, T, topk = expert_idx.shape
    if out is None:
        out = torch.empty((n_src, N), dtype=torch.int64, device=expert_idx.device)
    if status is None:
        status = torch.empty(1, dtype=torch.int32, device=expert_idx.device)
    _check(_load().vp_demand_from_routing(_ptr(expert_idx), int(n_src), int(T), int(topk), int(experts_per_rank), int(N),
                                          int(src0), int(row_bytes), _ptr(out), _ptr(status), _stream(stream)),
           "vp_demand_from_routing")
    return out, status


def pack_workspace_bytes(N: int, T: int, topk: int, k_max: int) -> int:
    return int(_load().vp_pack_workspace_bytes(int(N), int(T), int(topk), int(k_max)))


def _pack_call(fn, plan, b, N, rank, expert_idx, experts_per_rank, rows, row_bytes, staged, src_map, status,
               scratch, stream):
    T, topk = expert_idx.shape
    return fn(_ptr(plan.n_steps[b:b + 1]), _ptr(plan.lane_dst[b]), _ptr(plan.lane_bytes[b]), _ptr(plan.send_off[b]),
              int(N), int(rank), int(plan.k_max), _ptr(expert_idx), int(T), int(topk), int(experts_per_rank),
              _ptr(rows), int(row_bytes), _ptr(staged), staged.numel() * staged.element_size(), _ptr(src_map),
              _ptr(status), _ptr(scratch), scratch.numel(), _stream(stream))


def pack(plan: Plan, b: int, rank: int, expert_idx: torch.Tensor, experts_per_rank: int, rows: torch.Tensor,
         staged: torch.Tensor, src_map: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
         workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """``vp_pack`` for matrix ``b`` of a device plan.  ``rows`` is ``[T, H]`` (any dtype), ``staged`` a
    pre-allocated device buffer; returns the device status tensor (int32[1])."""
    N = plan.lane_dst.shape[2]
    assert expert_idx.is_cuda and expert_idx.dtype == torch.int32 and expert_idx.is_contiguous()
    assert rows.is_cuda and rows.is_contiguous() and staged.is_cuda and staged.is_contiguous()
    T, topk = expert_idx.shape
    row_bytes = rows.shape[1] * rows.element_size()
    if status is None:
        status = torch.empty(1, dtype=torch.int32, device=rows.device)
    if workspace is None:
        workspace = torch.empty(pack_workspace_bytes(N, T, topk, plan.k_max), dtype=torch.uint8, device=rows.device)
    _check(_pack_call(_load().vp_pack, plan, b, N, rank, expert_idx, experts_per_rank, rows, row_bytes, staged,
                      src_map, status, workspace, stream), "vp_pack")
    return status


PACK_STATIC_SCRATCH_BYTES = 4 * 1024 * 1024


def pack_static(plan: Plan, b: int, rank: int, expert_idx: torch.Tensor, experts_per_rank: int, rows: torch.Tensor,
                staged: torch.Tensor, src_map: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                stream=None) -> torch.Tensor:
    """``vp_pack_static``: the pack for callers that cannot hand over scratch memory (they run inside an
    engine's step, own no allocator and must not call cudaMalloc).  Same results as :func:`pack`; the library
    uses its own fixed 4 MiB device block instead of a workspace, so the problem has to fit it
    (``VpError`` with ``E_WORKSPACE`` otherwise) and calls that may overlap on the GPU must be ordered.
    ``status`` must be passed in by such callers; it is allocated here only when omitted."""
    N = plan.lane_dst.shape[2]
    assert expert_idx.is_cuda and expert_idx.dtype == torch.int32 and expert_idx.is_contiguous()
    assert rows.is_cuda and rows.is_contiguous() and staged.is_cuda and staged.is_contiguous()
    T, topk = expert_idx.shape
    row_bytes = rows.shape[1] * rows.element_size()
    if status is None:
        status = torch.empty(1, dtype=torch.int32, device=rows.device)
    rc = _load().vp_pack_static(_ptr(plan.n_steps[b:b + 1]), _ptr(plan.lane_dst[b]), _ptr(plan.lane_bytes[b]),
                                _ptr(plan.send_off[b]), int(N), int(rank), int(plan.k_max), _ptr(expert_idx), int(T),
                                int(topk), int(experts_per_rank), _ptr(rows), int(row_bytes), _ptr(staged),
                                staged.numel() * staged.element_size(), _ptr(src_map), _ptr(status), _stream(stream))
    _check(rc, "vp_pack_static")
    return status


def pack_host(plan: Plan, b: int, rank: int, expert_idx: torch.Tensor, experts_per_rank: int, rows: torch.Tensor,
              staged: torch.Tensor, src_map: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
              scratch: Optional[torch.Tensor] = None, device: int = 0, stream=None) -> torch.Tensor:
    """``vp_pack_host``: every array (plan included) in host memory."""
    N = plan.lane_dst.shape[2]
    assert not rows.is_cuda and not staged.is_cuda and not plan.lane_dst.is_cuda
    T, topk = expert_idx.shape
    row_bytes = rows.shape[1] * rows.element_size()
    if status is None:
        status = torch.zeros(1, dtype=torch.int32)
    if scratch is None:
        need = int(_load().vp_pack_host_scratch_bytes(N, T, topk, plan.k_max, row_bytes,
                                                      staged.numel() * staged.element_size()))
        scratch = torch.empty(need, dtype=torch.uint8, device=f"cuda:{device}")
    _check(_pack_call(_load().vp_pack_host, plan, b, N, rank, expert_idx, experts_per_rank, rows, row_bytes, staged,
                      src_map, status, scratch, stream), "vp_pack_host")
    return status


def unpack_workspace_bytes(N: int, capacity_rows: int, experts_per_rank: int, k_max: int) -> int:
    return int(_load().vp_unpack_workspace_bytes(int(N), int(capacity_rows), int(experts_per_rank), int(k_max)))


def unpack(plan: Plan, b: int, rank: int, recv: torch.Tensor, recv_expert: torch.Tensor, experts_per_rank: int,
           out: torch.Tensor, expert_off: Optional[torch.Tensor] = None, out_src: Optional[torch.Tensor] = None,
           out_map: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
           workspace: Optional[torch.Tensor] = None, stream=None):
    """``vp_unpack`` for matrix ``b`` of a device plan: ``recv`` ``[capacity_rows, H]`` is rank ``rank``'s
    receive buffer, ``recv_expert`` the local expert of each received row, ``out`` ``[capacity_rows, H]`` the
    expert-major output.  Returns ``(expert_off, status)`` (device int32 ``[experts_per_rank + 1]`` and ``[1]``)."""
    N = plan.lane_dst.shape[2]
    assert recv.is_cuda and recv.is_contiguous() and recv.dim() == 2 and out.is_cuda and out.is_contiguous()
    assert recv_expert.is_cuda and recv_expert.dtype == torch.int32 and recv_expert.is_contiguous()
    cap = recv.shape[0]
    assert recv_expert.numel() >= cap and out.numel() * out.element_size() >= recv.numel() * recv.element_size()
    row_bytes = recv.shape[1] * recv.element_size()
    if expert_off is None:
        expert_off = torch.empty(experts_per_rank + 1, dtype=torch.int32, device=recv.device)
    if status is None:
        status = torch.empty(1, dtype=torch.int32, device=recv.device)
    if workspace is None:
        need = unpack_workspace_bytes(N, cap, experts_per_rank, plan.k_max)
        if need == 0:
            raise VpError(E_UNSUPPORTED, "vp_unpack_workspace_bytes")
        workspace = torch.empty(need, dtype=torch.uint8, device=recv.device)
    rc = _load().vp_unpack(_ptr(plan.n_steps[b:b + 1]), _ptr(plan.lane_dst[b]), _ptr(plan.recv_off[b]), int(N), int(rank),
                           int(plan.k_max), _ptr(recv), int(row_bytes), int(cap), _ptr(recv_expert), int(experts_per_rank),
                           _ptr(out), _ptr(expert_off), _ptr(out_src), _ptr(out_map), _ptr(status), _ptr(workspace),
                           workspace.numel(), _stream(stream))
    _check(rc, "vp_unpack")
    return expert_off, status


def unpack_tokens(plan: Plan, b: int, rank: int, expert_idx: torch.Tensor, experts_per_rank: int, recv: torch.Tensor,
                  out: torch.Tensor, out_map: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                  workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """``vp_unpack_tokens`` for matrix ``b`` of the RETURN call's device plan: ``recv`` ``[capacity_rows, H]`` is rank
    ``rank``'s return receive buffer, ``expert_idx`` ``[T, topk]`` its routing, ``out`` ``[T*topk, H]`` the token
    layout.  Returns the device status tensor (int32[1])."""
    N = plan.lane_dst.shape[2]
    assert expert_idx.is_cuda and expert_idx.dtype == torch.int32 and expert_idx.is_contiguous() and expert_idx.dim() == 2
    assert recv.is_cuda and recv.is_contiguous() and recv.dim() == 2 and out.is_cuda and out.is_contiguous()
    T, topk = expert_idx.shape
    cap = recv.shape[0]
    row_bytes = recv.shape[1] * recv.element_size()
    assert out.numel() * out.element_size() >= T * topk * row_bytes
    if status is None:
        status = torch.empty(1, dtype=torch.int32, device=recv.device)
    if workspace is None:
        need = int(_load().vp_unpack_tokens_workspace_bytes(int(N), int(T), int(topk), int(experts_per_rank), int(cap), int(plan.k_max)))
        if need == 0:
            raise VpError(E_UNSUPPORTED, "vp_unpack_tokens_workspace_bytes")
        workspace = torch.empty(need, dtype=torch.uint8, device=recv.device)
    rc = _load().vp_unpack_tokens(_ptr(plan.n_steps[b:b + 1]), _ptr(plan.lane_dst[b]), _ptr(plan.lane_bytes[b]), _ptr(plan.recv_off[b]),
                                  int(N), int(rank), int(plan.k_max), _ptr(expert_idx), int(T), int(topk), int(experts_per_rank),
                                  _ptr(recv), int(row_bytes), int(cap), _ptr(out), _ptr(out_map), _ptr(status), _ptr(workspace),
                                  workspace.numel(), _stream(stream))
    _check(rc, "vp_unpack_tokens")
    return status


def prune_paths(topology_blob: bytes) -> bytes:
    """``vp_prune_paths``: the topology blob without its dominated path instances (host code, no GPU)."""
    need, kept = C.c_size_t(0), C.c_int32(0)
    lib = _load()
    _check(lib.vp_prune_paths(topology_blob, len(topology_blob), None, 0, C.byref(need), C.byref(kept)), "vp_prune_paths")
    out = C.create_string_buffer(need.value)
    _check(lib.vp_prune_paths(topology_blob, len(topology_blob), out, need.value, C.byref(need), C.byref(kept)), "vp_prune_paths")
    return out.raw[:need.value]


def build_template_catalog(topology_blob: bytes):
    """``vp_build_template_catalog``: (channels blob, shapes, families) of the node-template catalog (host code)."""
    need, ns, nf = C.c_size_t(0), C.c_int32(0), C.c_int32(0)
    lib = _load()
    _check(lib.vp_build_template_catalog(topology_blob, len(topology_blob), None, 0, C.byref(need), C.byref(ns), C.byref(nf)),
           "vp_build_template_catalog")
    out = C.create_string_buffer(need.value)
    _check(lib.vp_build_template_catalog(topology_blob, len(topology_blob), out, need.value, C.byref(need), C.byref(ns), C.byref(nf)),
           "vp_build_template_catalog")
    return out.raw[:need.value], int(ns.value), int(nf.value)
