"""ctypes binding of the C oracle (test infrastructure; see ``vp_oracle.c``)."""
from __future__ import annotations

import ctypes as C
import os
import struct
import subprocess
from concurrent.futures import ThreadPoolExecutor
from fractions import Fraction
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vp_oracle.c")
_LIB = os.path.join(_HERE, "libvp_oracle.so")

ST_NEGATIVE, ST_OVERFLOW, ST_DIAG, ST_GRANULE = 1, 2, 4, 8
ST_BAD_TAU, ST_UNCOVERED, ST_NO_PROGRESS, ST_STEP_LIMIT = 16, 32, 64, 128
ST_PACK_MISMATCH, ST_PACK_CAPACITY = 256, 512

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, no intrinsics)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.vpo_load.restype = C.c_void_p
        _lib.vpo_load.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.POINTER(C.c_int)]
        _lib.vpo_free.argtypes = [C.c_void_p]
        _lib.vpo_info.argtypes = [C.c_void_p, C.c_void_p]
        _lib.vpo_check_catalog.argtypes = [C.c_void_p]
        _lib.vpo_catalog_covers.argtypes = [C.c_void_p]
        _lib.vpo_lanes_feasible.argtypes = [C.c_void_p] * 3
        _lib.vpo_aggregate_bw_x5040.restype = C.c_int64
        _lib.vpo_aggregate_bw_x5040.argtypes = [C.c_void_p] * 3
        _lib.vpo_rate_lcm.restype = C.c_int64
        _lib.vpo_rate_lcm.argtypes = [C.c_void_p]
        _lib.vpo_modeled_time_xW.restype = C.c_int64
        _lib.vpo_modeled_time_xW.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64]
        _lib.vpo_check_plan.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_int64, C.c_int64]
        _lib.vpo_schedule.argtypes = ([C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int,
                                       C.c_int64, C.c_int] + [C.c_void_p] * 9 + [C.c_void_p, C.c_int, C.c_void_p])
        _lib.vpo_schedule_batch.argtypes = ([C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int64,
                                             C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int] + [C.c_void_p] * 9)
        _lib.vpo_demand_from_routing.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                                 C.c_int64, C.c_void_p]
        _lib.vpo_unpack.argtypes = ([C.c_void_p] * 3 + [C.c_int] * 3 + [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int]
                                    + [C.c_void_p] * 4)
        _lib.vpo_unpack_tokens.argtypes = ([C.c_void_p] * 4 + [C.c_int] * 3 + [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                            C.c_int64, C.c_int64, C.c_void_p, C.c_void_p])
        _lib.vpo_exchange_put.argtypes = [C.c_void_p] * 5 + [C.c_int] * 3 + [C.c_void_p] * 4
        _lib.vpo_pack.argtypes = ([C.c_void_p] * 4 + [C.c_int] * 3 + [C.c_void_p, C.c_int, C.c_int, C.c_int,
                                  C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p])
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _param(params, name, default=0):
    if isinstance(params, dict):
        return int(params.get(name, default))
    return int(getattr(params, name, default))


def demand_from_routing(expert_idx, experts_per_rank: int, N: int, row_bytes: int, src0: int = 0):
    """Demand rows ``[n_src, N]`` of the sources ``src0..`` from ``[n_src, T, topk]`` routing indices; also the
    out-of-range flag."""
    idx = np.ascontiguousarray(expert_idx, dtype=np.int32)
    n_src, T, topk = idx.shape
    rows = np.zeros((n_src, N), np.int64)
    bad = _load().vpo_demand_from_routing(_p(idx), n_src, T, topk, int(experts_per_rank), int(N), int(src0),
                                          int(row_bytes), _p(rows))
    return rows, int(bad)


class OracleCatalog:
    """A parsed topology + channel catalog held by the C oracle."""

    def __init__(self, topo_blob: bytes, chan_blob: bytes):
        lib = _load()
        err = C.c_int(0)
        self._topo, self._chan = bytes(topo_blob), bytes(chan_blob)
        self._h = lib.vpo_load(self._topo, len(self._topo), self._chan, len(self._chan), C.byref(err))
        if not self._h:
            raise ValueError(f"oracle rejected the catalog blobs (code {err.value})")
        info = np.zeros(8, dtype=np.int32)
        lib.vpo_info(self._h, _p(info))
        (self.N, self.G, self.g, self.n_inst, self.n_shapes, self.n_families,
         self.max_nnz, self.n_res) = (int(x) for x in info)
        self.W = int(lib.vpo_rate_lcm(self._h))

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.vpo_free(self._h)
            self._h = None

    # ---- catalog / channel model -------------------------------------
    def check(self) -> int:
        return int(_load().vpo_check_catalog(self._h))

    def covers(self) -> bool:
        return bool(_load().vpo_catalog_covers(self._h))

    def lanes_feasible(self, dst, inst) -> int:
        dst = np.ascontiguousarray(dst, dtype=np.int16)
        inst = np.ascontiguousarray(inst, dtype=np.uint16)
        return int(_load().vpo_lanes_feasible(self._h, _p(dst), _p(inst)))

    def aggregate_bw(self, dst, inst) -> Fraction:
        dst = np.ascontiguousarray(dst, dtype=np.int16)
        inst = np.ascontiguousarray(inst, dtype=np.uint16)
        return Fraction(int(_load().vpo_aggregate_bw_x5040(self._h, _p(dst), _p(inst))), 5040)

    def instances(self):
        """(src_group, dst_group, kind, bw, mult, resources) per instance, parsed from the blob."""
        n = struct.unpack_from("<I", self._topo, 28)[0]
        out = []
        for r in range(n):
            a, d, kind, nres, mult, bw, r0, r1, r2, r3 = struct.unpack_from("<HHBBHI4H", self._topo, 32 + 20 * r)
            out.append((a, d, kind, bw, mult, (r0, r1, r2, r3)[:nres]))
        return out

    def families(self) -> np.ndarray:
        off = 24 + 8 * (self.n_shapes + 1) + 8 * struct.unpack_from("<I", self._chan, 20)[0]
        return np.frombuffer(self._chan, dtype="<u2", count=self.n_families * self.N, offset=off).reshape(
            self.n_families, self.N)

    # ---- Algorithm 2 --------------------------------------------------
    def _alloc(self, B: int, k_max: int):
        N = self.N
        return dict(
            n_steps=np.zeros(B, np.int32), chan_id=np.zeros((B, k_max), np.int32),
            lane_dst=np.zeros((B, k_max, N), np.int16), lane_inst=np.zeros((B, k_max, N), np.uint16),
            lane_bytes=np.zeros((B, k_max, N), np.int64), send_off=np.zeros((B, k_max + 1, N), np.int64),
            recv_off=np.zeros((B, k_max + 1, N), np.int64), tau_ns=np.zeros(B, np.int64),
            status=np.zeros(B, np.int32))

    def schedule_batch(self, demand, params, tau_in=None, threads: int = 1) -> dict:
        """Plans for a ``[B,N,N]`` int64 demand batch; ``threads`` splits the batch statically."""
        lib = _load()
        D = np.ascontiguousarray(demand, dtype=np.int64)
        B, N = D.shape[0], self.N
        assert D.shape == (B, N, N)
        k_max = _param(params, "k_max") or 8 * N
        out = self._alloc(B, k_max)
        tau = None if tau_in is None else np.ascontiguousarray(tau_in, dtype=np.int64)
        args = (_param(params, "lambda_ns"), _param(params, "k_target"), _param(params, "n_start"),
                _param(params, "i_aa"), _param(params, "granule_bytes", 1), k_max)

        def run(lo, hi):
            rc = lib.vpo_schedule_batch(self._h, _p(D), _p(tau), lo, hi, *args,
                                        _p(out["n_steps"]), _p(out["chan_id"]), _p(out["lane_dst"]),
                                        _p(out["lane_inst"]), _p(out["lane_bytes"]), _p(out["send_off"]),
                                        _p(out["recv_off"]), _p(out["tau_ns"]), _p(out["status"]))
            if rc:
                raise ValueError("oracle: bad scheduler parameters")

        threads = max(1, min(int(threads), B))
        if threads == 1:
            run(0, B)
        else:
            cuts = [B * t // threads for t in range(threads + 1)]
            with ThreadPoolExecutor(threads) as ex:
                list(ex.map(lambda t: run(cuts[t], cuts[t + 1]), range(threads)))
        out["k_max"] = k_max
        return out

    def schedule(self, D, params, tau_in: int = 0, trace_cap: int = 0) -> dict:
        """One matrix; with ``trace_cap`` > 0 also returns the trace records: (step, family, start, sweep, F) per
        AA sweep, (step, family, -2 - start, slot, src * 65536 + dst) for the binding each run ends with, and
        (step, family, -1, sum of volumes, W * duration) per candidate."""
        lib = _load()
        D = np.ascontiguousarray(D, dtype=np.int64)
        N = self.N
        k_max = _param(params, "k_max") or 8 * N
        o = self._alloc(1, k_max)
        trace = np.zeros((max(trace_cap, 1), 5), np.int64)
        tl = np.zeros(1, np.int32)
        rc = lib.vpo_schedule(self._h, _p(D), int(tau_in), _param(params, "lambda_ns"), _param(params, "k_target"),
                              _param(params, "n_start"), _param(params, "i_aa"), _param(params, "granule_bytes", 1),
                              k_max, _p(o["n_steps"]), _p(o["chan_id"]), _p(o["lane_dst"]), _p(o["lane_inst"]),
                              _p(o["lane_bytes"]), _p(o["send_off"]), _p(o["recv_off"]), _p(o["tau_ns"]),
                              _p(o["status"]), _p(trace) if trace_cap else None, trace_cap, _p(tl))
        if rc:
            raise ValueError("oracle: bad scheduler parameters")
        out = {k: v[0] for k, v in o.items()}
        out["k_max"] = k_max
        out["trace"] = trace[: int(tl[0])]
        return out

    def sweep_plan_time(self, demand, params, lambdas, k_targets, threads: int = 1):
        """Eq. (2) over a grid: for every (lambda, K_target) decompose the batch with those two parameters and evaluate
        rate_lcm x T(S) with that lambda.  Returns (time_xw int64 [n_lambda, n_k, B], n_steps int32 of the same shape)."""
        import copy
        D = np.ascontiguousarray(demand, dtype=np.int64)
        B = D.shape[0]
        T = np.zeros((len(lambdas), len(k_targets), B), np.int64)
        K = np.zeros((len(lambdas), len(k_targets), B), np.int32)
        for i, lam in enumerate(lambdas):
            for j, kt in enumerate(k_targets):
                q = copy.copy(params)
                if isinstance(q, dict):
                    q = dict(q, lambda_ns=int(lam), k_target=int(kt))
                else:
                    q.lambda_ns, q.k_target = int(lam), int(kt)
                out = self.schedule_batch(D, q, threads=threads)
                K[i, j] = out["n_steps"]
                for b in range(B):
                    one = {k: out[k][b] for k in ("n_steps", "lane_dst", "lane_inst", "lane_bytes")}
                    T[i, j, b] = self.modeled_time_xw(one, int(lam))
        return T, K

    # ---- plan-level quantities ----------------------------------------
    def modeled_time(self, plan: dict, lambda_ns: int) -> Fraction:
        """Eq. (2): modeled completion time of a one-matrix plan, in nanoseconds."""
        v = _load().vpo_modeled_time_xW(self._h, int(plan["n_steps"]), _p(np.ascontiguousarray(plan["lane_dst"])),
                                        _p(np.ascontiguousarray(plan["lane_inst"])),
                                        _p(np.ascontiguousarray(plan["lane_bytes"])), int(lambda_ns))
        return Fraction(int(v), self.W)

    def modeled_time_xw(self, plan: dict, lambda_ns: int) -> int:
        """Eq. (2) scaled by the lcm of the path rates (an integer, nanoseconds x W)."""
        return int(self.modeled_time(plan, lambda_ns) * self.W)

    def check_plan(self, D, plan: dict, tau: int = 0, granule: int = 1) -> int:
        D = np.ascontiguousarray(D, dtype=np.int64)
        return int(_load().vpo_check_plan(self._h, _p(D), int(plan["n_steps"]),
                                          _p(np.ascontiguousarray(plan["lane_dst"])),
                                          _p(np.ascontiguousarray(plan["lane_inst"])),
                                          _p(np.ascontiguousarray(plan["lane_bytes"])), int(tau), int(granule)))

    def lower_bound(self, D) -> Fraction:
        """Link-load lower bound on Eq. (2) with lambda = 0, in nanoseconds: the largest of
        (i) every rank's send / receive volume over the fastest path rate,
        (ii) demand forced through one directed resource over its fastest path,
        (iii) traffic leaving (entering) a group over the largest total rate any catalog
        family offers out of (into) that group."""
        D = np.asarray(D, dtype=np.int64)
        N, G, g = self.N, self.G, self.g
        inst = self.instances()
        bw_max = max(i[3] for i in inst)
        lb = Fraction(int(max(D.sum(1).max(), D.sum(0).max())), bw_max)
        Dhat = D.reshape(G, g, G, g).sum(axis=(1, 3))
        pairs = {}
        for (a, d, kind, bw, mult, res) in inst:
            pairs.setdefault((a, d), []).append((bw, set(res)))
        forced, fbw = {}, {}
        for (a, d), lst in pairs.items():
            common = set.intersection(*[r for _, r in lst]) if lst else set()
            for l in common:
                forced[l] = forced.get(l, 0) + int(Dhat[a, d])
                fbw[l] = max(fbw.get(l, 0), max(b for b, _ in lst))
        for l, v in forced.items():
            lb = max(lb, Fraction(v, fbw[l]))
        fam = self.families()
        out_rate = np.zeros(G, dtype=np.int64)
        in_rate = np.zeros(G, dtype=np.int64)
        a_of = np.array([i[0] for i in inst]); d_of = np.array([i[1] for i in inst])
        bw_of = np.array([i[3] for i in inst], dtype=np.int64)
        cross = (a_of != d_of)
        for f in fam:
            o = np.bincount(a_of[f], weights=bw_of[f] * cross[f], minlength=G).astype(np.int64)
            i_ = np.bincount(d_of[f], weights=bw_of[f] * cross[f], minlength=G).astype(np.int64)
            out_rate = np.maximum(out_rate, o)
            in_rate = np.maximum(in_rate, i_)
        for a in range(G):
            leave = int(Dhat[a].sum() - Dhat[a, a]); enter = int(Dhat[:, a].sum() - Dhat[a, a])
            if leave:
                lb = max(lb, Fraction(leave, int(out_rate[a])))
            if enter:
                lb = max(lb, Fraction(enter, int(in_rate[a])))
        return lb

    # ---- pack -----------------------------------------------------------
    def pack(self, plan: dict, rank: int, expert_idx, experts_per_rank: int, rows, capacity_rows: int,
             staged: Optional[np.ndarray] = None):
        """Pack ``rank``'s rows for a one-matrix plan.  ``rows`` is ``[T, row_bytes]`` uint8 (or any
        2-D array viewed as bytes).  Returns (staged [capacity_rows,row_bytes] uint8, src_map, status)."""
        idx = np.ascontiguousarray(expert_idx, dtype=np.int32)
        T, topk = idx.shape
        rows_b = np.ascontiguousarray(rows).view(np.uint8).reshape(T, -1)
        row_bytes = rows_b.shape[1]
        if staged is None:
            staged = np.zeros((capacity_rows, row_bytes), np.uint8)
        src_map = np.full(capacity_rows, -1, np.int32)
        n_steps = np.asarray([plan["n_steps"]], dtype=np.int32)
        st = _load().vpo_pack(_p(n_steps), _p(np.ascontiguousarray(plan["lane_dst"])),
                              _p(np.ascontiguousarray(plan["lane_bytes"])),
                              _p(np.ascontiguousarray(plan["send_off"])), self.N, int(rank), int(plan["k_max"]),
                              _p(idx), T, topk, int(experts_per_rank), _p(rows_b), row_bytes, _p(staged),
                              capacity_rows * row_bytes, _p(src_map))
        return staged, src_map, int(st)

    # ---- exchange -------------------------------------------------------
    def exchange(self, plan: dict, staged_by_src: dict, row_bytes: int = 1):
        """Every rank in ``staged_by_src`` (rank -> staged bytes, 2-D or flat uint8) sends its chunks as the one-matrix
        plan says.  Returns (receive buffers per rank as flat uint8 arrays sized by the plan's receive totals,
        arrived bytes per rank, status)."""
        N, K = self.N, int(plan["n_steps"])
        cap = np.ascontiguousarray(plan["recv_off"][K], dtype=np.int64)
        bufs = [np.zeros(max(int(cap[j]), 1), np.uint8) for j in range(N)]
        ptrs = (C.c_void_p * N)(*[b.ctypes.data for b in bufs])
        arrived = np.zeros(N, np.uint64)
        n_steps = np.asarray([plan["n_steps"]], dtype=np.int32)
        st = 0
        for i, staged in staged_by_src.items():
            flat = np.ascontiguousarray(staged).view(np.uint8).reshape(-1)
            st |= _load().vpo_exchange_put(_p(n_steps), _p(np.ascontiguousarray(plan["lane_dst"])),
                                           _p(np.ascontiguousarray(plan["lane_bytes"])), _p(np.ascontiguousarray(plan["send_off"])),
                                           _p(np.ascontiguousarray(plan["recv_off"])), N, int(i), int(plan["k_max"]),
                                           _p(flat), ptrs, _p(cap), _p(arrived))
        return [b[: int(cap[j])] for j, b in enumerate(bufs)], arrived, int(st)

    # ---- unpack ---------------------------------------------------------
    def unpack_tokens(self, plan: dict, rank: int, expert_idx, experts_per_rank: int, recv, out=None):
        """Receive side of the return direction: ``plan`` is the one-matrix plan of the return call, ``expert_idx``
        ``[T, topk]`` this rank's routing, ``recv`` its return receive buffer ([R, row_bytes] bytes view).  Returns
        (out rows [T*topk, row_bytes], out_map, status); rows of copies that do not travel keep ``out``'s content."""
        recv_b = np.ascontiguousarray(recv).view(np.uint8)
        R = recv_b.shape[0]
        recv_b = recv_b.reshape(R, -1)
        row_bytes = recv_b.shape[1]
        idx = np.ascontiguousarray(expert_idx, dtype=np.int32)
        T, topk = idx.shape
        if out is None:
            out = np.zeros((T * topk, row_bytes), np.uint8)
        out_map = np.full(T * topk, -1, np.int32)
        n_steps = np.asarray([plan["n_steps"]], dtype=np.int32)
        st = _load().vpo_unpack_tokens(_p(n_steps), _p(np.ascontiguousarray(plan["lane_dst"])),
                                       _p(np.ascontiguousarray(plan["lane_bytes"])), _p(np.ascontiguousarray(plan["recv_off"])),
                                       self.N, int(rank), int(plan["k_max"]), _p(idx), T, topk, int(experts_per_rank),
                                       _p(recv_b), row_bytes, R, _p(out), _p(out_map))
        return out, out_map, int(st)

    def unpack(self, plan: dict, rank: int, recv, recv_expert, experts_per_rank: int):
        """Expert-major unpack of ``rank``'s receive buffer ``recv`` ([R, row_bytes] bytes view) for a one-matrix
        plan.  Returns (out rows, expert_off, out_src, out_map, status)."""
        recv_b = np.ascontiguousarray(recv).view(np.uint8)
        R = recv_b.shape[0]
        recv_b = recv_b.reshape(R, -1)
        row_bytes = recv_b.shape[1]
        exp = np.ascontiguousarray(recv_expert, dtype=np.int32)
        out = np.zeros_like(recv_b)
        expert_off = np.zeros(experts_per_rank + 1, np.int32)
        out_src = np.full(R, -1, np.int32)
        out_map = np.full(R, -1, np.int32)
        n_steps = np.asarray([plan["n_steps"]], dtype=np.int32)
        st = _load().vpo_unpack(_p(n_steps), _p(np.ascontiguousarray(plan["lane_dst"])),
                                _p(np.ascontiguousarray(plan["recv_off"])), self.N, int(rank), int(plan["k_max"]),
                                _p(recv_b), row_bytes, R, _p(exp), int(experts_per_rank), _p(out), _p(expert_off),
                                _p(out_src), _p(out_map))
        return out, expert_off, out_src, out_map, int(st)
