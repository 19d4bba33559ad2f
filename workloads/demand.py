"""Seeded synthetic demand matrices and routing indices.

The paper's communication workloads are synthetic: demand derived from
randomized top-k MoE routing (Section 6, "Workloads"), uniform AlltoAll, and
sequence-parallel head/sequence redistribution (Section 6.2).  These generators
reproduce their shapes and distributions; they stand in for the Qwen3 / Wan2.1
traces, which are not available.

MoE recipe: expert ``e`` lives on rank ``e // (E/N)``; popularity
``p_e ~ (1 + rho(e))^(-s)`` with ``rho`` a permutation of expert ids; every token
draws ``topk`` *distinct* experts without replacement in proportion to ``p``
(Gumbel-top-k on ``log p``); ``D[i][j] = row_bytes * #{copies from rank i to an
expert on rank j}``, ``D[i][i] = 0``.
"""
from __future__ import annotations

from typing import Optional, Sequence, Union

import numpy as np
import torch

_CHUNK_ELEMS = 1 << 26  # Gumbel keys materialised at once


def _log_popularity(E: int, s: float, perm: Optional[torch.Tensor], device) -> torch.Tensor:
    rho = torch.arange(E, dtype=torch.float64) if perm is None else perm.to(torch.float64).cpu()
    return (-float(s) * torch.log1p(rho)).to(torch.float32).to(device)


def moe_routing(n_tokens: int, E: int, topk: int, s: float, seed: int,
                perm: Optional[torch.Tensor] = None, device: str = "cpu") -> torch.Tensor:
    """``[n_tokens, topk]`` int32 expert ids, slot order = decreasing Gumbel key."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(int(seed))
    logp = _log_popularity(E, s, perm, dev)
    out = torch.empty((n_tokens, topk), dtype=torch.int32, device=dev)
    step = max(1, _CHUNK_ELEMS // E)
    for lo in range(0, n_tokens, step):
        hi = min(n_tokens, lo + step)
        u = torch.rand((hi - lo, E), generator=gen, device=dev, dtype=torch.float32)
        u.clamp_(min=1e-20, max=1.0 - 1e-7)
        keys = logp - torch.log(-torch.log(u))
        out[lo:hi] = torch.topk(keys, topk, dim=1).indices.to(torch.int32)
    return out


def demand_from_routing(idx: torch.Tensor, src: torch.Tensor, N: int, E: int,
                        row_bytes: int) -> torch.Tensor:
    """Histogram (source rank, destination rank) pairs of routed copies into ``D`` (bytes)."""
    dst = (idx.to(torch.int64) // (E // N))
    flat = (src.to(torch.int64).unsqueeze(1) * N + dst).reshape(-1)
    D = torch.bincount(flat, minlength=N * N).reshape(N, N) * int(row_bytes)
    D.fill_diagonal_(0)
    return D.to(torch.int64)


def moe_demand(N: int, tokens_per_rank: Union[int, Sequence[int]], E: int, topk: int, s: float,
               row_bytes: int, seed: int, perm: Optional[torch.Tensor] = None,
               device: str = "cpu", return_routing: bool = False):
    """One ``[N, N]`` int64 demand matrix (on CPU) from simulated top-k routing of all ranks."""
    if isinstance(tokens_per_rank, (int, np.integer)):
        counts = [int(tokens_per_rank)] * N
    else:
        counts = [int(t) for t in tokens_per_rank]
    total = sum(counts)
    idx = moe_routing(total, E, topk, s, seed, perm, device)
    src = torch.repeat_interleave(torch.arange(N, device=idx.device),
                                  torch.tensor(counts, device=idx.device))
    D = demand_from_routing(idx, src, N, E, row_bytes).cpu()
    if return_routing:
        return D, idx, counts
    return D


def sp_demand(N: int, seed: int, group: int = 8, heads: int = 40, head_dim: int = 128,
              elem_bytes: int = 2, lo: int = 1024, hi: int = 32768) -> torch.Tensor:
    """Ulysses-style head/sequence redistribution inside groups of ``group`` consecutive
    ranks: rank ``i`` holds a sequence shard of ``L_i`` tokens and sends every peer of
    its group the ``heads/group`` heads that peer owns."""
    rng = np.random.default_rng(int(seed))
    L = rng.integers(lo, hi + 1, size=N, dtype=np.int64)
    per_peer = L * (heads // group) * head_dim * elem_bytes
    D = np.zeros((N, N), dtype=np.int64)
    for i in range(N):
        b = (i // group) * group
        D[i, b:b + group] = per_peer[i]
        D[i, i] = 0
    return torch.from_numpy(D)


def uniform_demand(N: int, c: int) -> torch.Tensor:
    """AlltoAll: every rank sends ``c`` bytes to every other rank."""
    D = torch.full((N, N), int(c), dtype=torch.int64)
    D.fill_diagonal_(0)
    return D
