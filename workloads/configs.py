"""The five benchmark/parity configurations, as seeded synthetic inputs.

Config 1  N=8   one node                64 MoE matrices     complete catalog
Config 2  N=16  two nodes               256 MoE matrices    complete catalog
Config 3  N=64  eight nodes             1024 MoE matrices   node-template catalog
Config 4  N=256 thirty-two nodes        4096 MoE + SP       node-template catalog
Config 5  pack of one rank's rows on a config-2-topology plan
"""
from __future__ import annotations

from dataclasses import dataclass, asdict
from functools import lru_cache
from typing import Dict, Optional

import numpy as np
import torch

from .topology import Catalog, complete_catalog, node_template_catalog, tree_topology
from .demand import moe_demand, sp_demand


@dataclass
class SchedParams:
    lambda_ns: int = 8000  # per-activation overhead, about the paper's 7.872 us small-message P50
    k_target: int = 0      # 0 -> 2N  (Section 5: between N and 3N)
    n_start: int = 4
    i_aa: int = 3
    granule_bytes: int = 1
    k_max: int = 0         # 0 -> 8N

    def resolved(self, N: int) -> "SchedParams":
        p = SchedParams(**asdict(self))
        if p.k_target == 0:
            p.k_target = 2 * N
        if p.k_max == 0:
            p.k_max = 8 * N
        return p


CONFIGS: Dict[int, dict] = {
    1: dict(nodes=1, catalog="complete", batch=64, seed=0, row_bytes=14336),
    2: dict(nodes=2, catalog="complete", batch=256, seed=1, row_bytes=8192),
    3: dict(nodes=8, catalog="template", batch=1024, seed=2, row_bytes=14336),
    4: dict(nodes=32, catalog="template", batch=4096, seed=3, row_bytes=14336),
    5: dict(nodes=2, catalog="complete", batch=1, seed=4, row_bytes=14336),
}


@lru_cache(maxsize=None)
def catalog_for(nodes: int, kind: str, g: int = 4, pcie_bw: int = 64, nic_bw: int = 64) -> Catalog:
    topo = tree_topology(nodes, g=g, pcie_bw=pcie_bw, nic_bw=nic_bw)
    return complete_catalog(topo) if kind == "complete" else node_template_catalog(topo)


def _matrix_seed(base: int, b: int) -> int:
    return base * 1_000_000 + b


def build_config(idx: int, device: str = "cpu", batch: Optional[int] = None,
                 token_scale: float = 1.0) -> dict:
    """Inputs of scheduler config ``idx`` (1..4): catalog, ``[B,N,N]`` int64 demand (CPU), params.

    ``batch`` truncates the batch (matrix ``b`` is the same whatever the batch size);
    ``token_scale`` < 1 shrinks token counts for quick CPU tests.
    """
    cfg = CONFIGS[idx]
    cat = catalog_for(cfg["nodes"], cfg["catalog"])
    N = cat.topology.N
    B = cfg["batch"] if batch is None else min(batch, cfg["batch"])
    base = cfg["seed"]
    rb = cfg["row_bytes"]
    mats = []
    granule = rb
    if idx == 1:
        T = max(1, int(4096 * token_scale))
        for b in range(B):
            mats.append(moe_demand(N, T, 128, 8, 1.2, rb, _matrix_seed(base, b), device=device))
    elif idx == 2:
        T = max(1, int(8192 * token_scale))
        s_all = np.random.default_rng(base).uniform(0.0, 1.5, size=cfg["batch"])
        for b in range(B):
            mats.append(moe_demand(N, T, 256, 8, float(s_all[b]), rb, _matrix_seed(base, b), device=device))
    elif idx == 3:
        rng = np.random.default_rng(base)
        n_steps, n_layers = 64, 16
        tokens = rng.integers(256, 16384 + 1, size=(n_steps, N))
        perms = [torch.from_numpy(rng.permutation(128)) for _ in range(n_layers)]
        for b in range(B):
            step, layer = divmod(b, n_layers)
            T = np.maximum(1, (tokens[step] * token_scale).astype(np.int64))
            mats.append(moe_demand(N, T, 128, 8, 1.0, rb, _matrix_seed(base, b),
                                   perm=perms[layer], device=device))
    elif idx == 4:
        rng = np.random.default_rng(base)
        total = cfg["batch"]
        is_sp = np.zeros(total, dtype=bool)
        is_sp[total // 2:] = True
        rng.shuffle(is_sp)
        s_choice = rng.choice([0.0, 0.8, 1.5], size=total)
        e_choice = rng.integers(0, 15, size=total)
        granule = 256
        for b in range(B):
            if is_sp[b]:
                mats.append(sp_demand(N, _matrix_seed(base, b)))
            else:
                T = max(1, int((1 << int(e_choice[b])) * token_scale))
                mats.append(moe_demand(N, T, 256, 8, float(s_choice[b]), rb,
                                       _matrix_seed(base, b), device=device))
    else:
        raise ValueError("scheduler configs are 1..4; use build_pack_case for config 5")
    # the one-NIC-per-switch tree needs at least 16*(G-2) rounds for dense cross-node demand, which
    # at N=256 already exceeds 8N for skewed matrices: config 4 gets room for 16N activations
    params = SchedParams(granule_bytes=granule, k_max=16 * N if idx == 4 else 0).resolved(N)
    return dict(config=idx, catalog=cat, demand=torch.stack(mats), params=params)


def build_pack_case(device: str = "cpu", tokens: int = 16384, hidden: int = 7168,
                    rank: int = 8, nodes: int = 2, experts: int = 256, topk: int = 8,
                    s: float = 1.2, seed: Optional[int] = None) -> dict:
    """Config 5: all ranks route ``tokens`` tokens (top-k over ``experts``), giving one demand
    matrix; ``rank``'s routing indices and bf16 rows (random bits, every row distinct with
    overwhelming probability) are what the pack consumes.  ``rows`` stay on ``device``."""
    cfg = CONFIGS[5]
    cat = catalog_for(nodes, "complete")
    N = cat.topology.N
    row_bytes = hidden * 2
    base = cfg["seed"] if seed is None else seed
    D, idx_all, counts = moe_demand(N, tokens, experts, topk, s, row_bytes,
                                    _matrix_seed(base, 0), device=device, return_routing=True)
    lo = sum(counts[:rank])
    expert_idx = idx_all[lo:lo + counts[rank]].contiguous()
    gen = torch.Generator(device=torch.device(device))
    gen.manual_seed(_matrix_seed(base, 1))
    rows = torch.randint(-32768, 32768, (tokens, hidden), generator=gen,
                         device=torch.device(device), dtype=torch.int16)
    params = SchedParams(granule_bytes=row_bytes).resolved(N)
    return dict(config=5, catalog=cat, demand=D.unsqueeze(0), params=params, rank=rank,
                expert_idx=expert_idx, rows=rows, row_bytes=row_bytes, topk=topk,
                experts_per_rank=experts // N)
