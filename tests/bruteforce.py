"""Exhaustive search over schedules for tiny deployments (N <= 4).

Independent of the oracle's scheduler: it enumerates every concrete feasible
channel (Section 3: a fixed-point-free permutation plus one path per lane, no
directed resource used twice, Eq. 1), gives each lane the Eq. (9) volume
min(cap, D_rem), and minimises the modeled completion time of Eq. (2) over all
channel sequences by memoised depth-first search.
"""
from __future__ import annotations

from fractions import Fraction
from functools import lru_cache
from itertools import permutations, product
from typing import Dict, List, Sequence, Tuple


def concrete_channels(N: int, g: int, instances) -> List[Tuple[Tuple[int, ...], Tuple[int, ...]]]:
    """All feasible channels as (pi, instance id per source rank)."""
    by_pair: Dict[Tuple[int, int], List[int]] = {}
    for r, (a, d, kind, bw, mult, res) in enumerate(instances):
        by_pair.setdefault((a, d), []).append(r)
    out = []
    for pi in permutations(range(N)):
        if any(pi[i] == i for i in range(N)):
            continue
        choices = [by_pair.get((i // g, pi[i] // g), []) for i in range(N)]
        for paths in product(*choices):
            used = set()
            times: Dict[int, int] = {}
            ok = True
            for r in paths:
                times[r] = times.get(r, 0) + 1
                if times[r] > instances[r][4]:
                    ok = False
                    break
                for l in instances[r][5]:
                    if l in used:
                        ok = False
                        break
                    used.add(l)
                if not ok:
                    break
            if ok:
                out.append((pi, paths))
    return out


def optimal_time(N: int, g: int, instances, D: Sequence[Sequence[int]], cap: Sequence[int],
                 lambda_ns: int) -> Fraction:
    """min over valid schedules of sum_k (lambda + max_i x_ki / bw), in nanoseconds."""
    chans = concrete_channels(N, g, instances)
    bw = [i[3] for i in instances]

    @lru_cache(maxsize=None)
    def best(state: Tuple[int, ...]) -> Fraction:
        if not any(state):
            return Fraction(0)
        res = None
        seen = set()
        for pi, paths in chans:
            xs = tuple(min(cap[paths[i]], state[i * N + pi[i]]) for i in range(N))
            if not any(xs):
                continue
            key = (tuple(pi[i] if xs[i] else -1 for i in range(N)), xs,
                   tuple(bw[paths[i]] if xs[i] else 0 for i in range(N)))
            if key in seen:
                continue
            seen.add(key)
            dur = lambda_ns + max(Fraction(xs[i], bw[paths[i]]) for i in range(N))
            nxt = list(state)
            for i in range(N):
                nxt[i * N + pi[i]] -= xs[i]
            t = dur + best(tuple(nxt))
            if res is None or t < res:
                res = t
        assert res is not None, "demand not servable"
        return res

    return best(tuple(int(v) for row in D for v in row))
