"""TEST INFRASTRUCTURE: plain restatements of the two solver-free planner steps of the paper
(Section IV-C): the catalog cut (Eq. 3) and Filler Packing (Eq. 7).  Written out term by term from
the equations, in pure Python floats, with no shortcuts; nothing in the product path uses this file.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence


def catalog_cut(whole_prices: Sequence[float]) -> int:
    """Eq. 3.  `whole_prices` are the profiled whole-sequence times w_1 <= ... <= w_B of the catalog buckets
    in nondecreasing order.  Returns k*: buckets 1..k* are fillers, k*+1..B anchors.  For every cut
    1 <= k < B the score is the sum of squared deviations of log w_i from the mean log on its own side;
    the smallest score wins, ties go to the smallest k."""
    B = len(whole_prices)
    if B < 2:
        raise ValueError("a cut needs at least two buckets")
    for i in range(1, B):
        if whole_prices[i] < whole_prices[i - 1]:
            raise ValueError("buckets must be ordered by nondecreasing price")
    logs = [math.log(w) for w in whole_prices]
    best_k, best = None, None
    for k in range(1, B):
        fill, anc = logs[:k], logs[k:]
        mu_fill = sum(fill) / len(fill)
        mu_anc = sum(anc) / len(anc)
        score = sum((x - mu_fill) ** 2 for x in fill) + sum((x - mu_anc) ** 2 for x in anc)
        if best is None or score < best:
            best_k, best = k, score
    return best_k


def filler_packing(filler_prices: Sequence[float], filler_mem: Sequence[Sequence[float]],
                   load: Sequence[float], mem: Sequence[float], mem_cap: float, floor: float) -> Optional[List[int]]:
    """Eq. 7.  Fillers stay whole and are taken in decreasing price p_s (ties: input order).  With compute
    headroom h^C_r = F - C_r and memory headroom h^M_r = M_cap - M_r, sequence s goes to the feasible rank
    (h^M_r >= M_{s,r}) that maximises min{(h^C_r - p_s) / F, (h^M_r - M_{s,r}) / M_cap}; ties go to the
    lowest rank.  The ledgers C_r, M_r (initialised from the anchors: `load`, `mem`) are updated after every
    assignment.  Returns the rank of each filler in input order, or None when some filler fits nowhere.
    `filler_mem[s][r]` is the memory of s kept whole on rank r; `floor` is F, the zero-communication load
    floor sum_s P[b(s), whole] / N over ALL sequences of the batch."""
    C, M = list(load), list(mem)
    N = len(C)
    order = sorted(range(len(filler_prices)), key=lambda s: (-filler_prices[s], s))
    out = [-1] * len(filler_prices)
    for s in order:
        best_r, best = None, None
        for r in range(N):
            h_c, h_m = floor - C[r], mem_cap - M[r]
            if h_m < filler_mem[s][r]:
                continue
            rho_c = (h_c - filler_prices[s]) / floor
            rho_m = (h_m - filler_mem[s][r]) / mem_cap
            score = min(rho_c, rho_m)
            if best is None or score > best:
                best_r, best = r, score
        if best_r is None:
            return None
        out[s] = best_r
        C[best_r] += filler_prices[s]
        M[best_r] += filler_mem[s][best_r]
    return out
