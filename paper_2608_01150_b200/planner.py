"""The two solver-free steps of the paper's planner (Section IV-C), driven by the price table that
:mod:`.profiler` measures on the engine: the catalog cut that separates filler buckets from anchor
buckets (Eq. 3) and Filler Packing, which keeps fillers whole and places them in the compute and memory
headroom the anchors leave (Eq. 7).  Anchor Placement (Stage 1) needs a CP-SAT solver and is not here.

Host-side numpy code; placements it produces are fed to ``build_tasks`` rank by rank.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np


def catalog_cut(whole_prices: Sequence[float]) -> int:
    """Eq. 3: the contiguous cut k* of the price-ordered catalog that minimises the within-set dispersion
    of log w on both sides (a two-class Fisher break); buckets 1..k* are fillers.  O(B) with prefix sums:
    sum_i (x_i - mean)^2 = sum x_i^2 - (sum x_i)^2 / n on each side.  Ties go to the smallest k."""
    w = np.asarray(whole_prices, dtype=np.float64)
    if w.ndim != 1 or w.size < 2:
        raise ValueError("a cut needs at least two buckets")
    if np.any(np.diff(w) < 0):
        raise ValueError("buckets must be ordered by nondecreasing price")
    if not np.all(np.isfinite(w)) or np.any(w <= 0):
        raise ValueError("prices must be positive and finite (the cut works on their logarithms)")
    x = np.log(w)
    x = x - x.mean()                       # the dispersion is shift-invariant; centring keeps the sums small
    s1, s2 = np.cumsum(x), np.cumsum(x * x)
    k = np.arange(1, w.size)               # fillers = first k buckets
    left = s2[k - 1] - s1[k - 1] ** 2 / k
    right = (s2[-1] - s2[k - 1]) - (s1[-1] - s1[k - 1]) ** 2 / (w.size - k)
    score = left + right
    best = score.min()
    # ties (to rounding of the prefix-sum form) go to the smallest k
    tol = 1e-12 * max(1.0, float(s2[-1]))
    return int(k[np.nonzero(score <= best + tol)[0][0]])


def split_catalog(prices_whole: dict) -> Tuple[List[str], List[str]]:
    """Orders buckets by whole-sequence price and applies the cut: (filler buckets, anchor buckets)."""
    names = sorted(prices_whole, key=lambda b: (prices_whole[b], b))
    k = catalog_cut([prices_whole[b] for b in names])
    return names[:k], names[k:]


def filler_packing(filler_prices: Sequence[float], filler_mem, load: Sequence[float], mem: Sequence[float],
                   mem_cap: float, floor: float) -> Optional[List[int]]:
    """Eq. 7: fillers in decreasing price, each to the feasible rank whose tighter post-placement slack
    min{(F - C_r - p_s) / F, (M_cap - M_r - M_{s,r}) / M_cap} is largest (ties: lowest rank); ledgers start
    from the anchors' `load` and `mem`.  `filler_mem` is [n_fillers, n_ranks] (or [n_fillers], the same on
    every rank).  Returns the rank of each filler, or None if one fits on no rank."""
    p = np.asarray(filler_prices, dtype=np.float64)
    C = np.array(load, dtype=np.float64)
    M = np.array(mem, dtype=np.float64)
    fm = np.asarray(filler_mem, dtype=np.float64)
    if fm.ndim == 1:
        fm = np.repeat(fm[:, None], C.size, axis=1)
    out = [-1] * p.size
    for s in sorted(range(p.size), key=lambda i: (-p[i], i)):
        h_m = mem_cap - M
        feasible = h_m >= fm[s]
        if not feasible.any():
            return None
        score = np.minimum((floor - C - p[s]) / floor, (h_m - fm[s]) / mem_cap)
        score[~feasible] = -np.inf
        r = int(np.argmax(score))          # first maximum = lowest rank
        out[s] = r
        C[r] += p[s]
        M[r] += fm[s, r]
    return out
