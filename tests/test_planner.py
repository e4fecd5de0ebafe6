"""Catalog cut (paper Eq. 3) and Filler Packing (Eq. 7): the plain restatement in oracle/planner.py pinned by
facts the equations fix, and the numpy implementation checked against it decision for decision."""
import math

import numpy as np
import pytest

from oracle import planner as O
from paper_2608_01150_b200 import planner as P


# ---------------------------------------------------------------------------------------- pins of the oracle
def test_cut_separates_two_clusters_and_ignores_common_rescaling():
    w = [0.07, 0.08, 0.11, 20.0, 55.0, 110.0]        # images / short clips vs videos (ms)
    assert O.catalog_cut(w) == 3
    # Eq. 3 works on log prices: multiplying every price by a constant changes nothing
    for c in (1e-3, 7.0, 1e4):
        assert O.catalog_cut([c * x for x in w]) == 3
    # ... while an additive shift changes the multiplicative separation.  By hand, with x = log(w + 1000)
    # relative to the first: (0, 0, 0, .0197, .0534, .1042) -> scores k=3: .00361, k=4: .00158, k=5: .00217
    assert O.catalog_cut([x + 1000.0 for x in w]) == 4


def test_cut_ties_go_to_the_smallest_k_and_small_cases():
    assert O.catalog_cut([1.0, 10.0]) == 1                       # the only possible cut
    # geometric progression of three: cutting after 1 or after 2 disperses the same -> k = 1
    assert O.catalog_cut([1.0, 4.0, 16.0]) == 1
    # closed form for B = 3: score(k=1) = (x3-x2)^2/2, score(k=2) = (x2-x1)^2/2
    assert O.catalog_cut([1.0, 2.0, 16.0]) == 2 and O.catalog_cut([1.0, 8.0, 16.0]) == 1
    with pytest.raises(ValueError):
        O.catalog_cut([2.0, 1.0])


def test_cut_equals_exhaustive_two_class_variance():
    # the same objective written with numpy's variance: score(k) = k * var(left) + (B - k) * var(right)
    rng = np.random.RandomState(3)
    for _ in range(200):
        B = int(rng.randint(2, 12))
        w = np.sort(np.exp(rng.uniform(-3, 6, size=B)))
        x = np.log(w)
        scores = [k * x[:k].var() + (B - k) * x[k:].var() for k in range(1, B)]
        assert O.catalog_cut(list(w)) == 1 + int(np.argmin(scores))


def test_filler_packing_worked_example():
    # two ranks, F = 10, M_cap = 100.  Anchors left loads (6, 2) and memory (50, 20).
    # fillers by price: 3 (mem 10), 2 (mem 40), 1 (mem 10)
    #  p=3: rank0 min((10-6-3)/10, (50-10)/100) = 0.1 ; rank1 min((10-2-3)/10, (80-10)/100) = 0.5 -> rank 1
    #  p=2: rank0 min(0.2, 0.1) = 0.1 ; rank1 (C=5, M=30): min(0.3, 0.3) = 0.3 -> rank 1
    #  p=1: rank0 min(0.3, 0.4) = 0.3 ; rank1 (C=7, M=70): min(0.2, 0.2) = 0.2 -> rank 0
    out = O.filler_packing([1.0, 3.0, 2.0], [[10, 10], [10, 10], [40, 40]], [6.0, 2.0], [50.0, 20.0], 100.0, 10.0)
    assert out == [0, 1, 1]
    # memory decides feasibility: a filler that fits nowhere fails the plan
    assert O.filler_packing([1.0], [[60, 90]], [0.0, 0.0], [50.0, 20.0], 100.0, 10.0) is None
    assert O.filler_packing([1.0], [[60, 80]], [0.0, 0.0], [50.0, 20.0], 100.0, 10.0) == [1]
    # equal scores go to the lowest rank; equal prices keep input order
    assert O.filler_packing([1.0, 1.0], [[1, 1], [1, 1]], [0.0, 0.0], [0.0, 0.0], 100.0, 10.0) == [0, 1]


def test_filler_packing_balances_identical_fillers():
    # 50 identical images over 4 empty ranks with ample memory end up 13/13/12/12
    out = O.filler_packing([0.08] * 50, [[1.0] * 4] * 50, [0.0] * 4, [0.0] * 4, 1e3, 0.08 * 50 / 4)
    assert sorted(np.bincount(out, minlength=4).tolist()) == [12, 12, 13, 13]


# ---------------------------------------------------------------------------------------- implementation vs oracle
def test_numpy_cut_matches_oracle():
    rng = np.random.RandomState(11)
    for _ in range(500):
        B = int(rng.randint(2, 40))
        w = np.sort(np.exp(rng.uniform(-4, 7, size=B)))
        assert P.catalog_cut(w) == O.catalog_cut(list(w))
    assert P.catalog_cut([1.0, 4.0, 16.0]) == 1
    with pytest.raises(ValueError):
        P.catalog_cut([3.0])


def test_numpy_filler_packing_matches_oracle():
    rng = np.random.RandomState(12)
    for _ in range(300):
        n, R = int(rng.randint(1, 30)), int(rng.randint(1, 9))
        prices = rng.choice([0.05, 0.08, 0.3, 1.0], size=n) * rng.uniform(0.9, 1.1, size=n)
        fmem = rng.uniform(0.5, 6.0, size=(n, R))
        load, mem = rng.uniform(0, 3, size=R), rng.uniform(0, 20, size=R)
        cap = float(rng.uniform(15, 60))
        floor = float((prices.sum() + load.sum()) / R)
        a = P.filler_packing(prices, fmem, load, mem, cap, floor)
        b = O.filler_packing(list(prices), fmem.tolist(), list(load), list(mem), cap, floor)
        assert a == b


def test_measured_prices_put_images_with_the_fillers():
    # whole-sequence prices measured on a B200 by the profiler (12 heads, d=128), ms
    whole = {"image_480p": 0.077, "video_480p": 20.328, "video_720p": 110.545}
    fillers, anchors = P.split_catalog(whole)
    assert fillers == ["image_480p"] and anchors == ["video_480p", "video_720p"]
