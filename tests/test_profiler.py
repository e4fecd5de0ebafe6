"""The hardware profiler (paper Section IV-B: additive per-rank prices P[b, theta]; Section V-B: how well
their sum predicts a measured step).  Host logic with a synthetic timer, and one small run on the GPU."""
import numpy as np
import pytest

from paper_2608_01150_b200 import profiler as P


def test_placement_of_is_a_valid_placement():
    import paper_2608_01150_b200 as Z
    segs = [P.Segment("img", 300, 1), P.Segment("vid", 1000, 4), P.Segment("img", 300, 1), P.Segment("vid2", 515, 2)]
    cu, shards, tq, tkv = P.placement_of(segs)
    assert cu == [0, 300, 600]
    # one query chunk per sharded segment, `degree` key chunks each, in disjoint row ranges
    assert [s[:4] for s in shards[:4]] == [(600, 250, 600 + 250 * k, 250) for k in range(4)]
    assert [s[:4] for s in shards[4:]] == [(850, 258, 1600 + 258 * k, 258) for k in range(2)]
    assert (tq, tkv) == (600 + 250 + 258, 600 + 1000 + 516)
    h = Z.build_tasks(cu, shards, tq, tkv, 2, 64)          # accepted by the host validation
    assert h.info.n_tasks == 2 + 4 + 2 and h.info.n_merge_groups == 2


def test_prices_and_additivity_with_a_synthetic_timer():
    # a machine whose step time is exactly a constant plus a per-segment cost: the profile must recover the
    # costs and predict every plan exactly
    c0 = 0.25
    cost = lambda s: 1e-6 * s.tokens * s.chunk()
    measure = lambda segs: c0 + sum(cost(s) for s in segs if s.bucket != "floor") + (1e-6 * 128 * 128 if any(s.bucket == "floor" for s in segs) else 0.0)
    prices, step_cost = P.profile_prices(measure)
    assert abs(step_cost - (c0 + 1e-6 * 128 * 128)) < 1e-12
    for name, tokens in P.BUCKETS.items():
        for k in P.DEGREES:
            assert prices[f"{name}@{k}"] == pytest.approx(cost(P.Segment(name, tokens, k)) - 1e-6 * 128 * 128, rel=1e-9)
    plans = P.rotation_plans()
    rep = P.check_additivity(measure, prices, step_cost, plans)
    # the only mismatch is the floor sequence's own work, which every price gives up once
    assert rep["mape_pct"] < 0.5
    # every (video bucket, degree) pair occurs in some plan
    seen = {x for r in rep["plans"] for x in r["plan"]}
    for name in P.BUCKETS:
        if not name.startswith("image"):
            assert {f"{name}@{k}" for k in P.DEGREES} <= seen
    assert P.mape([(110.0, 100.0), (90.0, 100.0)]) == pytest.approx(10.0)


@pytest.mark.gpu
def test_profile_small_buckets_on_gpu():
    buckets = {"image_s": 300, "video_a": 2048, "video_b": 4096}
    measure = P.gpu_timer(2, 64, steps=3, warmup=1)
    prices, step_cost = P.profile_prices(measure, buckets, (1, 2, 4))
    assert step_cost > 0 and all(np.isfinite(v) and v >= 0 for v in prices.values())
    assert len(prices) == 8          # 300 tokens at degree 4 would be chunks below one tile: not profiled
    rep = P.check_additivity(measure, prices, step_cost, P.rotation_plans(buckets, (1, 2, 4), n_images=4))
    assert len(rep["plans"]) >= 4 and np.isfinite(rep["mape_pct"])
    # tiny sequences are dominated by launch and tail effects: the check is that the model is sane, not tight
    assert rep["mape_pct"] < 60.0
