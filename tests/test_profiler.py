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


def test_catalog_covers_the_paper_buckets_and_plans():
    # 15 s of 1080p is the 497,760-token sequence of the paper's introduction
    assert P.CATALOG["video_1080p_15s"] == 497760 and P.CATALOG["video_480p_5s"] == 32760 and P.CATALOG["image_1080p"] == 8160
    assert len(P.CATALOG) == 4 + 9
    # synthetic machine: time = constant + pairs; profile, whole-sequence prices, catalog cut, covering plans
    measure = lambda segs: 0.05 + sum(1e-9 * s.tokens * s.chunk() for s in segs)
    prices, step = P.profile_prices(measure, P.CATALOG, P.CATALOG_DEGREES, P.MAX_PAIRS_PER_HEAD)
    assert "video_1080p_15s@1" not in prices and "video_1080p_15s@8" in prices and "image_256p@2" in prices
    assert "image_256p@4" not in prices                      # 64-token chunks: below one tile
    whole = P.whole_prices(prices, P.CATALOG)
    assert set(whole) == set(P.CATALOG)
    # the reconstruction k * P[b, k] recovers the whole-sequence cost where degree 1 was not profiled
    assert whole["video_1080p_15s"] == pytest.approx(1e-9 * 497760 ** 2, rel=1e-3)
    from paper_2608_01150_b200 import planner
    fillers, anchors = planner.split_catalog(whole)
    assert set(fillers) == {"image_256p", "image_480p", "image_720p", "image_1080p"}      # images vs videos
    plans = P.covering_plans(prices, P.CATALOG, n_images=50)
    seen = {f"{s.bucket}@{s.degree}" for plan in plans for s in plan}
    for v in ("video_480p_5s", "video_720p_5s", "video_1080p_5s"):
        assert {k for k in prices if k.startswith(v + "@")} <= seen
    assert sum(1 for plan in plans if all(s.degree == 1 for s in plan)) == 3    # the three all-whole corner plans
    rep = P.check_additivity(measure, prices, step, plans)
    assert rep["mape_pct"] < 0.1


@pytest.mark.gpu
def test_profile_medium_buckets_on_gpu():
    """Images of 1.5-4 K tokens and videos of 16-32 K tokens at 12 heads, d = 128: prices (small buckets priced
    from a batch that fills the GPU) predict mixed plans within 10 %, and the measured whole-sequence prices
    drive the catalog cut."""
    from paper_2608_01150_b200 import planner
    buckets = {"image_a": 1560, "image_b": 3600, "video_a": 16384, "video_b": 32760}
    measure = P.gpu_timer(12, 128, steps=5, warmup=2)
    prices, step_cost = P.profile_prices(measure, buckets, (1, 2, 4), fill_rows=P.FILL_ROWS)
    assert step_cost > 0 and all(np.isfinite(v) and v > 0 for v in prices.values()) and len(prices) == 12
    # prices grow with the rank's share of the work: L^2 / k
    for b in buckets:
        assert prices[f"{b}@1"] > prices[f"{b}@2"] > prices[f"{b}@4"]
    plans = P.rotation_plans({k: v for k, v in buckets.items() if k != "image_b"}, (1, 2, 4), n_images=16)
    rep = P.check_additivity(measure, prices, step_cost, plans)
    print("additivity:", [(r["plan"][:2], round(r["error_pct"], 2)) for r in rep["plans"]], rep["mape_pct"])
    assert rep["mape_pct"] <= 10.0, rep
    fillers, anchors = planner.split_catalog(P.whole_prices(prices, buckets))
    assert fillers == ["image_a", "image_b"] and anchors == ["video_a", "video_b"]
