"""Fusion of local chunks (zl_build_tasks_ex with ZL_BUILD_FUSE_LOCAL_CHUNKS): a shard query range
whose key chunks tile one contiguous interval runs as one task over the interval, without partials
and without the merge.  The result is the same exact attention over the union of the chunks
(paper Section II-B), so it is checked against the same fp64 oracle values as the unfused path, and
against the unfused GPU results."""
import numpy as np
import pytest
import torch

import zl_workloads as W
from oracle import attention as orc
from zl_testlib import EngineRun, SENTINEL, bits, check_backward, check_forward, dev_to_f64, to_dev, to_f64

pytestmark = pytest.mark.gpu

FUSE = 1  # ZL_BUILD_FUSE_LOCAL_CHUNKS


def _run_both(p):
    hb = {t: bits(p, t) for t in ("Q", "K", "V", "dO")}
    Q, K, V, dO = (to_dev(hb[t]) for t in ("Q", "K", "V", "dO"))
    f = {t: to_f64(hb[t]) for t in hb}
    ref = orc.placement_fwd(p, f["Q"], f["K"], f["V"])
    gref = orc.placement_bwd(p, f["Q"], f["K"], f["V"], f["dO"])
    out = {}
    for name, flags in (("plain", 0), ("fused", FUSE)):
        run = EngineRun(p, flags=flags)
        O, LSE, OP, LP = run.forward(Q, K, V)
        check_forward(p, O, LSE, ref)
        dQ, dK, dV = run.backward(Q, K, V, O, LSE, dO)
        check_backward(p, dQ, dK, dV, gref)
        out[name] = (run, O, LSE, OP, dQ, dK, dV)
    return out


def test_fused_config1_matches_oracle_and_unfused():
    out = _run_both(W.config(1))
    run_f, O_f, LSE_f, OP_f = out["fused"][:4]
    run_p, O_p, LSE_p = out["plain"][:3]
    assert run_f.info.n_fused_ranges == 2 and run_f.info.partial_rows == 0 and run_f.info.n_merge_groups == 0
    assert run_p.info.n_fused_ranges == 0 and run_p.info.partial_rows > 0
    # no partial is written in fused mode (the dummy one-row buffer keeps its sentinel)
    assert torch.all(OP_f == SENTINEL)
    # both are exact attention over the same key rows, rounded differently
    assert float((O_f.float() - O_p.float()).abs().max()) <= 2e-2
    assert float((LSE_f - LSE_p).abs().max()) <= 1e-4


def test_fused_ragged_ranges_sharing_chunks():
    # an image, then two ragged query ranges over the same three ragged chunks (several tiles, ragged tails)
    shards = [(70, 150, 70, 129, 0), (70, 150, 199, 300, 0), (70, 150, 499, 77, 0),
              (220, 131, 70, 129, 1), (220, 131, 199, 300, 1), (220, 131, 499, 77, 1)]
    p = W.custom_placement("fused_ragged", 2, 64, 11, [0, 70], shards, 351, 576)
    out = _run_both(p)
    assert out["fused"][0].info.n_fused_ranges == 2
    assert out["fused"][0].info.n_tasks == 3 and out["plain"][0].info.n_tasks == 7


def test_fusion_falls_back_when_ranges_disagree():
    # the second query range uses two of the three chunks: nothing is fused, results as before
    shards = [(0, 140, 0, 128, 0), (0, 140, 128, 128, 0), (0, 140, 256, 60, 0),
              (140, 40, 0, 128, 1), (140, 40, 128, 128, 1)]
    p = W.custom_placement("fallback", 1, 128, 12, [0], shards, 180, 316)
    out = _run_both(p)
    assert out["fused"][0].info.n_fused_ranges == 0
    assert torch.equal(out["fused"][1], out["plain"][1]) and torch.equal(out["fused"][2], out["plain"][2])
