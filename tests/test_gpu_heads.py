"""GPU parity for placements whose tasks cover different head ranges (zl_build_tasks_heads): whole
sequences over all heads next to Ulysses-shaped sequences over a subset of the heads, in one launch
and one set of buffers (the engine's second coalescing mode)."""
import numpy as np
import pytest
import torch

import zl_workloads as W
from oracle import attention as A
from zl_testlib import (EngineRun, SENTINEL, bits, check_backward, check_forward, covered_rows, dev_to_f64, random_bits,
                        to_dev, to_f64, GATE_GRAD_REL, GATE_LSE_MAX, GATE_O_MAX)

pytestmark = pytest.mark.gpu


def _run(p, seed):
    rng = np.random.RandomState(seed)
    H, d = p.n_heads, p.head_dim
    Qb, dOb = random_bits(rng, p.total_q, H, d), random_bits(rng, p.total_q, H, d)
    Kb, Vb = random_bits(rng, p.total_kv, H, d), random_bits(rng, p.total_kv, H, d)
    run = EngineRun(p)
    Qd, Kd, Vd, dOd = (to_dev(x) for x in (Qb, Kb, Vb, dOb))
    O, LSE, _, _ = run.forward(Qd, Kd, Vd)
    dQ, dK, dV = run.backward(Qd, Kd, Vd, O, LSE, dOd)
    ref_f = A.placement_fwd(p, to_f64(Qb), to_f64(Kb), to_f64(Vb))
    ref_b = A.placement_bwd(p, to_f64(Qb), to_f64(Kb), to_f64(Vb), to_f64(dOb))
    fs = check_forward(p, O, LSE, ref_f)       # includes: (row, head) pairs no task covers keep the sentinel
    bs = check_backward(p, dQ, dK, dV, ref_b)
    assert fs["o_excess"] <= GATE_O_MAX and fs["lse_max"] <= GATE_LSE_MAX, fs
    assert max(bs[k] for k in ("dQ", "dK", "dV")) <= GATE_GRAD_REL, bs
    return run, (O, LSE, dQ, dK, dV), fs, bs


def test_whole_images_next_to_two_ulysses_sequences():
    """H = 12: six whole images over 12 heads + two sequences over heads [0,6) and [6,12) that share one
    block of rows (what decides isolation here is the oracle: each head of those rows belongs to a
    different sequence)."""
    p = W.ulysses_mix_placement(n_heads=12, head_dim=128, n_images=6, image_len=1560, seq_len=3600, degree=2)
    run, _, fs, bs = _run(p, 31)
    assert run.info.n_tasks == 8
    print("ulysses mix:", fs, bs)


def test_partial_head_coverage_leaves_other_heads_untouched():
    """A sequence over heads [1,3) of 4: heads 0 and 3 of its rows belong to no task and must keep their
    previous contents in O, LSE, dQ, dK and dV; ragged lengths."""
    whole = [(0, 130, 0, 4), (130, 257, 1, 2), (387, 77, 0, 1), (387, 77, 2, 2)]
    p = W.head_range_placement("partial", 4, 64, 5, whole, [], 470, 470)
    qmask, kvmask = covered_rows(p)
    assert (~qmask).sum() == 257 * 2 + 6 * 4 + 77     # heads 0,3 of seq 1; the uncovered tail rows; head 1 of the last block
    _run(p, 32)


def test_shard_groups_with_head_ranges_merge_and_backward():
    """One query range served on heads [0,2) by two K/V chunks and on heads [2,4) by three other chunks of
    the same rows: merge groups, kv groups and dQ accumulation are per (range, head range)."""
    whole = [(0, 100, 0, 4)]
    shards = [(100, 150, 100, 70, 0, 0, 2), (100, 150, 170, 200, 0, 0, 2),
              (100, 150, 100, 129, 1, 2, 2), (100, 150, 229, 1, 1, 2, 2), (100, 150, 230, 140, 1, 2, 2)]
    p = W.head_range_placement("hr_shards", 4, 128, 6, whole, shards, 250, 370)
    run, _, _, _ = _run(p, 33)
    assert run.info.n_merge_groups == 2 and run.info.n_kv_groups == 6
    # the merge-free schedule gives the same results
    import paper_2608_01150_b200 as Z
    rng = np.random.RandomState(33)
    H, d = p.n_heads, p.head_dim
    Qb, dOb = random_bits(rng, p.total_q, H, d), random_bits(rng, p.total_q, H, d)
    Kb, Vb = random_bits(rng, p.total_kv, H, d), random_bits(rng, p.total_kv, H, d)
    runf = EngineRun(p, flags=Z.BUILD_FUSE_LOCAL_CHUNKS)
    assert runf.info.n_fused_ranges == 2 and runf.info.n_merge_groups == 0
    Qd, Kd, Vd, dOd = (to_dev(x) for x in (Qb, Kb, Vb, dOb))
    O, LSE, _, _ = runf.forward(Qd, Kd, Vd)
    dQ, dK, dV = runf.backward(Qd, Kd, Vd, O, LSE, dOd)
    check_forward(p, O, LSE, A.placement_fwd(p, to_f64(Qb), to_f64(Kb), to_f64(Vb)))
    check_backward(p, dQ, dK, dV, A.placement_bwd(p, to_f64(Qb), to_f64(Kb), to_f64(Vb), to_f64(dOb)))
