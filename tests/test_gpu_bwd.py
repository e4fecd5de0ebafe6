"""GPU parity of zl_coalesced_attn_bwd against the fp64 CPU oracle's analytic gradients."""
import numpy as np
import pytest
import torch

import zl_workloads as W
from oracle import attention as A
from zl_testlib import (EngineRun, bits, check_backward, check_forward, dev_to_f64, random_bits, to_dev,
                        to_f64, GATE_GRAD_REL, SENTINEL)

pytestmark = pytest.mark.gpu


def _run(p, Qb, Kb, Vb, dOb, gate=True):
    run = EngineRun(p)
    Qd, Kd, Vd, dOd = (to_dev(x) for x in (Qb, Kb, Vb, dOb))
    O, LSE, _, _ = run.forward(Qd, Kd, Vd)
    dQ, dK, dV = run.backward(Qd, Kd, Vd, O, LSE, dOd)
    ref = A.placement_bwd(p, to_f64(Qb), to_f64(Kb), to_f64(Vb), to_f64(dOb))
    stats = check_backward(p, dQ, dK, dV, ref)
    if gate:
        assert max(stats[k] for k in ("dQ", "dK", "dV")) <= GATE_GRAD_REL, stats
    return run, (dQ, dK, dV), ref, stats


def test_config1_backward():
    """Config 1 is the case where two shard tasks share a key range (dK/dV summed across
    tasks without atomics) and two share a query range (dQ summed)."""
    p = W.config(1)
    _run(p, bits(p, "Q"), bits(p, "K"), bits(p, "V"), bits(p, "dO"))


EDGE = [1, 2, 15, 16, 17, 127, 128, 129, 255, 256, 257]


@pytest.mark.parametrize("d,H", [(64, 1), (128, 3)])
def test_tile_edge_lengths_whole(d, H):
    p = W.make_placement("edges", H, d, 11, EDGE + [24 + 128, 16 + 256, 126, 106 + 128, 6, 104])
    rng = np.random.RandomState(d + H)
    Qb, Kb, Vb, dOb = (random_bits(rng, p.total_q, H, d) for _ in range(4))
    _run(p, Qb, Kb, Vb, dOb)


@pytest.mark.parametrize("lq,lkv", [(1, 1), (1, 257), (257, 1), (129, 127), (17, 255), (130, 300)])
def test_tile_edge_lengths_shards(lq, lkv):
    d, H = 128, 2
    p = W.custom_placement("edge_shard", H, d, 5, [0, 40], [(40, lq, 40, lkv, 0), (40, lq, 40 + lkv, 3, 0)],
                           40 + lq + 5, 40 + lkv + 3 + 7)
    rng = np.random.RandomState(lq * 1000 + lkv)
    Qb, dOb = random_bits(rng, p.total_q, H, d), random_bits(rng, p.total_q, H, d)
    Kb, Vb = random_bits(rng, p.total_kv, H, d), random_bits(rng, p.total_kv, H, d)
    _run(p, Qb, Kb, Vb, dOb)


def test_backward_sum_identities_on_gpu_outputs():
    """sum_j dV_j = sum_i dO_i and sum_j dK_j = 0 over each sequence, evaluated on GPU outputs."""
    d, H = 128, 2
    p = W.make_placement("ident", H, d, 1, [300, 77])
    rng = np.random.RandomState(3)
    Qb, Kb, Vb, dOb = (random_bits(rng, p.total_q, H, d) for _ in range(4))
    _, (dQ, dK, dV), _, _ = _run(p, Qb, Kb, Vb, dOb)
    dOf = to_f64(dOb)
    for (a, b) in [(0, 300), (300, 377)]:
        sv = dev_to_f64(dV)[a:b].sum(0)
        so = dOf[a:b].sum(0)
        assert np.abs(sv - so).max() < 0.05 * np.sqrt(b - a)
        assert np.abs(dev_to_f64(dK)[a:b].sum(0)).max() < 0.05 * np.sqrt(b - a)


def test_isolation_with_finite_poison_in_neighbours():
    d, H = 64, 2
    p = W.custom_placement("iso", H, d, 1, [0, 100, 230], [(240, 50, 240, 70, 0)], 300, 320)
    rng = np.random.RandomState(2)
    Qb, dOb = random_bits(rng, 300, H, d), random_bits(rng, 300, H, d)
    Kb, Vb = random_bits(rng, 320, H, d), random_bits(rng, 320, H, d)
    run, (dQ1, dK1, dV1), _, _ = _run(p, Qb, Kb, Vb, dOb)
    big = W.f32_to_bf16_bits(np.full((1,), 3e38, dtype=np.float32))[0]
    Q2, K2, V2, dO2 = Qb.copy(), Kb.copy(), Vb.copy(), dOb.copy()
    Q2[230:240] = big; dO2[230:240] = big; K2[230:240] = big; V2[230:240] = big   # rows no task owns
    Q2[290:] = big; dO2[290:] = big; K2[310:] = big; V2[310:] = big
    run2 = EngineRun(p)
    Qd, Kd, Vd, dOd = (to_dev(x) for x in (Q2, K2, V2, dO2))
    O, LSE, _, _ = run2.forward(Qd, Kd, Vd)
    dQ2, dK2, dV2 = run2.backward(Qd, Kd, Vd, O, LSE, dOd)
    qkeep = np.r_[0:230, 240:290]
    kkeep = np.r_[0:230, 240:310]
    # dK/dV are bit-deterministic; dQ is accumulated with reductions whose order may vary
    assert torch.equal(dK1[kkeep], dK2[kkeep]) and torch.equal(dV1[kkeep], dV2[kkeep])
    assert torch.allclose(dQ1[qkeep].float(), dQ2[qkeep].float(), atol=2e-2, rtol=2e-2)
    assert torch.all(dQ2[230:240] == SENTINEL) and torch.all(dK2[310:] == SENTINEL)


def test_empty_kv_shard_gives_zero_dq():
    d, H = 64, 1
    p = W.custom_placement("empty", H, d, 1, [0, 10], [(10, 20, 10, 0, 0), (30, 5, 10, 33, 1)], 40, 50)
    rng = np.random.RandomState(4)
    Qb, dOb = random_bits(rng, 40, H, d), random_bits(rng, 40, H, d)
    Kb, Vb = random_bits(rng, 50, H, d), random_bits(rng, 50, H, d)
    _, (dQ, dK, dV), _, _ = _run(p, Qb, Kb, Vb, dOb)
    assert torch.all(dQ[10:30] == 0)


def test_randomised_small_placements():
    rng = np.random.RandomState(4321)
    for trial in range(6):
        d = int(rng.choice([64, 128]))
        H = int(rng.randint(1, 4))
        p = W.random_placement(rng, H, d)
        Qb, dOb = random_bits(rng, p.total_q, H, d), random_bits(rng, p.total_q, H, d)
        Kb, Vb = random_bits(rng, p.total_kv, H, d), random_bits(rng, p.total_kv, H, d)
        _run(p, Qb, Kb, Vb, dOb)
