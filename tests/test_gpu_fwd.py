"""GPU parity of the forward path (zl_coalesced_attn_fwd + zl_lse_merge) against the fp64
CPU oracle, called through the C ABI via the Python binding."""
import numpy as np
import pytest
import torch

import zl_workloads as W
from oracle import attention as A
from zl_testlib import (EngineRun, bits, check_forward, dev_to_f64, random_bits, to_dev, to_f64,
                        GATE_O_MAX, GATE_LSE_MAX, SENTINEL)

pytestmark = pytest.mark.gpu


def _run(p, Qb, Kb, Vb, gate=True):
    run = EngineRun(p)
    O, LSE, OP, LP = run.forward(to_dev(Qb), to_dev(Kb), to_dev(Vb))
    ref = A.placement_fwd(p, to_f64(Qb), to_f64(Kb), to_f64(Vb))
    stats = check_forward(p, O, LSE, ref)
    if gate:
        assert stats["o_excess"] <= GATE_O_MAX and stats["lse_max"] <= GATE_LSE_MAX, stats
    return run, (O, LSE, OP, LP), ref, stats


def test_config1_forward_and_partials():
    p = W.config(1)
    Qb, Kb, Vb = bits(p, "Q"), bits(p, "K"), bits(p, "V")
    run, (O, LSE, OP, LP), ref, stats = _run(p, Qb, Kb, Vb)
    # per-task partials: normalised within their own K/V chunk
    OPh, LPh = dev_to_f64(OP), dev_to_f64(LP)
    for si, s in enumerate(p.shards):
        off, padded = run.h.partial_slot(si)
        assert padded == 1024
        o_t, l_t = ref["partials"][si]
        assert np.abs(OPh[off:off + s[1]] - o_t).max() <= GATE_O_MAX
        assert np.abs(LPh[:, off:off + s[1]] - l_t).max() <= GATE_LSE_MAX


EDGE = [1, 2, 15, 16, 17, 127, 128, 129, 255, 256, 257]


@pytest.mark.parametrize("d,H", [(64, 1), (128, 3)])
def test_tile_edge_lengths_whole(d, H):
    """Whole sequences whose lengths straddle every tile edge, packed in one launch."""
    p = W.make_placement("edges", H, d, 11, EDGE + [24 + 128, 16 + 256, 126, 106 + 128, 6, 104])
    rng = np.random.RandomState(d + H)
    Qb, Kb, Vb = (random_bits(rng, p.total_q, H, d) for _ in range(3))
    _run(p, Qb, Kb, Vb)


@pytest.mark.parametrize("lq,lkv", [(1, 1), (1, 257), (257, 1), (129, 127), (17, 255), (130, 300)])
def test_tile_edge_lengths_shards(lq, lkv):
    d, H = 128, 2
    p = W.custom_placement("edge_shard", H, d, 5, [0, 40], [(40, lq, 40, lkv, 0), (40, lq, 40 + lkv, 3, 0)],
                           40 + lq + 5, 40 + lkv + 3 + 7)
    rng = np.random.RandomState(lq * 1000 + lkv)
    Qb = random_bits(rng, p.total_q, H, d)
    Kb = random_bits(rng, p.total_kv, H, d)
    Vb = random_bits(rng, p.total_kv, H, d)
    _run(p, Qb, Kb, Vb)


def test_spike_keys_at_tile_and_chunk_boundaries():
    """A key aligned with a query makes that query's output equal that key's value row, so
    a dropped, duplicated or leaked key is an O(1) error.  Keys of the NEIGHBOURING sequences (the
    previous one's last key, the next one's first key) aligned with queries of this sequence must
    have no effect at all."""
    d, H = 128, 1
    p = W.make_placement("spike", H, d, 3, [300, 200, 150], [(1, 2, 260)])
    rng = np.random.RandomState(9)
    Q = rng.standard_normal((p.total_q, H, d)).astype(np.float32)
    K = rng.standard_normal((p.total_kv, H, d)).astype(np.float32) * 0.1
    V = rng.standard_normal((p.total_kv, H, d)).astype(np.float32)
    beta = 4.0
    # (query row, key row) pairs inside the same logical problem
    pairs = [(0, 0), (5, 127), (6, 128), (7, 255), (8, 256), (9, 298),           # whole seq 0 (rows 0-299)
             (300, 300), (301, 498),                                              # whole seq 1 (rows 300-499)
             (505, 501), (506, 649),                                              # whole seq 2 (rows 500-649)
             (650, 650), (651, 777), (652, 778), (653, 909), (654, 910), (655, 1169)]  # shard chunks
    # (query row, key row of a NEIGHBOUR): seq 0's last key and seq 2's first key aligned with queries of
    # seq 1, seq 1's last key aligned with a query of seq 2
    foreign = [(310, 299), (311, 500), (510, 499)]
    for qi, kj in pairs + foreign:
        K[kj] = beta * Q[qi]
    Qb, Kb, Vb = (W.f32_to_bf16_bits(W._bf16_round_f32(x)) for x in (Q, K, V))
    run, (O, LSE, OP, LP), ref, stats = _run(p, Qb, Kb, Vb, gate=False)
    Og = dev_to_f64(O)
    Vf = to_f64(Vb)
    for qi, kj in pairs:
        assert np.abs(ref["O"][qi, 0] - Vf[kj, 0]).max() < 1e-6, "spike too weak for the test"
        assert np.abs(Og[qi, 0] - Vf[kj, 0]).max() < 2e-2, (qi, kj)
    for qi, kj in foreign:
        # had the foreign key leaked into the row's softmax, the row would equal its value row
        assert np.abs(ref["O"][qi, 0] - Vf[kj, 0]).max() > 0.5
        assert np.abs(Og[qi, 0] - ref["O"][qi, 0]).max() < 2e-2, (qi, kj)
        assert np.abs(Og[qi, 0] - Vf[kj, 0]).max() > 0.5, (qi, kj)


def test_isolation_and_untouched_rows():
    """Perturbing one sequence leaves every other sequence's output bit-identical, and rows
    that belong to no task keep their previous contents."""
    d, H = 64, 2
    p = W.custom_placement("iso", H, d, 1, [0, 100, 230], [(240, 50, 240, 70, 0)], 300, 320)
    rng = np.random.RandomState(2)
    Qb, Kb, Vb = random_bits(rng, 300, H, d), random_bits(rng, 320, H, d), random_bits(rng, 320, H, d)
    run, (O1, L1, _, _), ref, _ = _run(p, Qb, Kb, Vb)
    Q2, K2, V2 = Qb.copy(), Kb.copy(), Vb.copy()
    big = W.f32_to_bf16_bits(np.full((1,), 3e38, dtype=np.float32))[0]
    K2[100:230] = big                     # large finite poison in sequence 1
    V2[100:230] = big
    K2[230:240] = big                     # and in rows no task owns
    run2 = EngineRun(p)
    O2, L2, _, _ = run2.forward(to_dev(Q2), to_dev(K2), to_dev(V2))
    keep = np.r_[0:100, 240:290]
    assert torch.equal(O1[keep], O2[keep]) and torch.equal(L1[:, keep], L2[:, keep])
    assert torch.all(O2[290:] == SENTINEL) and torch.all(O2[230:240] == SENTINEL)


def test_forward_is_run_to_run_bit_identical():
    p = W.config(1)
    Qd, Kd, Vd = to_dev(bits(p, "Q")), to_dev(bits(p, "K")), to_dev(bits(p, "V"))
    run = EngineRun(p)
    a = run.forward(Qd, Kd, Vd)
    b = run.forward(Qd, Kd, Vd)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_empty_kv_shard_and_single_part_group():
    d, H = 64, 1
    p = W.custom_placement("empty", H, d, 1, [0, 10], [(10, 20, 10, 0, 0), (30, 5, 10, 33, 1)], 40, 50)
    rng = np.random.RandomState(4)
    Qb, Kb, Vb = random_bits(rng, 40, H, d), random_bits(rng, 50, H, d), random_bits(rng, 50, H, d)
    run, (O, LSE, _, _), ref, _ = _run(p, Qb, Kb, Vb)
    assert torch.all(O[10:30] == 0) and torch.all(torch.isneginf(LSE[:, 10:30]))


def test_randomised_small_placements():
    rng = np.random.RandomState(1234)
    for trial in range(6):
        d = int(rng.choice([64, 128]))
        H = int(rng.randint(1, 4))
        p = W.random_placement(rng, H, d)
        Qb = random_bits(rng, p.total_q, H, d)
        Kb = random_bits(rng, p.total_kv, H, d)
        Vb = random_bits(rng, p.total_kv, H, d)
        _run(p, Qb, Kb, Vb)


def test_bounded_wait_expires_and_is_reported():
    """A wait nobody satisfies returns after its limit, reports ZL_ERR_TIMEOUT through the device status
    word and leaves the context usable (no trap, no hang)."""
    p = W.config(1)
    run = EngineRun(p)
    run.h.selftest_bounded_wait(limit_us=500)
    torch.cuda.synchronize()
    code, where = run.h.last_device_status()
    assert (code, where) == (6, 9001)            # ZL_ERR_TIMEOUT at the self-test site
    assert run.h.last_device_status() == (0, 0)  # reading clears the word
    Qd, Kd, Vd = to_dev(bits(p, "Q")), to_dev(bits(p, "K")), to_dev(bits(p, "V"))
    O, LSE, _, _ = run.forward(Qd, Kd, Vd)       # the same handle and context still work
    assert torch.isfinite(O.float()).all()


def test_results_do_not_depend_on_the_work_order():
    p = W.make_placement("order", 2, 128, 5, [700, 130, 1000], [(1, 2, 300)])
    rng = np.random.RandomState(8)
    Qd = to_dev(random_bits(rng, p.total_q, 2, 128)); Kd = to_dev(random_bits(rng, p.total_kv, 2, 128))
    Vd = to_dev(random_bits(rng, p.total_kv, 2, 128))
    run = EngineRun(p)
    ref = run.forward(Qd, Kd, Vd)
    for mode in (1, 2, 0):
        run.h.set_fwd_order(mode)
        out = run.forward(Qd, Kd, Vd)
        assert torch.equal(out[0], ref[0]) and torch.equal(out[1], ref[1])
