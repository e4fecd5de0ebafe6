"""The CTA-pair form of the backward main kernel (zl_set_bwd_kernel(tasks, 2): tcgen05 cta_group::2, two key
tiles per pair of CTAs, dS exchanged inside the pair, dQ summed over 256 keys before the reduce) against the
fp64 oracle and against the one-CTA kernel."""
import numpy as np
import pytest
import torch

import zl_workloads as W
from oracle import attention as A
from zl_testlib import (EngineRun, bits, check_backward, dev_to_f64, random_bits, rel_fro, to_dev, to_f64, GATE_GRAD_REL,
                        SENTINEL)

pytestmark = pytest.mark.gpu

EDGE = [1, 2, 15, 16, 17, 127, 128, 129, 255, 256, 257, 383, 384, 385, 511, 512, 513]


def _both(p, seed):
    rng = np.random.RandomState(seed)
    H, d = p.n_heads, p.head_dim
    Qb, dOb = random_bits(rng, p.total_q, H, d), random_bits(rng, p.total_q, H, d)
    Kb, Vb = random_bits(rng, p.total_kv, H, d), random_bits(rng, p.total_kv, H, d)
    run = EngineRun(p)
    Qd, Kd, Vd, dOd = (to_dev(x) for x in (Qb, Kb, Vb, dOb))
    O, LSE, _, _ = run.forward(Qd, Kd, Vd)
    out = {}
    for kernel in (1, 2):
        run.h.set_bwd_kernel(kernel)
        out[kernel] = run.backward(Qd, Kd, Vd, O, LSE, dOd)
    ref = A.placement_bwd(p, to_f64(Qb), to_f64(Kb), to_f64(Vb), to_f64(dOb))
    stats = check_backward(p, *out[2], ref)       # includes: rows no task covers keep the sentinel
    assert max(stats[k] for k in ("dQ", "dK", "dV")) <= GATE_GRAD_REL, stats
    # same products in the same order: dK and dV agree bit for bit with the one-CTA kernel; dQ up to the fp32 adds
    assert torch.equal(out[1][1], out[2][1]) and torch.equal(out[1][2], out[2][2])
    assert rel_fro(dev_to_f64(out[2][0]), dev_to_f64(out[1][0])) <= 1e-3
    return stats


def test_pair_kernel_tile_edge_lengths():
    """Key ranges with one tile, an odd number of tiles, a ragged second tile, and several items per pair."""
    p = W.make_placement("edges", 3, 128, 11, EDGE + [24 + 128, 16 + 256, 126, 106 + 128, 6, 104])
    _both(p, 61)


def test_pair_kernel_shards_sharing_key_and_query_ranges():
    """2 x 2 chunk tasks (dK/dV summed over two query chunks inside one item, dQ summed over two key chunks) next to
    whole sequences; head_dim 128."""
    p = W.make_placement("cp", 2, 128, 12, [300, 77], [(2, 2, 330), (1, 3, 200)])
    _both(p, 62)


def test_pair_kernel_head_ranges():
    p = W.ulysses_mix_placement(n_heads=4, head_dim=128, n_images=2, image_len=700, seq_len=900, degree=2)
    _both(p, 63)


def test_pair_kernel_is_refused_for_head_dim_64():
    import paper_2608_01150_b200 as Z
    p = W.config(1)
    run = EngineRun(p)
    with pytest.raises(Z.ZlError) as e:
        run.h.set_bwd_kernel(2)
    assert e.value.status == 3      # ZL_ERR_UNSUPPORTED


@pytest.mark.slow
def test_pair_kernel_on_the_image_batch_configuration():
    """Configuration 2 in full (12 heads, 36 whole sequences): every row and column against the oracle."""
    import test_gpu_configs as C
    p = W.config(2)
    B = C._inputs(p)
    d = C._device_tensors(p, B)
    run = EngineRun(p)
    run.h.set_bwd_kernel(2)
    O, LSE, _, _ = run.forward(d["Q"], d["K"], d["V"])
    dQ, dK, dV = run.backward(d["Q"], d["K"], d["V"], O, LSE, d["dO"])
    src = {t: C._head_src(B, t) for t in B}
    ref_b = A.placement_bwd(p, src["Q"], src["K"], src["V"], src["dO"])
    print("config 2, pair kernel:", check_backward(p, dQ, dK, dV, ref_b))
