"""GPU tests of launch phases (zl_set_fwd_phases / zl_set_bwd_phases): running a placement's tasks in several
launches, in the order their inputs arrive, must give what the single launch gives -- bit for bit in the forward
and for dK/dV, up to the order of the fp32 reduce-adds for dQ -- and must not touch inputs of later phases."""
import numpy as np
import pytest
import torch

import zl_workloads as W
from zl_testlib import SENTINEL, EngineRun, random_bits, to_dev

pytestmark = pytest.mark.gpu


def _placement():
    # four whole sequences (one ragged) + a context-parallel rank of degree 4: one 1000-token query chunk against
    # four 1000-token K/V chunks (1000 = 7 x 128 + 104: every chunk ends in a ragged tile whose load reaches
    # into the next chunk's rows)
    return W.make_placement("phases", 4, 128, 7, [300, 1560, 128, 777], [(1, 4, 1000)])


def _inputs(p, seed):
    rng = np.random.RandomState(seed)
    H, d = p.n_heads, p.head_dim
    return tuple(to_dev(random_bits(rng, n, H, d)) for n in (p.total_q, p.total_kv, p.total_kv, p.total_q))


def _buffers(p, info, dev):
    H, d = p.n_heads, p.head_dim
    O = torch.full((p.total_q, H, d), SENTINEL, dtype=torch.bfloat16, device=dev)
    LSE = torch.full((H, p.total_q), SENTINEL, dtype=torch.float32, device=dev)
    pr = max(1, int(info.partial_rows))
    OP = torch.full((pr, H, d), SENTINEL, dtype=torch.float32, device=dev)
    LP = torch.full((H, pr), SENTINEL, dtype=torch.float32, device=dev)
    return O, LSE, OP, LP


def _same_bits(a, b):
    return torch.equal(a.view(torch.int16 if a.dtype == torch.bfloat16 else torch.int32),
                       b.view(torch.int16 if b.dtype == torch.bfloat16 else torch.int32))


def test_forward_phases_match_single_launch_while_chunks_arrive():
    p = _placement()
    Q, K, V, _ = _inputs(p, 3)
    ref = EngineRun(p)
    O0, LSE0, OP0, LP0 = ref.forward(Q, K, V)

    run = EngineRun(p)
    Z, h = run.Z, run.h
    n_whole, n_shards = len(p.cu_seqlens) - 1, len(p.shards)
    # phase 0: whole sequences and the local chunk (chunk 0); phase j: the chunk that arrives at ring step j
    run.h.set_fwd_phases([0] * n_whole, list(range(n_shards)), n_shards)
    fi, _ = h.phase_info()
    assert len(fi) == 4 and sum(fi) == int(h.info.n_fwd_items) and all(x > 0 for x in fi)
    # K/V as they would be on a rank: zero-filled buffers, chunks copied in as they "arrive"
    Kt, Vt = torch.zeros_like(K), torch.zeros_like(V)
    whole_rows = p.cu_seqlens[-1]
    Kt[:whole_rows], Vt[:whole_rows] = K[:whole_rows], V[:whole_rows]
    O, LSE, OP, LP = _buffers(p, h.info, Q.device)
    for j, (_, _, ko, kl, _) in enumerate(p.shards):
        Kt[ko:ko + kl], Vt[ko:ko + kl] = K[ko:ko + kl], V[ko:ko + kl]
        Z.coalesced_attn_fwd_phase(h, j, Q, Kt, Vt, run.scale, O, LSE, OP, LP)
        torch.cuda.synchronize()
    Z.lse_merge(h, OP, LP, O, LSE)
    torch.cuda.synchronize()
    assert h.last_device_status()[0] == 0
    assert _same_bits(O, O0) and _same_bits(LSE, LSE0) and _same_bits(OP, OP0) and _same_bits(LP, LP0)


def test_forward_phases_in_reverse_order_and_one_launch_after_regrouping():
    p = _placement()
    Q, K, V, _ = _inputs(p, 4)
    O0, LSE0, _, _ = EngineRun(p).forward(Q, K, V)
    run = EngineRun(p)
    Z, h = run.Z, run.h
    run.h.set_fwd_phases([1, 0, 1, 0], [2, 0, 1, 2], 3)
    O, LSE, OP, LP = _buffers(p, h.info, Q.device)
    for ph in (2, 0, 1):
        Z.coalesced_attn_fwd_phase(h, ph, Q, K, V, run.scale, O, LSE, OP, LP)
    Z.lse_merge(h, OP, LP, O, LSE)
    torch.cuda.synchronize()
    assert _same_bits(O, O0) and _same_bits(LSE, LSE0)
    # the plain entry point still runs everything (the list is only regrouped)
    O1, LSE1, _, _ = run.forward(Q, K, V)
    assert _same_bits(O1, O0) and _same_bits(LSE1, LSE0)
    with pytest.raises(Z.ZlError):
        Z.coalesced_attn_fwd_phase(h, 3, Q, K, V, run.scale, O, LSE, OP, LP)


@pytest.mark.parametrize("kernel", [1, 2])
def test_backward_phases_remote_chunks_first(kernel):
    p = _placement()
    Q, K, V, dO = _inputs(p, 5)
    ref = EngineRun(p)
    ref.h.set_bwd_kernel(kernel)
    O, LSE, _, _ = ref.forward(Q, K, V)
    dQ0, dK0, dV0 = ref.backward(Q, K, V, O, LSE, dO)

    run = EngineRun(p)
    Z, h = run.Z, run.h
    h.set_bwd_kernel(kernel)
    n_whole = len(p.cu_seqlens) - 1
    # phase 0: the three remote chunks (their dK/dV go back to their owners); phase 1: the local chunk and the
    # whole sequences
    h.set_bwd_phases([1] * n_whole, [1, 0, 0, 0], 2)
    _, bi = h.phase_info()
    assert len(bi) == 2 and all(x > 0 for x in bi)
    H, d = p.n_heads, p.head_dim
    dQ = torch.full((p.total_q, H, d), SENTINEL, dtype=torch.bfloat16, device=Q.device)
    dK = torch.full((p.total_kv, H, d), SENTINEL, dtype=torch.bfloat16, device=Q.device)
    dV = torch.full_like(dK, SENTINEL)
    nbytes = int(h.info.bwd_workspace_bytes)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=Q.device)
    Z.coalesced_attn_bwd_phase(h, 0, Q, K, V, O, LSE, dO, run.scale, dQ, dK, dV, ws, nbytes)
    torch.cuda.synchronize()
    # after phase 0: gradients of the remote chunks are final, nothing else has been written
    remote = [(ko, kl) for (_, _, ko, kl, _) in p.shards[1:]]
    for ko, kl in remote:
        assert _same_bits(dK[ko:ko + kl], dK0[ko:ko + kl]) and _same_bits(dV[ko:ko + kl], dV0[ko:ko + kl])
    lo = p.shards[0][2] + p.shards[0][3]
    assert bool((dK[:lo] == SENTINEL).all()) and bool((dV[:lo] == SENTINEL).all()) and bool((dQ == SENTINEL).all())
    Z.coalesced_attn_bwd_phase(h, 1, Q, K, V, O, LSE, dO, run.scale, dQ, dK, dV, ws, nbytes)
    torch.cuda.synchronize()
    assert h.last_device_status()[0] == 0
    assert _same_bits(dK, dK0) and _same_bits(dV, dV0)
    a, b = dQ.float(), dQ0.float()
    assert float((a - b).norm() / b.norm()) <= 1e-4
    assert bool((dQ[:1] != SENTINEL).any())
    # the plain entry point still does everything in one call
    dQ1, dK1, dV1 = run.backward(Q, K, V, O, LSE, dO)
    assert _same_bits(dK1, dK0) and _same_bits(dV1, dV0)


def test_sm_margin_changes_no_result():
    """Leaving SMs free for communication kernels (zl_set_sm_margin) only changes which CTA runs which item."""
    p = _placement()
    Q, K, V, dO = _inputs(p, 6)
    ref = EngineRun(p)
    O0, LSE0, _, _ = ref.forward(Q, K, V)
    dQ0, dK0, dV0 = ref.backward(Q, K, V, O0, LSE0, dO)
    for margin in (8, 147, 1000):
        run = EngineRun(p)
        run.h.set_sm_margin(margin)
        O, LSE, _, _ = run.forward(Q, K, V)
        dQ, dK, dV = run.backward(Q, K, V, O, LSE, dO)
        assert _same_bits(O, O0) and _same_bits(LSE, LSE0) and _same_bits(dK, dK0) and _same_bits(dV, dV0)
        assert float((dQ.float() - dQ0.float()).norm() / dQ0.float().norm()) <= 1e-4
    with pytest.raises(run.Z.ZlError):
        run.h.set_sm_margin(-1)


def test_phases_with_head_ranges():
    """Whole images over all heads in phase 0; two Ulysses-shaped sequences over half of the heads each, sharing
    one block of rows, released one after the other (the arrival of two all-to-all batches)."""
    p = W.ulysses_mix_placement(n_heads=4, head_dim=128, n_images=3, image_len=700, seq_len=900, degree=2)
    Q, K, V, dO = _inputs(p, 8)
    ref = EngineRun(p)
    O0, LSE0, _, _ = ref.forward(Q, K, V)
    dQ0, dK0, dV0 = ref.backward(Q, K, V, O0, LSE0, dO)
    run = EngineRun(p)
    Z, h = run.Z, run.h
    h.set_fwd_phases([0, 0, 0, 1, 2], None, 3)
    h.set_bwd_phases([1, 1, 1, 0, 0], None, 2)
    O, LSE, OP, LP = _buffers(p, h.info, Q.device)
    # the Ulysses rows arrive head range by head range: fill them just before their phase
    base = 3 * 700
    Kt, Vt, Qt = K.clone(), V.clone(), Q.clone()
    Kt[base:], Vt[base:], Qt[base:] = 0, 0, 0
    Z.coalesced_attn_fwd_phase(h, 0, Qt, Kt, Vt, run.scale, O, LSE, OP, LP)
    torch.cuda.synchronize()
    for ph, (hb, he) in ((1, (0, 2)), (2, (2, 4))):
        Qt[base:, hb:he], Kt[base:, hb:he], Vt[base:, hb:he] = Q[base:, hb:he], K[base:, hb:he], V[base:, hb:he]
        Z.coalesced_attn_fwd_phase(h, ph, Qt, Kt, Vt, run.scale, O, LSE, OP, LP)
        torch.cuda.synchronize()
    Z.lse_merge(h, OP, LP, O, LSE)
    torch.cuda.synchronize()
    assert _same_bits(O, O0) and _same_bits(LSE, LSE0)
    H, d = p.n_heads, p.head_dim
    dQ = torch.full((p.total_q, H, d), SENTINEL, dtype=torch.bfloat16, device=Q.device)
    dK, dV = torch.full_like(dQ, SENTINEL), torch.full_like(dQ, SENTINEL)
    nbytes = int(h.info.bwd_workspace_bytes)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=Q.device)
    Z.coalesced_attn_bwd_phase(h, 0, Q, K, V, O, LSE, dO, run.scale, dQ, dK, dV, ws, nbytes)
    torch.cuda.synchronize()
    assert _same_bits(dK[base:], dK0[base:]) and _same_bits(dV[base:], dV0[base:]) and bool((dK[:base] == SENTINEL).all())
    Z.coalesced_attn_bwd_phase(h, 1, Q, K, V, O, LSE, dO, run.scale, dQ, dK, dV, ws, nbytes)
    torch.cuda.synchronize()
    assert h.last_device_status()[0] == 0
    assert _same_bits(dK, dK0) and _same_bits(dV, dV0)
    assert float((dQ.float() - dQ0.float()).norm() / dQ0.float().norm()) <= 1e-4
