"""QKV-packed entry points (zl_coalesced_attn_fwd_packed / zl_coalesced_attn_bwd_packed) against the
separate-tensor entry points and the fp64 oracle.  The packed layout is [T, 3, H, d] (row t holds
q_t | k_t | v_t), what a fused QKV projection or a QKV-packed all-to-all produces (paper Section
IV-D).  The kernels fetch their tiles through strided tensor maps, so forward results and dK / dV
must be bit-identical to the unpacked call; dQ is reduced with fp32 adds in any order."""
import numpy as np
import pytest
import torch

import zl_workloads as W
from oracle import attention as orc
from zl_testlib import (EngineRun, SENTINEL, bits, check_backward, check_forward, dev_to_f64, rel_fro, to_dev,
                        to_f64, TOL_GRAD_REL)

pytestmark = pytest.mark.gpu


def _packed_case(p):
    import paper_2608_01150_b200 as Z
    assert p.total_q == p.total_kv
    H, d, T = p.n_heads, p.head_dim, p.total_q
    run = EngineRun(p)
    hb = {t: bits(p, t) for t in ("Q", "K", "V", "dO")}
    Q, K, V, dO = (to_dev(hb[t]) for t in ("Q", "K", "V", "dO"))
    qkv = torch.stack([Q, K, V], dim=1).contiguous()          # [T, 3, H, d]
    assert qkv.shape == (T, 3, H, d)
    O, LSE, _, _ = run.forward(Q, K, V)
    dQ, dK, dV = run.backward(Q, K, V, O, LSE, dO)

    pr = max(int(run.info.partial_rows), 1)
    O2 = torch.full_like(O, SENTINEL)
    LSE2 = torch.full_like(LSE, SENTINEL)
    OP = torch.full((pr, H, d), SENTINEL, dtype=torch.float32, device="cuda")
    LP = torch.full((H, pr), SENTINEL, dtype=torch.float32, device="cuda")
    Z.coalesced_attn_fwd_packed(run.h, qkv, p.scale, O2, LSE2, OP, LP)
    Z.lse_merge(run.h, OP, LP, O2, LSE2)
    torch.cuda.synchronize()
    assert run.h.last_device_status() == (0, 0)
    assert torch.equal(O2, O) and torch.equal(LSE2, LSE)

    dqkv = torch.full_like(qkv, SENTINEL)
    ws = torch.empty(int(run.info.bwd_workspace_bytes) + 256, dtype=torch.uint8, device="cuda")
    Z.coalesced_attn_bwd_packed(run.h, qkv, O2, LSE2, dO, p.scale, dqkv, ws, int(run.info.bwd_workspace_bytes))
    torch.cuda.synchronize()
    assert run.h.last_device_status() == (0, 0)
    assert torch.equal(dqkv[:, 1], dK) and torch.equal(dqkv[:, 2], dV)
    assert rel_fro(dev_to_f64(dqkv[:, 0].contiguous()), dev_to_f64(dQ)) <= TOL_GRAD_REL
    return p, hb, O2, LSE2, dqkv


def test_packed_matches_unpacked_and_oracle_on_config1():
    # whole sequences and context-parallel shards in one row space (total_q == total_kv)
    p, hb, O2, LSE2, dqkv = _packed_case(W.config(1))
    f = {t: to_f64(hb[t]) for t in hb}
    ref = orc.placement_fwd(p, f["Q"], f["K"], f["V"])
    check_forward(p, O2, LSE2, ref)
    gref = orc.placement_bwd(p, f["Q"], f["K"], f["V"], f["dO"])
    check_backward(p, dqkv[:, 0].contiguous(), dqkv[:, 1].contiguous(), dqkv[:, 2].contiguous(), gref)


def test_packed_ragged_whole_sequences():
    # block-diagonal batch of ragged whole sequences (several tiles and ragged tails), d = 64 and 128
    for d, lens in ((64, [1, 130, 257, 300]), (128, [129, 5, 384])):
        p = W.make_placement("packed", 3, d, 77 + d, lens, [])
        _packed_case(p)


def test_packed_needs_one_row_space():
    import paper_2608_01150_b200 as Z
    p = W.custom_placement("two_spaces", 1, 64, 0, [0, 8], [(8, 8, 8, 16, 0)], 16, 24)
    h = Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, p.n_heads, p.head_dim)
    x = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(4096, dtype=torch.float32, device="cuda")
    with pytest.raises(Z.ZlError) as e:
        Z.coalesced_attn_fwd_packed(h, x, p.scale, x, y, y, y)
    assert e.value.status == 1           # ZL_ERR_INVALID_ARG, nothing launched
    with pytest.raises(Z.ZlError) as e:
        Z.coalesced_attn_bwd_packed(h, x, x, y, x, p.scale, x, x, 4096)
    assert e.value.status == 1
