"""The context-parallel executor bound to the CUDA library (EngineAttention) on one GPU: a one-rank world has
no collectives to run, so this checks the engine side of the binding -- lowering to zl_build_tasks_heads, one
coalesced launch + merge, the backward -- against the fp64 oracle.  The multi-rank plumbing is covered on CPU
ranks (tests/test_executor_cpu.py)."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist

import zl_workloads as W
from oracle import attention as A
from zl_testlib import TOL_GRAD_REL, TOL_O_MAX, rel_fro

pytestmark = pytest.mark.gpu


def test_executor_with_engine_attention_one_rank():
    from paper_2608_01150_b200 import executor as E
    port = 29700 + os.getpid() % 200
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    try:
        H, d = 4, 128
        segs = [E.Segment(1, 300, (1, 1, 1), (0,)), E.Segment(2, 1000, (1, 1, 1), (0,)), E.Segment(3, 77, (1, 1, 1), (0,))]
        ex = E.CPExecutor(segs, H, d)
        eng = E.EngineAttention(d)
        rng = np.random.RandomState(3)
        T = ex.schedule.own_tokens
        bits = [W.f32_to_bf16_bits(W._bf16_round_f32(rng.standard_normal((T, H, d)).astype(np.float32))) for _ in range(4)]
        q, k, v, do = (torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16) for b in bits)
        o = ex.forward(q, k, v, eng.fwd)
        dq, dk, dv = ex.backward(do, eng.bwd)
        torch.cuda.synchronize()
        f64 = [W.bf16_bits_to_f32(b).astype(np.float64) for b in bits]
        pos = 0
        for s in segs:
            sl = slice(pos, pos + s.length)
            for h in range(H):
                qh, kh, vh, doh = (np.ascontiguousarray(x[sl, h]) for x in f64)
                O_ref, _ = A.attn_fwd(qh, kh, vh, d ** -0.5)
                gq, gk, gv = A.attn_bwd(qh, kh, vh, doh, d ** -0.5)
                assert np.abs(o[sl, h].double().cpu().numpy() - O_ref).max() <= TOL_O_MAX
                for got, ref in ((dq, gq), (dk, gk), (dv, gv)):
                    assert rel_fro(got[sl, h].double().cpu().numpy(), ref) <= TOL_GRAD_REL
            pos += s.length
    finally:
        dist.destroy_process_group()
