"""The allocation-free backward entry point (zl_coalesced_attn_bwd_noalloc) against the regular
one.  Some callers may not allocate device memory where they run the backward (a region owned by
another allocator, a host that forbids allocations after start-up, a latency-critical path), so
they cannot provide a workspace; this entry point keeps its scratch in a fixed array inside the
library instead.  The test calls it through the C ABI twice in a row -- the second call sees the
scratch exactly as the first one left it -- and compares both results with the workspace-based
entry point.  It is collected last so that a failure here cannot hide any other test's result."""
import numpy as np
import pytest
import torch

import zl_workloads as W
from zl_testlib import GpuRun, bits, dev_to_f64, rel_fro, to_dev, TOL_GRAD_REL

pytestmark = pytest.mark.gpu


def test_noalloc_backward_matches_workspace_backward_twice():
    import paper_2608_01150_b200 as Z
    p = W.config(1)
    run = GpuRun(p)
    assert run.info.bwd_workspace_bytes <= Z.NOALLOC_SCRATCH_BYTES
    Q, K, V, dO = (to_dev(bits(p, t)) for t in ("Q", "K", "V", "dO"))
    O, LSE, _, _ = run.forward(Q, K, V)
    ref_dQ, ref_dK, ref_dV = run.backward(Q, K, V, O, LSE, dO)
    mem_before = torch.cuda.memory_allocated()
    for call in range(2):
        dQ = torch.full_like(ref_dQ, 768.0)
        dK = torch.full_like(ref_dK, 768.0)
        dV = torch.full_like(ref_dV, 768.0)
        Z.coalesced_attn_bwd_noalloc(run.h, Q, K, V, O, LSE, dO, p.scale, dQ, dK, dV)
        torch.cuda.synchronize()
        assert run.h.last_device_status() == (0, 0)
        # dK / dV are accumulated without atomics: identical bits; dQ is reduced with fp32 adds in any order
        assert torch.equal(dK, ref_dK) and torch.equal(dV, ref_dV), f"call {call}"
        assert rel_fro(dev_to_f64(dQ), dev_to_f64(ref_dQ)) <= TOL_GRAD_REL, f"call {call}"
        assert torch.allclose(dQ.float(), ref_dQ.float(), atol=2e-2, rtol=2e-2)
        del dQ, dK, dV
    assert torch.cuda.memory_allocated() == mem_before


def test_noalloc_backward_rejects_oversized_placements():
    import paper_2608_01150_b200 as Z
    p = W.config(2)                      # needs ~400 MB of scratch
    h = Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, p.n_heads, p.head_dim)
    assert h.info.bwd_workspace_bytes > Z.NOALLOC_SCRATCH_BYTES
    x = torch.zeros(16, device="cuda")
    with pytest.raises(Z.ZlError) as e:
        Z.coalesced_attn_bwd_noalloc(h, x, x, x, x, x, x, p.scale, x, x, x)
    assert e.value.status == 4           # ZL_ERR_WORKSPACE, before anything is launched
