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
from zl_testlib import EngineRun, bits, dev_to_f64, rel_fro, to_dev, TOL_GRAD_REL

pytestmark = pytest.mark.gpu


def test_noalloc_backward_matches_workspace_backward_twice():
    import paper_2608_01150_b200 as Z
    p = W.config(1)
    run = EngineRun(p)
    assert run.info.bwd_workspace_bytes <= Z.NOALLOC_SCRATCH_BYTES
    Q, K, V, dO = (to_dev(bits(p, t)) for t in ("Q", "K", "V", "dO"))
    O, LSE, _, _ = run.forward(Q, K, V)
    ref_dQ, ref_dK, ref_dV = run.backward(Q, K, V, O, LSE, dO)
    # output buffers exist before the measured region; a warm-up call takes the one-time costs
    # (symbol address lookup, kernel code load) out of it
    outs = [tuple(torch.full_like(r, 768.0) for r in (ref_dQ, ref_dK, ref_dV)) for _ in range(3)]
    Z.coalesced_attn_bwd_noalloc(run.h, Q, K, V, O, LSE, dO, p.scale, *outs[2])
    torch.cuda.synchronize()
    # free device memory as the driver sees it: a cudaMalloc / cudaFree inside the library would move
    # it, which torch's own allocator statistics cannot see
    free_before = torch.cuda.mem_get_info()[0]
    launches_before = Z.launch_count()
    for call in range(2):
        dQ, dK, dV = outs[call]
        Z.coalesced_attn_bwd_noalloc(run.h, Q, K, V, O, LSE, dO, p.scale, dQ, dK, dV)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "device memory was allocated or freed by the calls"
    assert Z.launch_count() - launches_before == 2 * 3      # preprocess, main, dQ conversion per call
    assert run.h.last_device_status() == (0, 0)
    for call in range(2):
        dQ, dK, dV = outs[call]
        # dK / dV are accumulated without atomics: identical bits; dQ is reduced with fp32 adds in any order
        assert torch.equal(dK, ref_dK) and torch.equal(dV, ref_dV), f"call {call}"
        assert rel_fro(dev_to_f64(dQ), dev_to_f64(ref_dQ)) <= TOL_GRAD_REL, f"call {call}"
        assert torch.allclose(dQ.float(), ref_dQ.float(), atol=2e-2, rtol=2e-2)


def test_noalloc_backward_rejects_oversized_placements():
    import paper_2608_01150_b200 as Z
    p = W.config(2)                      # needs ~400 MB of scratch
    h = Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, p.n_heads, p.head_dim)
    assert h.info.bwd_workspace_bytes > Z.NOALLOC_SCRATCH_BYTES
    x = torch.zeros(16, device="cuda")
    with pytest.raises(Z.ZlError) as e:
        Z.coalesced_attn_bwd_noalloc(h, x, x, x, x, x, x, p.scale, x, x, x)
    assert e.value.status == 4           # ZL_ERR_WORKSPACE, before anything is launched
