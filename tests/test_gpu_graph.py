"""A whole step (forward launch, LSE merge, backward) captured once in a CUDA graph and replayed: every
entry point only enqueues work on the stream it is given, so the replay must reproduce the eager
results (forward and dK / dV bit for bit; dQ is reduced with fp32 adds in any order).  Small placements
are launch-bound, which is what the capture is for."""
import pytest
import torch

import zl_workloads as W
from zl_testlib import EngineRun, bits, dev_to_f64, rel_fro, to_dev, TOL_GRAD_REL

pytestmark = pytest.mark.gpu


def test_step_replays_from_a_cuda_graph():
    import paper_2608_01150_b200 as Z
    p = W.config(1)
    run = EngineRun(p)
    H, d = p.n_heads, p.head_dim
    Q, K, V, dO = (to_dev(bits(p, t)) for t in ("Q", "K", "V", "dO"))
    O_ref, LSE_ref, _, _ = run.forward(Q, K, V)
    dQ_ref, dK_ref, dV_ref = run.backward(Q, K, V, O_ref, LSE_ref, dO)

    O = torch.empty_like(O_ref)
    LSE = torch.empty_like(LSE_ref)
    pr = max(1, int(run.info.partial_rows))
    OP = torch.empty((pr, H, d), dtype=torch.float32, device="cuda")
    LP = torch.empty((H, pr), dtype=torch.float32, device="cuda")
    dQ, dK, dV = torch.empty_like(dQ_ref), torch.empty_like(dK_ref), torch.empty_like(dV_ref)
    ws = torch.empty(int(run.info.bwd_workspace_bytes) + 256, dtype=torch.uint8, device="cuda")

    def step():
        Z.coalesced_attn_fwd(run.h, Q, K, V, p.scale, O, LSE, OP, LP)
        Z.lse_merge(run.h, OP, LP, O, LSE)
        Z.coalesced_attn_bwd(run.h, Q, K, V, O, LSE, dO, p.scale, dQ, dK, dV, ws, int(run.info.bwd_workspace_bytes))

    step()                                   # first call outside the capture (one-time kernel attributes)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    for rep in range(2):
        for t in (O, LSE, dQ, dK, dV):
            t.fill_(768.0)
        graph.replay()
        torch.cuda.synchronize()
        assert run.h.last_device_status() == (0, 0)
        assert torch.equal(O, O_ref) and torch.equal(LSE, LSE_ref), f"replay {rep}"
        assert torch.equal(dK, dK_ref) and torch.equal(dV, dV_ref), f"replay {rep}"
        assert rel_fro(dev_to_f64(dQ), dev_to_f64(dQ_ref)) <= TOL_GRAD_REL, f"replay {rep}"
