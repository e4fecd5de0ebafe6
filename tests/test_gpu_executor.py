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
        # the phased form degenerates to one phase each way on a rank without remote chunks: same bits
        o2 = ex.forward(q, k, v, eng)
        dq2, dk2, dv2 = ex.backward(do, eng)
        torch.cuda.synchronize()
        assert ex.schedule.n_fwd_phases == 1 and ex.schedule.n_bwd_phases == 1
        assert torch.equal(o2.view(torch.int16), o.view(torch.int16)) and torch.equal(dk2.view(torch.int16), dk.view(torch.int16))
        assert torch.equal(dv2.view(torch.int16), dv.view(torch.int16))
        assert float((dq2.float() - dq.float()).norm() / dq.float().norm()) <= 1e-4
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


# -------------------------------------------------------------------------------------------------------------------
# Two ranks as two processes on ONE GPU: collectives go through gloo with the tensors staged in host memory (the
# shim below), every kernel only ever sees its own process's memory and none waits for the other process.  This
# runs the phased attention step of the engine under real CUDA streams: tasks released chunk by chunk, gradients of
# remote chunks reduce-scattered under the second backward phase.
class _HostStagedDist:
    """torch.distributed (gloo) for CUDA tensors: every tensor crosses through host memory."""

    def __init__(self):
        self.group = dist.group

    def __getattr__(self, name):              # get_rank, get_world_size, get_backend, new_group, ...
        return getattr(dist, name)

    def all_gather_into_tensor(self, out, inp, group=None):
        o = torch.empty(out.shape, dtype=out.dtype)
        dist.all_gather_into_tensor(o, inp.cpu(), group=group)
        out.copy_(o)

    def broadcast(self, t, src, group=None):
        c = t.cpu()
        dist.broadcast(c, src=src, group=group)
        t.copy_(c)

    def reduce(self, t, dst, group=None):
        c = t.float().cpu()                   # gloo has no bf16 sum
        dist.reduce(c, dst=dst, group=group)
        t.copy_(c.to(t.dtype))

    def all_to_all_single(self, out, inp, output_split_sizes=None, input_split_sizes=None, group=None):
        o = torch.empty(out.shape, dtype=out.dtype)
        dist.all_to_all_single(o, inp.cpu(), output_split_sizes=output_split_sizes, input_split_sizes=input_split_sizes,
                               group=group)
        out.copy_(o)

    isend, irecv = "isend", "irecv"

    class P2POp:
        def __init__(self, op, tensor, peer, group=None):
            self.op, self.tensor, self.peer, self.group = op, tensor, peer, group

    class _Work:
        def __init__(self, work, dev, host):
            self.work, self.dev, self.host = work, dev, host

        def wait(self):
            self.work.wait()
            if self.dev is not None:
                self.dev.copy_(self.host)

    def batch_isend_irecv(self, ops):
        real, pairs = [], []
        for o in ops:
            host = o.tensor.cpu() if o.op == "isend" else torch.empty(o.tensor.shape, dtype=o.tensor.dtype)
            real.append(dist.P2POp(dist.isend if o.op == "isend" else dist.irecv, host, o.peer, group=o.group))
            pairs.append((None if o.op == "isend" else o.tensor, host))
        return [self._Work(w, dev, host) for w, (dev, host) in zip(dist.batch_isend_irecv(real), pairs)]


def _two_rank_worker(rank, port, out_dir):
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    sys.path.insert(0, os.path.join(root, "tests"))
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=2)
    torch.cuda.set_device(0)
    from paper_2608_01150_b200 import executor as E
    H, d = 4, 128
    segs = [E.Segment(1, 700, (1, 1, 1), (0,)), E.Segment(2, 333, (1, 1, 1), (1,)),
            E.Segment(3, 2000, (2, 1, 1), (0, 1)),        # all-gather context parallelism, 1000-token chunks (ragged tiles)
            E.Segment(4, 1536, (1, 1, 2), (1, 0)),        # ring
            E.Segment(5, 900, (1, 2, 1), (0, 1))]         # Ulysses: heads [0,2) and [2,4)
    rng = np.random.RandomState(11)
    data = {s.seq_id: [W.f32_to_bf16_bits(W._bf16_round_f32(rng.standard_normal((s.length, H, d)).astype(np.float32)))
                       for _ in range(4)] for s in segs}
    ex = E.CPExecutor(segs, H, d, dist=_HostStagedDist())
    sch = ex.schedule
    assert sch.n_fwd_phases == 4 and sch.n_bwd_phases == 2
    own = [torch.from_numpy(np.concatenate([data[pc.seq_id][t][pc.g0:pc.g1] for pc in sch.pieces]).view(np.int16))
           .cuda().view(torch.bfloat16) for t in range(4)]
    eng = E.EngineAttention(d)
    o = ex.forward(own[0], own[1], own[2], eng)            # the object itself: phased
    assert sorted(ex.phase_log) == [0, 1, 2, 3] and ex.phase_log[0] == 0
    dq, dk, dv = ex.backward(own[3], eng)
    torch.cuda.synchronize()
    # the same layer with one launch after all collectives must agree (forward bit for bit; dK/dV up to the order
    # of the two-term sum at the chunk owner; dQ up to the order of the fp32 reduce-adds)
    ex1 = E.CPExecutor(segs, H, d, cache=ex.cache, dist=_HostStagedDist())
    eng1 = E.EngineAttention(d)
    o1 = ex1.forward(own[0], own[1], own[2], eng1.fwd)
    dq1, dk1, dv1 = ex1.backward(own[3], eng1.bwd)
    torch.cuda.synchronize()
    assert torch.equal(o.view(torch.int16), o1.view(torch.int16))
    for a, b in ((dq, dq1), (dk, dk1), (dv, dv1)):
        assert float((a.float() - b.float()).norm() / b.float().norm()) <= 4e-3
    # and against single-rank attention over each whole sequence (fp64 oracle)
    f64 = {sid: [W.bf16_bits_to_f32(b).astype(np.float64) for b in v] for sid, v in data.items()}
    worst = 0.0
    for pc in sch.pieces:
        qf, kf, vf, dof = f64[pc.seq_id]
        sl = slice(pc.own_off, pc.own_off + pc.g1 - pc.g0)
        for h in range(H):
            qh, kh, vh, doh = (np.ascontiguousarray(x[:, h]) for x in (qf, kf, vf, dof))
            O_ref, _ = A.attn_fwd(qh, kh, vh, d ** -0.5)
            gq, gk, gv = A.attn_bwd(qh, kh, vh, doh, d ** -0.5)
            assert np.abs(o[sl, h].double().cpu().numpy() - O_ref[pc.g0:pc.g1]).max() <= TOL_O_MAX
            for got, ref in ((dq, gq), (dk, gk), (dv, gv)):
                # a chunk's dK/dV is the bf16 sum of two ranks' bf16 contributions: one more rounding than usual
                worst = max(worst, rel_fro(got[sl, h].double().cpu().numpy(), ref[pc.g0:pc.g1]))
    assert worst <= 2 * TOL_GRAD_REL, worst
    dist.barrier()
    with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
        f.write(f"{worst:.3e}")
    dist.destroy_process_group()


def test_phased_executor_two_processes_on_one_gpu(tmp_path):
    import torch.multiprocessing as mp
    port = 29300 + os.getpid() % 200
    mp.spawn(_two_rank_worker, args=(port, str(tmp_path)), nprocs=2, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(2))
