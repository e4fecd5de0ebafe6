"""The context-parallel executor on CPU ranks (gloo): per-rank lowering of a global placement, the
process-group cache, the order of collectives, and -- with the attention step supplied by this test
(the fp64 oracle; the package itself never imports it) -- exact equality of what the ranks produce
together with single-rank attention over the whole sequences, forward and backward."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
H, D = 4, 8


def _segments(world):
    from paper_2608_01150_b200.executor import Segment
    if world == 2:
        return [Segment(10, 7, (1, 1, 1), (0,)), Segment(11, 9, (1, 1, 1), (1,)),
                Segment(12, 24, (2, 1, 1), (0, 1)),            # all-gather, equal chunks
                Segment(13, 11, (1, 1, 2), (1, 0)),            # ring, unequal chunks, reversed rank order
                Segment(14, 10, (1, 2, 1), (0, 1)), Segment(15, 6, (1, 2, 1), (0, 1)),   # two Ulysses sequences, one batch
                Segment(16, 5, (1, 1, 1), (0,))]
    return [Segment(20, 13, (1, 1, 1), (2,)), Segment(21, 32, (4, 1, 1), (0, 1, 2, 3)),
            Segment(22, 18, (1, 1, 2), (1, 3)), Segment(23, 21, (1, 1, 3), (0, 2, 3)),
            Segment(24, 12, (1, 2, 1), (0, 1)), Segment(25, 9, (1, 2, 1), (0, 1)), Segment(26, 16, (1, 4, 1), (3, 2, 1, 0)),
            Segment(27, 8, (1, 1, 1), (0,)), Segment(28, 10, (2, 1, 1), (2, 3))]


def _global_tensors(segments, seed):
    rng = np.random.RandomState(seed)
    return {s.seq_id: tuple(rng.standard_normal((s.length, H, D)) for _ in range(4)) for s in segments}  # q, k, v, dO


def _oracle_attention():
    """attn_fwd / attn_bwd callables built on the oracle: the schedule's whole tasks and shard groups evaluated
    by definition on the engine's token spaces."""
    sys.path.insert(0, ROOT)
    from oracle import attention as A
    import zl_workloads as W
    scale = D ** -0.5

    def placement_of(sch):
        shards = [tuple(s) + (0, sch.n_heads) for s in sch.shards]
        return W.head_range_placement("rank", sch.n_heads, D, 0, sch.whole, shards, sch.total_q, sch.total_kv)

    def fwd(sch, Q, K, V):
        p = placement_of(sch)
        out = A.placement_fwd(p, Q.numpy(), K.numpy(), V.numpy(), scale=scale, with_partials=False)
        return torch.from_numpy(np.nan_to_num(out["O"])), (p, Q, K, V)

    def bwd(sch, saved, dO):
        p, Q, K, V = saved
        g = A.placement_bwd(p, Q.numpy(), K.numpy(), V.numpy(), dO.numpy(), scale=scale)
        return tuple(torch.from_numpy(g[n]) for n in ("dQ", "dK", "dV"))

    return fwd, bwd


class _PhasedOracle:
    """The phased attention step on the oracle.  A forward phase evaluates its tasks with the K/V rows as they are
    at the time of the call (so a task released before its chunk has arrived gives wrong numbers); a backward
    phase delivers the dK/dV rows of the kv groups of that phase, and dQ with the last one."""

    def __init__(self):
        sys.path.insert(0, ROOT)
        from oracle import attention as A
        self.A, self.scale = A, D ** -0.5
        self.fwd_calls, self.bwd_calls = [], []

    def fwd_begin(self, sch, Q, K, V):
        return {"Q": Q, "K": K, "V": V, "whole": {}, "parts": {}}

    def fwd_phase(self, sch, st, phase):
        A = self.A
        self.fwd_calls.append(phase)
        Q, K, V = (st[n].numpy().copy() for n in ("Q", "K", "V"))
        for w, (off, ln, hb, hc) in enumerate(sch.whole):
            if sch.fwd_whole_phase[w] != phase:
                continue
            st["whole"][w] = {h: A.attn_fwd(np.ascontiguousarray(Q[off:off + ln, h]), np.ascontiguousarray(K[off:off + ln, h]),
                                            np.ascontiguousarray(V[off:off + ln, h]), self.scale)[0] for h in range(hb, hb + hc)}
        for si, (qo, ql, ko, kl, _) in enumerate(sch.shards):
            if sch.fwd_shard_phase[si] != phase:
                continue
            st["parts"][si] = [A.attn_fwd(np.ascontiguousarray(Q[qo:qo + ql, h]), np.ascontiguousarray(K[ko:ko + kl, h]),
                                          np.ascontiguousarray(V[ko:ko + kl, h]), self.scale) for h in range(sch.n_heads)]

    def fwd_end(self, sch, st):
        A = self.A
        assert len(st["whole"]) == len(sch.whole) and len(st["parts"]) == len(sch.shards)
        O = np.zeros(tuple(st["Q"].shape))
        for w, (off, ln, hb, hc) in enumerate(sch.whole):
            for h, o in st["whole"][w].items():
                O[off:off + ln, h] = o
        groups = {}
        for si, (qo, ql, _, _, _) in enumerate(sch.shards):
            groups.setdefault((qo, ql), []).append(si)
        for (qo, ql), members in groups.items():
            for h in range(sch.n_heads):
                O[qo:qo + ql, h] = A.lse_merge([st["parts"][si][h] for si in members])[0]
        return torch.from_numpy(O), (sch, st["Q"], st["K"], st["V"])

    def bwd_begin(self, sch, saved, dO):
        import zl_workloads as W
        _, Q, K, V = saved
        shards = [tuple(s) + (0, sch.n_heads) for s in sch.shards]
        p = W.head_range_placement("rank", sch.n_heads, D, 0, sch.whole, shards, sch.total_q, sch.total_kv)
        g = self.A.placement_bwd(p, Q.numpy(), K.numpy(), V.numpy(), dO.numpy(), scale=self.scale)
        return {"g": g, "dQ": torch.zeros_like(Q), "dK": torch.zeros_like(K), "dV": torch.zeros_like(V)}

    def bwd_phase(self, sch, st, phase):
        self.bwd_calls.append(phase)
        rows = [(off, ln) for w, (off, ln, _, _) in enumerate(sch.whole) if sch.bwd_whole_phase[w] == phase]
        rows += [(ko, kl) for si, (_, _, ko, kl, _) in enumerate(sch.shards) if sch.bwd_shard_phase[si] == phase]
        for off, ln in rows:
            st["dK"][off:off + ln] = torch.from_numpy(st["g"]["dK"][off:off + ln])
            st["dV"][off:off + ln] = torch.from_numpy(st["g"]["dV"][off:off + ln])
        if phase == sch.n_bwd_phases - 1:
            st["dQ"].copy_(torch.from_numpy(st["g"]["dQ"]))

    def bwd_grads(self, st):
        return st["dK"], st["dV"]

    def bwd_end(self, sch, st):
        return st["dQ"], st["dK"], st["dV"]


def _worker(rank, world, port, out_dir, phased=False):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2608_01150_b200 import executor as E
    from oracle import attention as A

    segments = _segments(world)
    data = _global_tensors(segments, 5)
    cache = E.ProcessGroupCache()
    ex = E.CPExecutor(segments, H, D, cache=cache)
    sch = ex.schedule

    # ---- lowering: the rank materialises exactly its token ranges; the engine placement covers them
    for pc in sch.pieces:
        s = segments[pc.seg_index]
        pos = s.ranks.index(rank)
        want = (0, s.length) if s.kind == E.WHOLE else E.chunk_bounds(s.length, s.degree, pos)
        assert (pc.g0, pc.g1) == want
    assert sch.own_tokens == sum(pc.g1 - pc.g0 for pc in sch.pieces)
    for i, s in enumerate(segments):
        if rank not in s.ranks:
            continue
        if s.kind in (E.ALL_GATHER, E.RING):
            assert sum(l for _, l in sch.chunk_rows[i]) == s.length
            assert [sh for sh in sch.shards if sh[4] == s.seq_id] == \
                [(sch.q_rows[i][0], sch.q_rows[i][1], off, ln, s.seq_id) for off, ln in sch.chunk_rows[i]]
        elif s.kind == E.ULYSSES:
            hc = H // s.degree
            assert sch.heads[i] == (s.ranks.index(rank) * hc, hc) and sch.q_rows[i][1] == s.length
    # shards lie after the whole region of both token spaces
    whole_end = max([o + l for (o, l, _, _) in sch.whole], default=0)
    assert all(sh[0] >= whole_end and sh[2] >= whole_end for sh in sch.shards)

    # ---- process groups: one per rank set, created once, reused by a second executor
    n_sets = len({tuple(sorted(s.ranks)) for s in segments if s.degree > 1})
    assert len(cache.groups) == n_sets
    created = cache.created
    ex2 = E.CPExecutor(segments, H, D, cache=cache)
    assert cache.created == created and ex2.cache.get(segments[-1].ranks) is cache.get(segments[-1].ranks) \
        if segments[-1].degree > 1 else cache.created == created

    # ---- one layer, forward and backward, with the oracle as the attention step
    fwd, bwd = _oracle_attention()
    own = {n: torch.from_numpy(np.concatenate([data[pc.seq_id][t][pc.g0:pc.g1] for pc in sch.pieces]))
           for t, n in enumerate(("q", "k", "v", "do"))}
    if phased:
        step = _PhasedOracle()
        o = ex.forward(own["q"], own["k"], own["v"], step)
        log_f = list(ex.log)
        dq, dk, dv = ex.backward(own["do"], step)
        log_b = list(ex.log)
        # every launch phase ran exactly once, the first one before any collective; the backward in order
        assert sorted(step.fwd_calls) == list(range(sch.n_fwd_phases)) and step.fwd_calls[0] == 0
        assert step.bwd_calls == list(range(sch.n_bwd_phases))
        assert sch.n_fwd_phases > 1 and all(ph == 0 for w, ph in enumerate(sch.fwd_whole_phase)
                                            if segments[[i for i, x in sch.whole_index.items() if x == w][0]].kind == E.WHOLE)
    else:
        o = ex.forward(own["q"], own["k"], own["v"], fwd)
        log_f = list(ex.log)
        dq, dk, dv = ex.backward(own["do"], bwd)
        log_b = list(ex.log)

    # ---- collectives: decreasing split degree, ties by placement order; the same order on every participant
    degs = [len(e[2]) for e in log_f if e[0] in (E.ALL_GATHER, E.RING, "ulysses_all_to_all")]
    assert degs == sorted(degs, reverse=True)
    logs = [None] * world
    dist.all_gather_object(logs, (log_f, log_b))
    for other in range(world):
        for mine, theirs in zip((log_f, log_b), logs[other]):
            common_mine = [e for e in mine if other in e[2]]
            common_theirs = [e for e in theirs if rank in e[2]]
            assert common_mine == common_theirs, (rank, other, common_mine, common_theirs)
    # Ulysses sequences with the same configuration and rank set share one exchange
    a2a = [e for e in log_f if e[0] == "ulysses_all_to_all"]
    batched = [e for e in a2a if len(e[1]) > 1]
    if any(segments[i].kind == E.ULYSSES for i in sch.order):
        assert len(a2a) == len(sch.ulysses_batches)
        assert any(len(b) > 1 for b in sch.ulysses_batches) == bool(batched)

    # ---- numerics: together the ranks reproduce single-rank attention over each whole sequence
    scale = D ** -0.5
    worst = 0.0
    for pc in sch.pieces:
        q, k, v, do = data[pc.seq_id]
        sl = slice(pc.own_off, pc.own_off + pc.g1 - pc.g0)
        for h in range(H):
            O_ref, _ = A.attn_fwd(np.ascontiguousarray(q[:, h]), np.ascontiguousarray(k[:, h]), np.ascontiguousarray(v[:, h]), scale)
            gq, gk, gv = A.attn_bwd(np.ascontiguousarray(q[:, h]), np.ascontiguousarray(k[:, h]), np.ascontiguousarray(v[:, h]),
                                    np.ascontiguousarray(do[:, h]), scale)
            for got, ref in ((o, O_ref), (dq, gq), (dk, gk), (dv, gv)):
                worst = max(worst, float(np.abs(got[sl, h].numpy() - ref[pc.g0:pc.g1]).max()))
    assert worst < 1e-11, worst
    dist.barrier()
    with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
        f.write(f"{worst:.3e} {len(log_f)} {len(log_b)}")
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_executor_on_gloo_ranks(tmp_path, world):
    port = 29900 + (os.getpid() * 7 + world) % 300
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(world))


@pytest.mark.parametrize("world", [2, 4])
def test_executor_with_launch_phases_on_gloo_ranks(tmp_path, world):
    """The same layer with the phased attention step: tasks are released as their K/V arrive, the gradients of
    remote chunks are reduce-scattered after the first backward phase."""
    port = 29600 + (os.getpid() * 7 + world) % 300
    mp.spawn(_worker, args=(world, port, str(tmp_path), True), nprocs=world, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(world))


def test_lowering_and_order_without_a_process_group():
    sys.path.insert(0, ROOT)
    from paper_2608_01150_b200 import executor as E
    segs = _segments(4)
    order = E.collective_order(segs)
    assert [segs[i].degree for i in order] == sorted((s.degree for s in segs), reverse=True)
    # stable: equal degrees keep placement order
    for a, b in zip(order, order[1:]):
        if segs[a].degree == segs[b].degree:
            assert a < b
    assert [E.chunk_bounds(11, 3, i) for i in range(3)] == [(0, 4), (4, 8), (8, 11)]
    sch = E.lower(segs, 3, 4, H)
    assert [p.seq_id for p in sch.pieces] == [21, 22, 23, 26, 28]
    assert sch.heads[6] == (0, 1)                       # rank 3 is first in sequence 26's rank list: heads [0, 1)
    for bad in ([E.Segment(1, 8, (2, 2, 1), (0, 1, 2, 3))], [E.Segment(1, 8, (1, 3, 1), (0, 1, 2))],
                [E.Segment(1, 8, (2, 1, 1), (0, 0))], [E.Segment(1, 8, (2, 1, 1), (0, 9))], [E.Segment(1, 1, (2, 1, 1), (0, 1))]):
        with pytest.raises(ValueError):
            E.lower(bad, 0, 4, H)
