"""Context-parallel executor above the coalesced attention engine (paper Section IV-D, second
paragraph, and Table II).

A global placement assigns every sequence a parallelism configuration and a set of ranks.  Each
rank lowers the placement into its rank-local schedule -- which of the sequence's global token
ranges it materialises, the K/V movement it takes part in, and the one coalesced attention
launch (whole sequences + shard tasks + head-range tasks) it runs -- caches one process group
per rank set, and issues its collectives in an order that is identical on every participant:
segments sorted by decreasing split degree, ties by global placement order.

Supported configurations (the three single-axis primitives of Table II and the whole-sequence
configuration):

  (1,1,1)  whole sequence on one rank: no communication.
  (q,1,1)  all-gather context parallelism: rank i owns query/key/value chunk i; K and V are
           gathered once; in the backward dK/dV are reduce-scattered to the chunk owners.
  (1,1,k)  ring context parallelism: the same chunks, K/V streamed in k-1 neighbour exchanges
           (the chunks that arrived are consumed as local shard tasks; gradients of the
           gathered chunks travel back with a reduce-scatter).
  (1,h,1)  Ulysses: rank i owns L/h tokens; one QKV-packed all-to-all gives it all L tokens for
           n_heads/h heads, one inverse all-to-all returns the outputs.  Ulysses sequences that
           share configuration and rank set are batched into one all-to-all each way.

Overlap (Section IV-D): with a phased attention step (an object with fwd_begin / fwd_phase / fwd_end
and bwd_begin / bwd_phase / bwd_end, see :class:`EngineAttention`) the tasks whose K/V are already local
are launched first and the collectives run beside them on a second stream; every arrival -- the
gathered chunks of an all-gather segment, the chunk of each ring step, the sequences of a Ulysses
batch -- releases the launch phase of the tasks that were waiting for it.  In the backward the
gradients of remote K/V chunks are computed first and travel to their owners (reduce-scatter) while
the rest of the backward runs.

The attention step itself is a pair of callables, so that the executor is plumbing only:
:class:`EngineAttention` (below) binds it to the CUDA library; tests bind it to a checker.  The
kernels only ever see this GPU's memory: K/V chunks of other ranks are first moved into local
buffers with ``torch.distributed`` collectives.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import torch

ALL_GATHER, RING, ULYSSES, WHOLE = "all_gather", "ring", "ulysses", "whole"
MAX_PHASES = 64  # launch phases of one handle (ZL_MAX_PHASES of the C ABI)


@dataclass(frozen=True)
class Segment:
    """One sequence of the global placement: `length` tokens, configuration (q, h, k) as in Table II,
    executed by `ranks` (chunk / slice i belongs to ranks[i])."""
    seq_id: int
    length: int
    config: Tuple[int, int, int]
    ranks: Tuple[int, ...]

    @property
    def kind(self) -> str:
        q, h, k = self.config
        active = [(q, ALL_GATHER), (h, ULYSSES), (k, RING)]
        on = [name for deg, name in active if deg > 1]
        if not on:
            return WHOLE
        if len(on) > 1:
            raise ValueError(f"sequence {self.seq_id}: multi-axis configuration {self.config} is not supported")
        return on[0]

    @property
    def degree(self) -> int:
        q, h, k = self.config
        return q * h * k


def chunk_bounds(length: int, degree: int, i: int) -> Tuple[int, int]:
    """Global token range [a, b) of chunk i when `length` tokens are split into `degree` nearly equal
    contiguous chunks (the first length % degree chunks are one token longer)."""
    base, extra = divmod(length, degree)
    a = i * base + min(i, extra)
    return a, a + base + (1 if i < extra else 0)


def validate(segments: Sequence[Segment], world_size: int, n_heads: int) -> None:
    seen = set()
    for s in segments:
        if s.seq_id in seen:
            raise ValueError(f"sequence id {s.seq_id} appears twice")
        seen.add(s.seq_id)
        if s.length <= 0 or min(s.config) < 1:
            raise ValueError(f"sequence {s.seq_id}: bad length or configuration")
        if len(s.ranks) != s.degree or len(set(s.ranks)) != len(s.ranks):
            raise ValueError(f"sequence {s.seq_id}: needs {s.degree} distinct ranks")
        if any(r < 0 or r >= world_size for r in s.ranks):
            raise ValueError(f"sequence {s.seq_id}: rank outside the world")
        if s.kind == ULYSSES and n_heads % s.degree != 0:
            raise ValueError(f"sequence {s.seq_id}: a Ulysses degree must divide the number of heads")
        if s.kind in (ALL_GATHER, RING) and s.length < s.degree:
            raise ValueError(f"sequence {s.seq_id}: fewer tokens than chunks")


def collective_order(segments: Sequence[Segment]) -> List[int]:
    """Indices of the segments in execution order: decreasing split degree, ties by placement order
    (a stable sort).  Wider collectives first keeps disjoint rank groups from serialising, and every
    participant of a collective meets it at the same position of its own sequence of collectives."""
    return sorted(range(len(segments)), key=lambda i: -segments[i].degree)


class ProcessGroupCache:
    """Process groups keyed by their sorted rank set, reused across steps.  Creating a group is a
    collective over the WORLD, so `ensure` must be called by every rank with the same placement; it
    creates the missing groups in a deterministic order."""

    def __init__(self, dist=None, world_size: Optional[int] = None):
        import torch.distributed as tdist
        self.dist = dist or tdist
        self.world_size = world_size if world_size is not None else self.dist.get_world_size()
        self.groups: Dict[Tuple[int, ...], object] = {}
        self.created = 0

    def ensure(self, segments: Sequence[Segment]) -> None:
        need = sorted({tuple(sorted(s.ranks)) for s in segments if s.degree > 1})
        for key in need:
            if key in self.groups:
                continue
            if len(key) == self.world_size:
                self.groups[key] = self.dist.group.WORLD
            else:
                self.groups[key] = self.dist.new_group(ranks=list(key))
                self.created += 1

    def get(self, ranks: Sequence[int]):
        return self.groups[tuple(sorted(ranks))]


# --------------------------------------------------------------------------------------------------
# Rank-local schedule
# --------------------------------------------------------------------------------------------------

@dataclass
class LocalPiece:
    """What this rank owns of one segment before any communication: global tokens [g0, g1) of sequence
    seq_id (all heads), stored at rows [own_off, own_off + g1 - g0) of the rank's owned-token buffers."""
    seg_index: int
    seq_id: int
    g0: int
    g1: int
    own_off: int


@dataclass
class RankSchedule:
    rank: int
    n_heads: int
    pieces: List[LocalPiece] = field(default_factory=list)
    own_tokens: int = 0
    # engine placement (zl_build_tasks_heads)
    whole: List[Tuple[int, int, int, int]] = field(default_factory=list)      # (off, len, head_begin, head_count)
    shards: List[Tuple[int, int, int, int, int]] = field(default_factory=list)
    total_q: int = 0
    total_kv: int = 0
    # per segment index: where its data sits in the engine's token spaces
    q_rows: Dict[int, Tuple[int, int]] = field(default_factory=dict)          # seg -> (q_off, q_len)
    kv_rows: Dict[int, Tuple[int, int]] = field(default_factory=dict)         # seg -> (kv_off, kv_len) (all chunks)
    chunk_rows: Dict[int, List[Tuple[int, int]]] = field(default_factory=dict)  # seg -> per chunk (kv_off, len)
    heads: Dict[int, Tuple[int, int]] = field(default_factory=dict)           # seg -> (head_begin, head_count)
    order: List[int] = field(default_factory=list)                            # this rank's segments in collective order
    ulysses_batches: List[List[int]] = field(default_factory=list)            # segment indices batched per all-to-all
    # launch phases (phase 0 = runnable before any collective); indices follow `whole` and `shards`
    fwd_whole_phase: List[int] = field(default_factory=list)
    fwd_shard_phase: List[int] = field(default_factory=list)
    n_fwd_phases: int = 1
    bwd_whole_phase: List[int] = field(default_factory=list)
    bwd_shard_phase: List[int] = field(default_factory=list)
    n_bwd_phases: int = 1
    whole_index: Dict[int, int] = field(default_factory=dict)                 # seg -> index into `whole`
    shard_index: Dict[int, List[int]] = field(default_factory=dict)           # seg -> index into `shards` per chunk
    arrival_phase: Dict[int, List[int]] = field(default_factory=dict)         # seg -> forward phase per chunk (CP) / [phase] (Ulysses)


def lower(segments: Sequence[Segment], rank: int, world_size: int, n_heads: int) -> RankSchedule:
    """The rank-local schedule of `rank`: owned token ranges, the engine placement, and the order of
    collectives."""
    validate(segments, world_size, n_heads)
    sch = RankSchedule(rank=rank, n_heads=n_heads)
    mine = [i for i in collective_order(segments) if rank in segments[i].ranks]
    sch.order = mine
    # ---- owned tokens, in placement order (the order a data loader would deliver them)
    for i, s in enumerate(segments):
        if rank not in s.ranks:
            continue
        pos = s.ranks.index(rank)
        g0, g1 = (0, s.length) if s.kind == WHOLE else chunk_bounds(s.length, s.degree, pos)
        sch.pieces.append(LocalPiece(i, s.seq_id, g0, g1, sch.own_tokens))
        sch.own_tokens += g1 - g0
    # ---- engine rows: sequences run as whole tasks first (same rows in both token spaces) ...
    row = 0
    for i in [j for j in range(len(segments)) if rank in segments[j].ranks]:
        s = segments[i]
        if s.kind == WHOLE:
            hb, hc = 0, n_heads
        elif s.kind == ULYSSES:
            hc = n_heads // s.degree
            hb = s.ranks.index(rank) * hc
        else:
            continue
        sch.whole_index[i] = len(sch.whole)
        sch.whole.append((row, s.length, hb, hc))
        sch.q_rows[i] = (row, s.length)
        sch.kv_rows[i] = (row, s.length)
        sch.heads[i] = (hb, hc)
        row += s.length
    # ---- ... then the context-parallel chunks: this rank's query chunk, and every K/V chunk of the sequence
    q_row = kv_row = row
    for i in [j for j in range(len(segments)) if rank in segments[j].ranks]:
        s = segments[i]
        if s.kind not in (ALL_GATHER, RING):
            continue
        pos = s.ranks.index(rank)
        a, b = chunk_bounds(s.length, s.degree, pos)
        sch.q_rows[i] = (q_row, b - a)
        sch.kv_rows[i] = (kv_row, s.length)
        sch.heads[i] = (0, n_heads)
        chunks = []
        sch.shard_index[i] = []
        for j in range(s.degree):
            ca, cb = chunk_bounds(s.length, s.degree, j)
            chunks.append((kv_row + ca, cb - ca))
            sch.shard_index[i].append(len(sch.shards))
            sch.shards.append((q_row, b - a, kv_row + ca, cb - ca, s.seq_id))
        sch.chunk_rows[i] = chunks
        q_row += b - a
        kv_row += s.length
    sch.total_q, sch.total_kv = q_row, kv_row
    # ---- Ulysses sequences that share configuration and rank set travel in one all-to-all
    batches: Dict[Tuple, List[int]] = {}
    for i in mine:
        s = segments[i]
        if s.kind == ULYSSES:
            batches.setdefault((s.config, s.ranks), []).append(i)
    sch.ulysses_batches = list(batches.values())
    # ---- launch phases, numbered in the order the collectives deliver: forward phase 0 holds the whole sequences
    # and every context-parallel query chunk against its own K/V chunk
    sch.fwd_whole_phase, sch.fwd_shard_phase = [0] * len(sch.whole), [0] * len(sch.shards)
    sch.bwd_whole_phase, sch.bwd_shard_phase = [0] * len(sch.whole), [0] * len(sch.shards)
    phase, seen_batches = 0, set()

    def next_phase():
        nonlocal phase
        phase = min(phase + 1, MAX_PHASES - 1)
        return phase

    for i in mine:
        s = segments[i]
        if s.kind == WHOLE:
            continue
        if s.kind == ULYSSES:
            bi = next(n for n, b in enumerate(sch.ulysses_batches) if i in b)
            if bi in seen_batches:
                continue
            seen_batches.add(bi)
            ph = next_phase()
            for j in sch.ulysses_batches[bi]:
                sch.fwd_whole_phase[sch.whole_index[j]] = ph
                sch.arrival_phase[j] = [ph]
            continue
        k, pos = s.degree, s.ranks.index(rank)
        per_chunk = [0] * k
        if s.kind == ALL_GATHER:
            ph = next_phase()
            per_chunk = [0 if j == pos else ph for j in range(k)]
        else:
            for t in range(1, k):                      # ring step t delivers the chunk of the rank t places back
                per_chunk[(pos - t) % k] = next_phase()
        sch.arrival_phase[i] = per_chunk
        for j in range(k):
            sch.fwd_shard_phase[sch.shard_index[i][j]] = per_chunk[j]
    sch.n_fwd_phases = phase + 1
    # backward: gradients of remote K/V chunks first (phase 0), everything else after (phase 1)
    if sch.shards:
        sch.n_bwd_phases = 2
        sch.bwd_whole_phase = [1] * len(sch.whole)
        for i, idx in sch.shard_index.items():
            pos = segments[i].ranks.index(rank)
            for j, si in enumerate(idx):
                sch.bwd_shard_phase[si] = 1 if j == pos else 0
    return sch


# --------------------------------------------------------------------------------------------------
# Executor
# --------------------------------------------------------------------------------------------------

AttnFwd = Callable[[RankSchedule, torch.Tensor, torch.Tensor, torch.Tensor], Tuple[torch.Tensor, object]]
AttnBwd = Callable[[RankSchedule, object, torch.Tensor], Tuple[torch.Tensor, torch.Tensor, torch.Tensor]]


class CPExecutor:
    """Runs one attention layer of a global placement on this rank.

    forward(q, k, v, attn_fwd): q, k, v are the rank's OWNED tokens [own_tokens, H, d] in placement
    order; returns o for the same tokens.  backward(d_o, attn_bwd) returns dq, dk, dv for the owned
    tokens.  `attn_fwd(schedule, Q, K, V) -> (O, saved)` and `attn_bwd(schedule, saved, dO) -> (dQ,
    dK, dV)` work on the engine's token spaces ([total_q, H, d] / [total_kv, H, d]); Ulysses rows carry
    data only in the rank's head range.  `log` records the collectives in issue order.
    """

    def __init__(self, segments: Sequence[Segment], n_heads: int, head_dim: int, cache: Optional[ProcessGroupCache] = None,
                 dist=None):
        import torch.distributed as tdist
        self.dist = dist or tdist
        self.rank = self.dist.get_rank()
        self.world_size = self.dist.get_world_size()
        self.segments = list(segments)
        self.n_heads, self.head_dim = n_heads, head_dim
        self.cache = cache or ProcessGroupCache(self.dist)
        self.cache.ensure(self.segments)
        self.schedule = lower(self.segments, self.rank, self.world_size, n_heads)
        self.log: List[Tuple] = []
        self.phase_log: List[int] = []
        self._saved = None
        self._comm_stream = None

    # ---- helpers
    def _piece(self, seg_index: int) -> LocalPiece:
        return next(p for p in self.schedule.pieces if p.seg_index == seg_index)

    def _gloo(self, group) -> bool:
        return self.dist.get_backend(group) == "gloo"

    def _all_gather_chunks(self, dst: torch.Tensor, chunks: List[Tuple[int, int]], mine: torch.Tensor, seg: Segment):
        """Every rank of the segment contributes its chunk; chunk j lands at rows chunks[j] of dst (the
        chunks of a sequence are consecutive rows)."""
        group = self.cache.get(seg.ranks)
        if len({ln for _, ln in chunks}) == 1:
            a, b = chunks[0][0], chunks[-1][0] + chunks[-1][1]
            self.dist.all_gather_into_tensor(dst[a:b], mine.contiguous(), group=group)
            return
        # unequal chunk lengths: one broadcast per chunk owner, in the same order on every participant
        for j, r in enumerate(seg.ranks):
            off, ln = chunks[j]
            buf = mine.contiguous() if r == self.rank else torch.empty_like(dst[off:off + ln])
            self.dist.broadcast(buf, src=r, group=group)
            dst[off:off + ln].copy_(buf)

    def _ring_gather(self, dst: torch.Tensor, chunks: List[Tuple[int, int]], mine: torch.Tensor, seg: Segment):
        """k-1 neighbour exchanges: at step t every rank passes on the chunk it received at step t-1."""
        group = self.cache.get(seg.ranks)
        k, pos = seg.degree, seg.ranks.index(self.rank)
        off, ln = chunks[pos]
        dst[off:off + ln].copy_(mine)
        nxt, prv = seg.ranks[(pos + 1) % k], seg.ranks[(pos - 1) % k]
        for t in range(1, k):
            send_j, recv_j = (pos - t + 1) % k, (pos - t) % k
            so, sl = chunks[send_j]
            ro, rl = chunks[recv_j]
            recv = torch.empty_like(dst[ro:ro + rl])
            ops = [self.dist.P2POp(self.dist.isend, dst[so:so + sl].contiguous(), nxt, group=group),
                   self.dist.P2POp(self.dist.irecv, recv, prv, group=group)]
            for w in self.dist.batch_isend_irecv(ops):
                w.wait()
            dst[ro:ro + rl].copy_(recv)

    def _reduce_scatter_chunks(self, src: torch.Tensor, chunks: List[Tuple[int, int]], seg: Segment) -> torch.Tensor:
        """Sum over the segment's ranks of src rows chunks[j], delivered to ranks[j]; returns this rank's chunk."""
        group = self.cache.get(seg.ranks)
        pos = seg.ranks.index(self.rank)
        equal = len({ln for _, ln in chunks}) == 1
        if equal and not self._gloo(group):
            a, b = chunks[0][0], chunks[-1][0] + chunks[-1][1]
            out = torch.empty_like(src[chunks[pos][0]:chunks[pos][0] + chunks[pos][1]])
            self.dist.reduce_scatter_tensor(out, src[a:b].contiguous(), group=group)
            return out
        # gloo has no reduce-scatter, and ragged chunks do not fit the tensor form: one reduce per chunk owner
        out = None
        for j, r in enumerate(seg.ranks):
            off, ln = chunks[j]
            buf = src[off:off + ln].contiguous()
            self.dist.reduce(buf, dst=r, group=group)
            if j == pos:
                out = buf
        return out

    def _ulysses_exchange(self, batch: List[int], x_own: torch.Tensor, inverse: bool, full: Optional[torch.Tensor] = None):
        """One all-to-all for a batch of Ulysses sequences (same configuration and rank set).

        forward direction: x_own [own rows of the batch, C, H, d] (C = 3 for packed q|k|v) -> per sequence
        [L, C, H/h, d] for this rank's heads.  inverse: `full` holds per-sequence [L, C, H/h, d] -> returns
        [own rows of the batch, C, H, d]."""
        seg0 = self.segments[batch[0]]
        group = self.cache.get(seg0.ranks)
        h, pos = seg0.degree, seg0.ranks.index(self.rank)
        hc = self.n_heads // h
        lens = [[chunk_bounds(self.segments[i].length, h, j)[1] - chunk_bounds(self.segments[i].length, h, j)[0]
                 for i in batch] for j in range(h)]               # lens[j][b]: tokens of sequence b owned by ranks[j]
        rows_of_rank = [sum(l) for l in lens]
        if not inverse:
            C = x_own.shape[1]
            # to ranks[j]: my tokens, heads of ranks[j]
            send = torch.cat([x_own[:, :, j * hc:(j + 1) * hc, :].reshape(-1) for j in range(h)])
            per_tok = C * hc * self.head_dim
            recv = torch.empty(sum(rows_of_rank) * per_tok, dtype=x_own.dtype, device=x_own.device)
            self.dist.all_to_all_single(recv, send, output_split_sizes=[r * per_tok for r in rows_of_rank],
                                        input_split_sizes=[rows_of_rank[pos] * per_tok] * h, group=group)
            # recv: for each source rank j, its tokens of every sequence of the batch; regroup per sequence
            parts = torch.split(recv, [r * per_tok for r in rows_of_rank])
            out = []
            for b in range(len(batch)):
                pieces = []
                for j in range(h):
                    start = sum(lens[j][:b])
                    pieces.append(parts[j].view(rows_of_rank[j], C, hc, self.head_dim)[start:start + lens[j][b]])
                out.append(torch.cat(pieces, dim=0))
            return out
        C = full[0].shape[1]
        per_tok = C * hc * self.head_dim
        send_parts = []
        for j in range(h):
            for b in range(len(batch)):
                a, bb = chunk_bounds(self.segments[batch[b]].length, h, j)
                send_parts.append(full[b][a:bb].reshape(-1))
        send = torch.cat(send_parts)
        recv = torch.empty(rows_of_rank[pos] * per_tok * h, dtype=send.dtype, device=send.device)
        self.dist.all_to_all_single(recv, send, output_split_sizes=[rows_of_rank[pos] * per_tok] * h,
                                    input_split_sizes=[r * per_tok for r in rows_of_rank], group=group)
        # recv: for each source rank j, my tokens with the heads of ranks[j]
        parts = recv.view(h, rows_of_rank[pos], C, hc, self.head_dim)
        return parts.permute(1, 2, 0, 3, 4).reshape(rows_of_rank[pos], C, self.n_heads, self.head_dim)

    # ---- forward
    def forward(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, attn_fwd) -> torch.Tensor:
        """`attn_fwd`: a callable (one launch after all collectives) or a phased attention step (overlap)."""
        sch, H, d = self.schedule, self.n_heads, self.head_dim
        assert q.shape == (sch.own_tokens, H, d) and k.shape == q.shape and v.shape == q.shape
        if hasattr(attn_fwd, "fwd_phase"):
            return self._forward_phased(q, k, v, attn_fwd)
        Q = torch.zeros((sch.total_q, H, d), dtype=q.dtype, device=q.device)
        K = torch.zeros((sch.total_kv, H, d), dtype=q.dtype, device=q.device)
        V = torch.zeros_like(K)
        self.log = []
        done_batches = set()
        for i in sch.order:
            s, pc = self.segments[i], self._piece(i)
            own = slice(pc.own_off, pc.own_off + pc.g1 - pc.g0)
            if s.kind == WHOLE:
                qo, ql = sch.q_rows[i]
                Q[qo:qo + ql], K[qo:qo + ql], V[qo:qo + ql] = q[own], k[own], v[own]
            elif s.kind in (ALL_GATHER, RING):
                qo, ql = sch.q_rows[i]
                Q[qo:qo + ql] = q[own]
                move = self._all_gather_chunks if s.kind == ALL_GATHER else self._ring_gather
                self.log.append((s.kind, s.seq_id, tuple(s.ranks)))
                move(K, sch.chunk_rows[i], k[own], s)
                move(V, sch.chunk_rows[i], v[own], s)
            else:
                bi = next(n for n, b in enumerate(sch.ulysses_batches) if i in b)
                if bi in done_batches:
                    continue
                done_batches.add(bi)
                batch = sch.ulysses_batches[bi]
                self.log.append(("ulysses_all_to_all", tuple(self.segments[j].seq_id for j in batch), tuple(s.ranks)))
                rows = torch.cat([torch.arange(self._piece(j).own_off, self._piece(j).own_off + self._piece(j).g1 - self._piece(j).g0)
                                  for j in batch]).to(q.device)
                packed = torch.stack([q[rows], k[rows], v[rows]], dim=1)          # [rows, 3, H, d]: one QKV-packed exchange
                full = self._ulysses_exchange(batch, packed, inverse=False)
                for j, f in zip(batch, full):
                    (ro, rl), (hb, hc) = sch.q_rows[j], sch.heads[j]
                    Q[ro:ro + rl, hb:hb + hc], K[ro:ro + rl, hb:hb + hc], V[ro:ro + rl, hb:hb + hc] = f[:, 0], f[:, 1], f[:, 2]
        O, saved = attn_fwd(sch, Q, K, V)
        self._saved = (saved, Q.shape, K.shape)
        return self._scatter_q_space(O, q.dtype, q.device, tag="ulysses_inverse_all_to_all")

    def _scatter_q_space(self, X: torch.Tensor, dtype, device, tag: str) -> torch.Tensor:
        """Engine Q-space rows -> owned-token order (Ulysses sequences through the inverse all-to-all)."""
        sch, H, d = self.schedule, self.n_heads, self.head_dim
        out = torch.zeros((sch.own_tokens, H, d), dtype=dtype, device=device)
        done_batches = set()
        for i in sch.order:
            s, pc = self.segments[i], self._piece(i)
            own = slice(pc.own_off, pc.own_off + pc.g1 - pc.g0)
            if s.kind != ULYSSES:
                qo, ql = sch.q_rows[i]
                out[own] = X[qo:qo + ql]
                continue
            bi = next(n for n, b in enumerate(sch.ulysses_batches) if i in b)
            if bi in done_batches:
                continue
            done_batches.add(bi)
            batch = sch.ulysses_batches[bi]
            self.log.append((tag, tuple(self.segments[j].seq_id for j in batch), tuple(s.ranks)))
            full = []
            for j in batch:
                (ro, rl), (hb, hc) = sch.q_rows[j], sch.heads[j]
                full.append(X[ro:ro + rl, hb:hb + hc].unsqueeze(1).contiguous())   # [L, 1, H/h, d]
            back = self._ulysses_exchange(batch, None, inverse=True, full=full)[:, 0]
            pos = 0
            for j in batch:
                p = self._piece(j)
                n = p.g1 - p.g0
                out[p.own_off:p.own_off + n] = back[pos:pos + n]
                pos += n
        return out

    # ---- overlap: launch phases under the collectives
    def _streams(self, ref: torch.Tensor):
        """(compute stream, communication stream) on CUDA, (None, None) on CPU."""
        if not ref.is_cuda:
            return None, None
        if self._comm_stream is None:
            self._comm_stream = torch.cuda.Stream(device=ref.device)
        return torch.cuda.current_stream(ref.device), self._comm_stream

    class _On:
        """`with _On(stream):` -- torch.cuda.stream(stream), or nothing on CPU."""
        def __init__(self, stream):
            self.ctx = torch.cuda.stream(stream) if stream is not None else None

        def __enter__(self):
            if self.ctx is not None:
                self.ctx.__enter__()

        def __exit__(self, *a):
            if self.ctx is not None:
                self.ctx.__exit__(*a)

    def _release(self, main, comm, fn):
        """Runs `fn` (a launch on the compute stream) after everything issued so far on the communication stream."""
        if comm is not None:
            ev = torch.cuda.Event()
            ev.record(comm)
            main.wait_event(ev)
        fn()

    def _forward_phased(self, q, k, v, attn) -> torch.Tensor:
        sch, H, d = self.schedule, self.n_heads, self.head_dim
        Q = torch.zeros((sch.total_q, H, d), dtype=q.dtype, device=q.device)
        K = torch.zeros((sch.total_kv, H, d), dtype=q.dtype, device=q.device)   # zero-filled: rows in flight stay finite
        V = torch.zeros_like(K)
        main, comm = self._streams(q)
        self.log = []
        # 1. everything that needs no communication
        for i in sch.order:
            s, pc = self.segments[i], self._piece(i)
            own = slice(pc.own_off, pc.own_off + pc.g1 - pc.g0)
            if s.kind == WHOLE:
                qo, ql = sch.q_rows[i]
                Q[qo:qo + ql], K[qo:qo + ql], V[qo:qo + ql] = q[own], k[own], v[own]
            elif s.kind in (ALL_GATHER, RING):
                qo, ql = sch.q_rows[i]
                Q[qo:qo + ql] = q[own]
                co, cl = sch.chunk_rows[i][s.ranks.index(self.rank)]
                K[co:co + cl], V[co:co + cl] = k[own], v[own]
        if comm is not None:
            comm.wait_stream(main)
            for t in (Q, K, V, q, k, v):
                t.record_stream(comm)
        st = attn.fwd_begin(sch, Q, K, V)
        attn.fwd_phase(sch, st, 0)
        self.phase_log = [0]

        def launch(ph):
            if ph not in self.phase_log:          # phases are capped at MAX_PHASES: the last one may be shared
                self.phase_log.append(ph)
                self._release(main, comm, lambda: attn.fwd_phase(sch, st, ph))

        # 2. the collectives, in the common order, on the communication stream; each arrival releases its phase
        done_batches = set()
        for i in sch.order:
            s, pc = self.segments[i], self._piece(i)
            own = slice(pc.own_off, pc.own_off + pc.g1 - pc.g0)
            if s.kind == WHOLE:
                continue
            if s.kind == ALL_GATHER:
                self.log.append((s.kind, s.seq_id, tuple(s.ranks)))
                with self._On(comm):
                    self._all_gather_chunks(K, sch.chunk_rows[i], k[own], s)
                    self._all_gather_chunks(V, sch.chunk_rows[i], v[own], s)
                launch(max(sch.arrival_phase[i]))
            elif s.kind == RING:
                self.log.append((s.kind, s.seq_id, tuple(s.ranks)))
                self._ring_gather_kv(K, V, sch.chunk_rows[i], s, comm,
                                     lambda j, i=i: launch(sch.arrival_phase[i][j]))
            else:
                bi = next(n for n, b in enumerate(sch.ulysses_batches) if i in b)
                if bi in done_batches:
                    continue
                done_batches.add(bi)
                batch = sch.ulysses_batches[bi]
                self.log.append(("ulysses_all_to_all", tuple(self.segments[j].seq_id for j in batch), tuple(s.ranks)))
                with self._On(comm):
                    rows = torch.cat([torch.arange(self._piece(j).own_off, self._piece(j).own_off + self._piece(j).g1 - self._piece(j).g0)
                                      for j in batch]).to(q.device)
                    packed = torch.stack([q[rows], k[rows], v[rows]], dim=1)
                    full = self._ulysses_exchange(batch, packed, inverse=False)
                    for j, f in zip(batch, full):
                        (ro, rl), (hb, hc) = sch.q_rows[j], sch.heads[j]
                        Q[ro:ro + rl, hb:hb + hc], K[ro:ro + rl, hb:hb + hc], V[ro:ro + rl, hb:hb + hc] = f[:, 0], f[:, 1], f[:, 2]
                launch(sch.arrival_phase[i][0])
        assert sorted(self.phase_log) == list(range(sch.n_fwd_phases)), (self.phase_log, sch.n_fwd_phases)
        O, saved = attn.fwd_end(sch, st)
        self._saved = (saved, Q.shape, K.shape)
        return self._scatter_q_space(O, q.dtype, q.device, tag="ulysses_inverse_all_to_all")

    def _ring_gather_kv(self, K, V, chunks, seg: Segment, comm, arrived):
        """The ring of _ring_gather for K and V together; `arrived(j)` is called when chunk j is in place."""
        group = self.cache.get(seg.ranks)
        k, pos = seg.degree, seg.ranks.index(self.rank)
        nxt, prv = seg.ranks[(pos + 1) % k], seg.ranks[(pos - 1) % k]
        for t in range(1, k):
            send_j, recv_j = (pos - t + 1) % k, (pos - t) % k
            (so, sl), (ro, rl) = chunks[send_j], chunks[recv_j]
            with self._On(comm):
                recv_k, recv_v = torch.empty_like(K[ro:ro + rl]), torch.empty_like(V[ro:ro + rl])
                ops = [self.dist.P2POp(self.dist.isend, K[so:so + sl].contiguous(), nxt, group=group),
                       self.dist.P2POp(self.dist.isend, V[so:so + sl].contiguous(), nxt, group=group),
                       self.dist.P2POp(self.dist.irecv, recv_k, prv, group=group),
                       self.dist.P2POp(self.dist.irecv, recv_v, prv, group=group)]
                for w in self.dist.batch_isend_irecv(ops):
                    w.wait()
                K[ro:ro + rl].copy_(recv_k)
                V[ro:ro + rl].copy_(recv_v)
            arrived(recv_j)

    def _backward_phased(self, attn, saved, dO, early):
        """Phase 0 computes dK/dV of the remote chunks; their reduce-scatter runs on the communication stream
        while phase 1 computes the rest.  `early[seg]` receives what the other ranks contributed to this rank's
        own chunk (the rank's own contribution is a result of phase 1 and is added by the caller)."""
        sch = self.schedule
        main, comm = self._streams(dO)
        st = attn.bwd_begin(sch, saved, dO)
        attn.bwd_phase(sch, st, 0)
        dK, dV = attn.bwd_grads(st)
        # snapshot of the remote chunks' gradients with zeros in the own chunk: phase 1 writes the own chunk while
        # the collective reads
        staged = {}
        for i in sch.order:
            s = self.segments[i]
            if s.kind not in (ALL_GATHER, RING):
                continue
            a, b = sch.kv_rows[i][0], sch.kv_rows[i][0] + sch.kv_rows[i][1]
            co, cl = sch.chunk_rows[i][s.ranks.index(self.rank)]
            sk, sv = dK[a:b].clone(), dV[a:b].clone()
            sk[co - a:co - a + cl] = 0
            sv[co - a:co - a + cl] = 0
            staged[i] = (sk, sv, a)
        if comm is not None:
            comm.wait_stream(main)
            for sk, sv, _ in staged.values():
                sk.record_stream(comm)
                sv.record_stream(comm)
        attn.bwd_phase(sch, st, 1)
        for i in sch.order:
            if i not in staged:
                continue
            s = self.segments[i]
            sk, sv, a = staged[i]
            rel = [(off - a, ln) for off, ln in sch.chunk_rows[i]]
            self.log.append(("reduce_scatter", s.seq_id, tuple(s.ranks)))
            with self._On(comm):
                early[i] = (self._reduce_scatter_chunks(sk, rel, s), self._reduce_scatter_chunks(sv, rel, s))
        out = attn.bwd_end(sch, st)
        if comm is not None:
            main.wait_stream(comm)
        return out

    # ---- backward
    def backward(self, d_o: torch.Tensor, attn_bwd) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """`attn_bwd`: a callable, or a phased attention step (gradients of remote chunks leave early)."""
        sch, H, d = self.schedule, self.n_heads, self.head_dim
        saved, q_shape, k_shape = self._saved
        phased = hasattr(attn_bwd, "bwd_phase") and sch.n_bwd_phases == 2
        dO = torch.zeros(q_shape, dtype=d_o.dtype, device=d_o.device)
        self.log = []
        done_batches = set()
        for i in sch.order:
            s, pc = self.segments[i], self._piece(i)
            own = slice(pc.own_off, pc.own_off + pc.g1 - pc.g0)
            if s.kind != ULYSSES:
                qo, ql = sch.q_rows[i]
                dO[qo:qo + ql] = d_o[own]
                continue
            bi = next(n for n, b in enumerate(sch.ulysses_batches) if i in b)
            if bi in done_batches:
                continue
            done_batches.add(bi)
            batch = sch.ulysses_batches[bi]
            self.log.append(("ulysses_all_to_all", tuple(self.segments[j].seq_id for j in batch), tuple(s.ranks)))
            rows = torch.cat([torch.arange(self._piece(j).own_off, self._piece(j).own_off + self._piece(j).g1 - self._piece(j).g0)
                              for j in batch]).to(d_o.device)
            full = self._ulysses_exchange(batch, d_o[rows].unsqueeze(1), inverse=False)
            for j, f in zip(batch, full):
                (ro, rl), (hb, hc) = sch.q_rows[j], sch.heads[j]
                dO[ro:ro + rl, hb:hb + hc] = f[:, 0]
        dq = torch.zeros((sch.own_tokens, H, d), dtype=d_o.dtype, device=d_o.device)
        dk, dv = torch.zeros_like(dq), torch.zeros_like(dq)
        early: Dict[int, Tuple[torch.Tensor, torch.Tensor]] = {}
        if phased:
            dQ, dK, dV = self._backward_phased(attn_bwd, saved, dO, early)
        elif hasattr(attn_bwd, "bwd_phase"):      # a phased step on a rank without remote chunks: one phase
            st = attn_bwd.bwd_begin(sch, saved, dO)
            attn_bwd.bwd_phase(sch, st, 0)
            dQ, dK, dV = attn_bwd.bwd_end(sch, st)
        else:
            dQ, dK, dV = attn_bwd(sch, saved, dO)
        done_batches = set()
        for i in sch.order:
            s, pc = self.segments[i], self._piece(i)
            own = slice(pc.own_off, pc.own_off + pc.g1 - pc.g0)
            qo, ql = sch.q_rows[i]
            if s.kind == WHOLE:
                dq[own], dk[own], dv[own] = dQ[qo:qo + ql], dK[qo:qo + ql], dV[qo:qo + ql]
            elif s.kind in (ALL_GATHER, RING):
                dq[own] = dQ[qo:qo + ql]
                if i in early:
                    # the other ranks' contributions arrived under the second phase; add this rank's own
                    co, cl = sch.chunk_rows[i][s.ranks.index(self.rank)]
                    dk[own], dv[own] = early[i][0] + dK[co:co + cl], early[i][1] + dV[co:co + cl]
                    continue
                # every rank holds the gradient of ALL chunks with respect to its own queries: sum them at the owners
                self.log.append(("reduce_scatter", s.seq_id, tuple(s.ranks)))
                dk[own] = self._reduce_scatter_chunks(dK, sch.chunk_rows[i], s)
                dv[own] = self._reduce_scatter_chunks(dV, sch.chunk_rows[i], s)
            else:
                bi = next(n for n, b in enumerate(sch.ulysses_batches) if i in b)
                if bi in done_batches:
                    continue
                done_batches.add(bi)
                batch = sch.ulysses_batches[bi]
                self.log.append(("ulysses_inverse_all_to_all", tuple(self.segments[j].seq_id for j in batch), tuple(s.ranks)))
                full = []
                for j in batch:
                    (ro, rl), (hb, hc) = sch.q_rows[j], sch.heads[j]
                    full.append(torch.stack([dQ[ro:ro + rl, hb:hb + hc], dK[ro:ro + rl, hb:hb + hc],
                                             dV[ro:ro + rl, hb:hb + hc]], dim=1).contiguous())
                back = self._ulysses_exchange(batch, None, inverse=True, full=full)   # [own rows, 3, H, d]
                pos = 0
                for j in batch:
                    p = self._piece(j)
                    n = p.g1 - p.g0
                    dq[p.own_off:p.own_off + n] = back[pos:pos + n, 0]
                    dk[p.own_off:p.own_off + n] = back[pos:pos + n, 1]
                    dv[p.own_off:p.own_off + n] = back[pos:pos + n, 2]
                    pos += n
        return dq, dk, dv


# --------------------------------------------------------------------------------------------------
# The attention step on the CUDA library
# --------------------------------------------------------------------------------------------------

class EngineAttention:
    """The attention step of :class:`CPExecutor` on libzellige: one task handle per schedule (cached).
    Pass the bound methods `fwd` / `bwd` for one coalesced forward launch + merge and one backward call after
    all collectives, or the object itself for launch phases under the collectives.  bf16 CUDA tensors."""

    def __init__(self, head_dim: int, scale: Optional[float] = None, flags: int = 0, sm_margin: int = 0):
        self.head_dim = head_dim
        self.scale = scale if scale is not None else head_dim ** -0.5
        self.flags = flags
        self.sm_margin = sm_margin   # SMs left to the communication kernels that run beside a launch phase
        self._handles: Dict[int, object] = {}

    def _handle(self, sch: RankSchedule):
        from . import binding as Z
        h = self._handles.get(id(sch))
        if h is None:
            h = Z.build_tasks_heads(sch.whole, sch.shards, None, sch.total_q, sch.total_kv, sch.n_heads, self.head_dim,
                                    flags=self.flags)
            h.set_fwd_phases(sch.fwd_whole_phase, sch.fwd_shard_phase, sch.n_fwd_phases)
            h.set_bwd_phases(sch.bwd_whole_phase, sch.bwd_shard_phase, sch.n_bwd_phases)
            if self.sm_margin:
                h.set_sm_margin(self.sm_margin)
            self._handles[id(sch)] = h
        return h

    # ---- phased form
    def fwd_begin(self, sch: RankSchedule, Q, K, V):
        h = self._handle(sch)
        H, d = sch.n_heads, self.head_dim
        pr = max(1, int(h.info.partial_rows))
        return {"h": h, "Q": Q, "K": K, "V": V, "O": torch.zeros_like(Q),
                "LSE": torch.zeros((H, sch.total_q), dtype=torch.float32, device=Q.device),
                "OP": torch.empty((pr, H, d), dtype=torch.float32, device=Q.device),
                "LP": torch.empty((H, pr), dtype=torch.float32, device=Q.device)}

    def fwd_phase(self, sch: RankSchedule, st, phase: int):
        from . import binding as Z
        Z.coalesced_attn_fwd_phase(st["h"], phase, st["Q"], st["K"], st["V"], self.scale, st["O"], st["LSE"], st["OP"], st["LP"])

    def fwd_end(self, sch: RankSchedule, st):
        from . import binding as Z
        Z.lse_merge(st["h"], st["OP"], st["LP"], st["O"], st["LSE"])
        return st["O"], (st["Q"], st["K"], st["V"], st["O"], st["LSE"])

    def bwd_begin(self, sch: RankSchedule, saved, dO):
        h = self._handle(sch)
        Q, K, V, O, LSE = saved
        n = int(h.info.bwd_workspace_bytes)
        return {"h": h, "saved": saved, "dO": dO.contiguous(), "dQ": torch.zeros_like(Q), "dK": torch.zeros_like(K),
                "dV": torch.zeros_like(V), "ws": torch.empty(n + 256, dtype=torch.uint8, device=Q.device), "n": n}

    def bwd_phase(self, sch: RankSchedule, st, phase: int):
        from . import binding as Z
        Q, K, V, O, LSE = st["saved"]
        Z.coalesced_attn_bwd_phase(st["h"], phase, Q, K, V, O, LSE, st["dO"], self.scale, st["dQ"], st["dK"], st["dV"],
                                   st["ws"], st["n"])

    def bwd_grads(self, st):
        return st["dK"], st["dV"]

    def bwd_end(self, sch: RankSchedule, st):
        return st["dQ"], st["dK"], st["dV"]

    def fwd(self, sch: RankSchedule, Q, K, V):
        from . import binding as Z
        h = self._handle(sch)
        H, d = sch.n_heads, self.head_dim
        O = torch.zeros_like(Q)
        LSE = torch.zeros((H, sch.total_q), dtype=torch.float32, device=Q.device)
        pr = max(1, int(h.info.partial_rows))
        OP = torch.empty((pr, H, d), dtype=torch.float32, device=Q.device)
        LP = torch.empty((H, pr), dtype=torch.float32, device=Q.device)
        Z.coalesced_attn_fwd(h, Q, K, V, self.scale, O, LSE, OP, LP)
        Z.lse_merge(h, OP, LP, O, LSE)
        return O, (Q, K, V, O, LSE)

    def bwd(self, sch: RankSchedule, saved, dO):
        from . import binding as Z
        h = self._handle(sch)
        Q, K, V, O, LSE = saved
        dQ, dK, dV = torch.zeros_like(Q), torch.zeros_like(K), torch.zeros_like(V)
        ws = torch.empty(int(h.info.bwd_workspace_bytes) + 256, dtype=torch.uint8, device=Q.device)
        Z.coalesced_attn_bwd(h, Q, K, V, O, LSE, dO.contiguous(), self.scale, dQ, dK, dV, ws, int(h.info.bwd_workspace_bytes))
        return dQ, dK, dV
