"""Seeded synthetic workloads for the coalesced attention engine.

This module holds placements (which token ranges form which attention problems) and
seeded tensor generators. It contains none of the method's arithmetic, so both the
CPU oracle's tests and the CUDA path's tests / benchmark may import it.

A *placement* describes what one rank executes in one launch (Section IV-D of the
paper: whole sequences packed block-diagonally plus shards of distributed-attention
groups):

  * ``cu_seqlens``  -- whole sequence i owns rows [cu[i], cu[i+1]) of BOTH token spaces
    (Q-space: Q, O, dO, dQ, LSE; KV-space: K, V, dK, dV).
  * ``shards``      -- (q_off, q_len, kv_off, kv_len, seq_id) tuples: one query chunk
    attending to one K/V chunk.  Shards that share a query range form a merge group.

The five named configurations use Wan latent token counts (1560 = one 480p latent
frame, 3600 = one 720p frame, x21 latent frames for videos; 497,760 tokens for a 15 s
1080p video as stated in the paper's introduction) and the paper's mix structure of a
few long video shards plus many short whole images.  They stand in for the paper's
image/video suites, which are not available offline.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

TENSOR_ID = {"Q": 0, "K": 1, "V": 2, "dO": 3}


@dataclass(frozen=True)
class Placement:
    name: str
    n_heads: int
    head_dim: int
    seed: int
    cu_seqlens: Tuple[int, ...]
    shards: Tuple[Tuple[int, int, int, int, int], ...]
    total_q: int
    total_kv: int
    # Head ranges (Ulysses-shaped tasks: all tokens of a sequence for a subset of the heads).  None = every
    # task covers all heads.  With `whole_ranges` the whole sequences are given as (off, len) pairs instead
    # of cu_seqlens, which lets two sequences own the same rows on disjoint head ranges.
    whole_heads: Optional[Tuple[Tuple[int, int], ...]] = None   # (head_begin, head_count) per whole sequence
    shard_heads: Optional[Tuple[Tuple[int, int], ...]] = None   # (head_begin, head_count) per shard
    whole_ranges: Optional[Tuple[Tuple[int, int], ...]] = None  # (off, len) per whole sequence

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    @property
    def n_whole(self) -> int:
        return len(self.whole_ranges) if self.whole_ranges is not None else len(self.cu_seqlens) - 1

    @property
    def has_head_ranges(self) -> bool:
        return self.whole_heads is not None or self.shard_heads is not None or self.whole_ranges is not None

    def whole_descs(self) -> List[Tuple[int, int, int, int]]:
        """(off, len, head_begin, head_count) per whole sequence."""
        rng = self.whole_ranges if self.whole_ranges is not None else \
            [(self.cu_seqlens[i], self.cu_seqlens[i + 1] - self.cu_seqlens[i]) for i in range(len(self.cu_seqlens) - 1)]
        hd = self.whole_heads if self.whole_heads is not None else [(0, self.n_heads)] * len(rng)
        assert len(hd) == len(rng)
        return [(int(o), int(l), int(hb), int(hc)) for (o, l), (hb, hc) in zip(rng, hd)]

    def shard_head_ranges(self) -> List[Tuple[int, int]]:
        if self.shard_heads is None:
            return [(0, self.n_heads)] * len(self.shards)
        assert len(self.shard_heads) == len(self.shards)
        return [(int(a), int(b)) for a, b in self.shard_heads]

    def whole_lengths(self) -> List[int]:
        return [w[1] for w in self.whole_descs()]

    def pairs_per_head(self) -> int:
        """Number of (query, key) score elements per head over all tasks (all-head placements)."""
        n = sum(l * l for l in self.whole_lengths())
        n += sum(s[1] * s[3] for s in self.shards)
        return n

    def fwd_flops(self) -> float:
        """Counted forward FLOPs: 4 * Lq * Lkv * d * (heads of the task) summed over tasks."""
        pairs = sum(l * l * hc for (_, l, _, hc) in self.whole_descs())
        pairs += sum(s[1] * s[3] * hc for s, (_, hc) in zip(self.shards, self.shard_head_ranges()))
        return 4.0 * pairs * self.head_dim

    def bwd_flops(self) -> float:
        return 2.5 * self.fwd_flops()


def make_placement(name: str, n_heads: int, head_dim: int, seed: int,
                   whole: Sequence[int],
                   cp_groups: Sequence[Tuple[int, int, int]] = ()) -> Placement:
    """Build a placement from whole-sequence lengths and context-parallel groups.

    ``cp_groups`` holds (n_q_chunks, n_kv_chunks, chunk_len) per long sequence: the
    rank owns ``n_q_chunks`` query chunks, each attending to all ``n_kv_chunks`` K/V
    chunks (which on one GPU are simply local inputs).  When n_q_chunks equals
    n_kv_chunks and both spaces have the same size, the query chunks are the same
    tokens as the K/V chunks (a whole long sequence split into chunk tasks).
    """
    cu = [0]
    for l in whole:
        cu.append(cu[-1] + int(l))
    q_pos = cu[-1]
    kv_pos = cu[-1]
    shards = []
    for sid, (nq, nkv, cl) in enumerate(cp_groups):
        for qi in range(nq):
            for ki in range(nkv):
                shards.append((q_pos + qi * cl, cl, kv_pos + ki * cl, cl, sid))
        q_pos += nq * cl
        kv_pos += nkv * cl
    return Placement(name, n_heads, head_dim, seed, tuple(cu), tuple(shards), q_pos, kv_pos)


# Filler lengths of config 5: log-uniform in [256, 8192], total exactly 65,536 tokens.
# They were drawn once with CPython's random.Random(5) (L = round(exp(uniform(ln 256,
# ln 8192))), last one trimmed to the total) and are pinned literally so that no
# generator has to reproduce them.
CONFIG5_FILLERS = (2217, 3348, 4028, 6711, 3326, 6259, 283, 1285, 6732, 2427, 5811, 379,
                   1301, 602, 1685, 1871, 268, 543, 674, 6130, 3637, 445, 4056, 414, 1104)


def config(idx: int) -> Placement:
    """The five named configurations (1-based index)."""
    if idx == 1:
        # 3 whole sequences + one 2048-token sequence as 2 q-chunks x 2 kv-chunks.
        return make_placement("cfg1_tiny", 2, 64, 0, [256, 512, 1000], [(2, 2, 1024)])
    if idx == 2:
        return make_placement("cfg2_images", 12, 128, 1, [1560] * 32 + [3600] * 4)
    if idx == 3:
        return make_placement("cfg3_mixed_cp4", 12, 128, 2, [1560] * 16,
                              [(1, 4, 8190), (1, 4, 8190)])
    if idx == 4:
        return make_placement("cfg4_wan14b_cp8", 40, 128, 3, [1560] * 6, [(1, 8, 9450)])
    if idx == 5:
        assert sum(CONFIG5_FILLERS) == 65536
        return make_placement("cfg5_longvideo_cp16", 40, 128, 4, list(CONFIG5_FILLERS),
                              [(1, 16, 31110)])
    raise ValueError(f"no config {idx}")


def straggler_placement() -> Placement:
    """Config 3's images next to one 32,760-token video placed WHOLE (the naive
    data-parallel placement the paper's motivation section describes): used to show
    what longest-first ordering removes from the tail of the launch."""
    return make_placement("straggler_whole_video", 12, 128, 7, [1560] * 16 + [32760])


# --------------------------------------------------------------------------------------
# Tensor generators
# --------------------------------------------------------------------------------------

def _bf16_round_f32(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bfloat16 (ties to even); result kept as float32."""
    u = x.astype(np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def head_tensor(seed: int, tensor: str, head: int, rows: int, head_dim: int) -> np.ndarray:
    """Canonical generator: one [rows, head_dim] block of i.i.d. N(0,1) values rounded
    float64 -> float32 -> bfloat16, returned as float32 holding exact bf16 values.

    The stream is ``numpy.random.RandomState(seed*1000003 + tensor_id*10007 + head)``
    (frozen across numpy versions); per-head streams let a checker build only the heads
    it needs.
    """
    rs = np.random.RandomState(seed * 1000003 + TENSOR_ID[tensor] * 10007 + head)
    x = rs.standard_normal((rows, head_dim)).astype(np.float32)
    return _bf16_round_f32(x)


def rows_of(p: Placement, tensor: str) -> int:
    return p.total_q if tensor in ("Q", "dO") else p.total_kv


def head_tensor_for(p: Placement, tensor: str, head: int) -> np.ndarray:
    return head_tensor(p.seed, tensor, head, rows_of(p, tensor), p.head_dim)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Exact-bf16-valued float32 -> uint16 bit patterns."""
    return (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def packed_bf16_bits(p: Placement, tensor: str, heads: Optional[Sequence[int]] = None,
                     workers: int = 0) -> np.ndarray:
    """[rows, H, d] uint16 array of bf16 bit patterns in the library's packed layout.

    ``workers`` > 1 generates the per-head blocks in a process pool.
    """
    rows = rows_of(p, tensor)
    out = np.zeros((rows, p.n_heads, p.head_dim), dtype=np.uint16)
    hs = list(range(p.n_heads)) if heads is None else list(heads)
    if workers and workers > 1 and len(hs) > 1:
        import concurrent.futures as cf
        with cf.ProcessPoolExecutor(max_workers=workers) as ex:
            futs = {h: ex.submit(_head_bits, p.seed, tensor, h, rows, p.head_dim) for h in hs}
            for h, f in futs.items():
                out[:, h, :] = f.result()
    else:
        for h in hs:
            out[:, h, :] = _head_bits(p.seed, tensor, h, rows, p.head_dim)
    return out


def _head_bits(seed, tensor, head, rows, head_dim):
    return f32_to_bf16_bits(head_tensor(seed, tensor, head, rows, head_dim))


def device_normal_bf16(shape, seed: int, device):
    """Fast seeded N(0,1) bf16 tensor created on the device (benchmark inputs at full
    size, where only shapes and value distribution matter for timing)."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


# --------------------------------------------------------------------------------------
# Randomised small placements and adversarial edge structure (tests)
# --------------------------------------------------------------------------------------

def random_placement(rng: np.random.RandomState, n_heads: int, head_dim: int,
                     max_whole: int = 4, max_len: int = 300,
                     max_groups: int = 2) -> Placement:
    """A small random placement with ragged lengths, for randomised parity tests."""
    whole = [int(rng.randint(1, max_len + 1)) for _ in range(int(rng.randint(0, max_whole + 1)))]
    groups = []
    for _ in range(int(rng.randint(0, max_groups + 1))):
        nkv = int(rng.randint(1, 4))
        nq = int(rng.choice([1, nkv]))
        groups.append((nq, nkv, int(rng.randint(1, max_len + 1))))
    if not whole and not groups:
        whole = [int(rng.randint(1, max_len + 1))]
    return make_placement("random", n_heads, head_dim, int(rng.randint(0, 1 << 30)), whole, groups)


def custom_placement(name: str, n_heads: int, head_dim: int, seed: int,
                     cu_seqlens: Sequence[int], shards: Sequence[Sequence[int]],
                     total_q: int, total_kv: int) -> Placement:
    return Placement(name, n_heads, head_dim, seed, tuple(int(c) for c in cu_seqlens),
                     tuple(tuple(int(v) for v in s) for s in shards), int(total_q), int(total_kv))


def head_range_placement(name: str, n_heads: int, head_dim: int, seed: int,
                         whole: Sequence[Sequence[int]], shards: Sequence[Sequence[int]],
                         total_q: int, total_kv: int) -> Placement:
    """A placement whose tasks cover head ranges: `whole` holds (off, len, head_begin, head_count) per
    whole sequence, `shards` holds (q_off, q_len, kv_off, kv_len, seq_id, head_begin, head_count)."""
    return Placement(name, n_heads, head_dim, seed, (0,),
                     tuple(tuple(int(v) for v in s[:5]) for s in shards), int(total_q), int(total_kv),
                     whole_heads=tuple((int(w[2]), int(w[3])) for w in whole),
                     shard_heads=tuple((int(s[5]), int(s[6])) for s in shards),
                     whole_ranges=tuple((int(w[0]), int(w[1])) for w in whole))


def ulysses_mix_placement(n_heads: int = 12, head_dim: int = 128, seed: int = 21, n_images: int = 6,
                          image_len: int = 1560, seq_len: int = 3600, degree: int = 2) -> Placement:
    """Whole images over all heads next to `degree` Ulysses-shaped sequences, each holding all of its
    `seq_len` tokens for n_heads / degree heads; the Ulysses sequences share one block of rows, side by
    side in the head dimension (the layout a QKV-packed all-to-all over `degree` ranks delivers)."""
    assert n_heads % degree == 0
    hc = n_heads // degree
    whole = [(i * image_len, image_len, 0, n_heads) for i in range(n_images)]
    base = n_images * image_len
    whole += [(base, seq_len, r * hc, hc) for r in range(degree)]
    total = base + seq_len
    return head_range_placement("ulysses_mix", n_heads, head_dim, seed, whole, [], total, total)
