"""Host-side tests (no GPU): the C-ABI library loads and exports every declared symbol, and
zl_build_tasks validates placements and orders work longest-first."""
import ctypes
import os
import re

import numpy as np
import pytest

import zl_workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def Z():
    from paper_2608_01150_b200 import build
    build.build()
    import paper_2608_01150_b200 as Z
    return Z


def test_library_exports_every_declared_symbol(Z):
    with open(os.path.join(ROOT, "include", "zellige.h")) as f:
        header = f.read()
    names = set(re.findall(r"\b(zl_[a-z_0-9]+)\s*\(", header))
    assert {"zl_build_tasks", "zl_coalesced_attn_fwd", "zl_lse_merge", "zl_coalesced_attn_bwd"} <= names
    lib = ctypes.CDLL(Z.library_path())
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} declared in zellige.h but not exported"


def _build(Z, p):
    return Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, p.n_heads, p.head_dim)


def test_counts_of_named_configs(Z):
    expect_tasks = {1: 7, 2: 36, 3: 24, 4: 14, 5: 41}
    expect_items = {1: 92, 2: 6384, 3: 8640, 4: 26800, 5: 177160}   # 128-row query tiles x heads
    for ci in range(1, 6):
        p = W.config(ci)
        h = _build(Z, p)
        assert h.info.n_tasks == expect_tasks[ci]
        tiles = sum(-(-l // 128) for l in p.whole_lengths()) + sum(-(-s[1] // 128) for s in p.shards)
        assert tiles * p.n_heads == expect_items[ci]
        rows = sum(r for (_, _, _, r) in h.fwd_items())
        assert rows == (sum(p.whole_lengths()) + sum(s[1] for s in p.shards)) * p.n_heads


def _tasks_of(p):
    t = [(p.cu_seqlens[i], p.cu_seqlens[i + 1] - p.cu_seqlens[i], p.cu_seqlens[i], p.cu_seqlens[i + 1] - p.cu_seqlens[i])
         for i in range(p.n_whole) if p.cu_seqlens[i + 1] > p.cu_seqlens[i]]
    t += [s[:4] for s in p.shards if s[1] > 0]
    return t


@pytest.mark.parametrize("seed", range(8))
def test_work_lists_cover_everything_once_and_are_longest_first(Z, seed):
    rng = np.random.RandomState(seed)
    p = W.random_placement(rng, int(rng.randint(1, 4)), 64, max_whole=5, max_len=700, max_groups=3)
    h = _build(Z, p)
    tasks = _tasks_of(p)
    items = h.fwd_items()
    # every query row of every (task, head) exactly once
    seen = {}
    for (t, hd, r0, rows) in items:
        assert 0 < rows and r0 + rows <= tasks[t][1]
        cov = seen.setdefault((t, hd), np.zeros(tasks[t][1], dtype=int))
        cov[r0:r0 + rows] += 1
    assert len(seen) == len(tasks) * p.n_heads and all((c == 1).all() for c in seen.values())
    # non-increasing cost: key length, then rows
    keys = [(tasks[t][3], rows) for (t, _, _, rows) in items]
    assert all(keys[i] >= keys[i + 1] for i in range(len(keys) - 1))
    # backward: every key row of every (kv range, head) exactly once
    kv_ranges = sorted({(t[2], t[3]) for t in tasks if t[3] > 0})
    bitems = h.bwd_items()
    assert h.info.n_kv_groups == len(kv_ranges)
    cover = {}
    for (g, hd, r0, rows) in bitems:
        cover.setdefault((g, hd), []).append((r0, rows))
    assert len(cover) == len(kv_ranges) * p.n_heads
    lens = sorted(l for (_, l) in kv_ranges)
    got = sorted(sum(r for _, r in v) for (g, hd), v in cover.items() if hd == 0)
    assert got == lens
    # partial slots tile [0, partial_rows) without gaps, each padded to 128 rows
    pos = 0
    for si, s in enumerate(p.shards):
        off, padded = h.partial_slot(si)
        if s[1] == 0:
            assert padded == 0
            continue
        assert off == pos and padded == -(-s[1] // 128) * 128
        pos += padded
    assert pos == h.info.partial_rows


def test_backward_list_cost_is_total_query_rows_served(Z):
    # kv range A serves two query chunks (cost 600), kv range B one (cost 300), an image of 200
    p = W.custom_placement("c", 1, 64, 0, [0, 200],
                           [(200, 300, 200, 256, 0), (500, 300, 200, 256, 1), (200, 300, 456, 256, 0)], 800, 712)
    h = _build(Z, p)
    order = [g for (g, _, _, _) in h.bwd_items()]
    firsts = list(dict.fromkeys(order))
    # groups are numbered in order of first appearance: 0 = image, 1 = range A, 2 = range B
    assert firsts == [1, 2, 0]


def test_zero_length_entries_are_ignored(Z):
    p = W.custom_placement("z", 2, 64, 0, [0, 0, 10, 10], [(10, 0, 10, 5, 0), (10, 4, 10, 0, 1)], 20, 20)
    h = _build(Z, p)
    assert h.info.n_tasks == 2          # one whole sequence of 10 rows, one shard with empty K/V
    assert h.partial_slot(0) == (0, 0) and h.partial_slot(1) == (0, 128)


@pytest.mark.parametrize("cu,shards,tq,tkv,hd,status", [
    ([1, 5], [], 5, 5, 64, 1),                                   # cu[0] != 0
    ([0, 5, 3], [], 5, 5, 64, 1),                                # decreasing
    ([0, 9], [], 5, 9, 64, 1),                                   # beyond total_q
    ([0, 4], [(2, 4, 4, 4, 0)], 10, 10, 64, 2),                  # shard inside the whole region
    ([0, 4], [(4, 4, 4, 4, 0), (6, 4, 8, 2, 0)], 12, 12, 64, 2),  # partially overlapping query ranges
    ([0, 4], [(4, 4, 4, 4, 0), (8, 2, 6, 4, 1)], 12, 12, 64, 2),  # partially overlapping key ranges
    ([0, 4], [(4, 4, 4, 4, 0), (4, 4, 4, 4, 0)], 12, 12, 64, 2),  # duplicate task
    ([0, 4], [(4, 4, 4, 4, 0), (4, 4, 8, 4, 1)], 12, 12, 64, 1),  # seq_id differs inside a merge group
    ([0, 4], [(4, 4, 4, 9, 0)], 12, 12, 64, 1),                  # key range beyond total_kv
    ([0, 4], [], 4, 4, 96, 3),                                   # unsupported head_dim
])
def test_invalid_placements_are_rejected_on_the_host(Z, cu, shards, tq, tkv, hd, status):
    with pytest.raises(Z.ZlError) as e:
        Z.build_tasks(cu, shards, tq, tkv, 2, hd)
    assert e.value.status == status


def test_launch_without_device_fails_loudly(Z):
    import torch
    if torch.cuda.is_available():
        pytest.skip("host-only behaviour")
    p = W.config(1)
    h = _build(Z, p)
    with pytest.raises(Z.ZlError) as e:
        Z.coalesced_attn_fwd(h, 16, 16, 16, 0.125, 16, 16, 16, 16, stream=0)
    assert e.value.status == 5      # ZL_ERR_CUDA: no fallback path exists


# ---------------------------------------------------------------- fusion of local chunks (zl_build_tasks_ex)
def _build_fused(Z, p):
    return Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, p.n_heads, p.head_dim,
                         flags=Z.BUILD_FUSE_LOCAL_CHUNKS)


def test_fusion_lowers_contiguous_chunks_to_one_final_task(Z):
    # one image of 100 rows; query range A = [100,300) over three chunks given out of order that tile
    # [100,700); query range B = [300,500) over the same three chunks
    shards = [(100, 200, 300, 200, 0), (100, 200, 100, 200, 0), (100, 200, 500, 200, 0),
              (300, 200, 100, 200, 1), (300, 200, 300, 200, 1), (300, 200, 500, 200, 1)]
    p = W.custom_placement("fuse", 2, 64, 0, [0, 100], shards, 500, 700)
    plain, fused = _build(Z, p), _build_fused(Z, p)
    assert (plain.info.n_tasks, plain.info.n_merge_groups, plain.info.n_fused_ranges) == (7, 2, 0)
    assert plain.info.partial_rows == 6 * 256
    assert (fused.info.n_tasks, fused.info.n_merge_groups, fused.info.n_fused_ranges) == (3, 0, 2)
    assert fused.info.partial_rows == 0 and fused.info.n_kv_groups == 2    # the image and [100,700)
    assert all(fused.partial_slot(i) == (0, 0) for i in range(len(shards)))
    # forward items: every query row of the 3 tasks once per head; key length 600 sorts first
    items = fused.fwd_items()
    assert sorted({t for (t, _, _, _) in items}) == [0, 1, 2]
    rows = {}
    for (t, hd, r0, n) in items:
        rows[(t, hd)] = rows.get((t, hd), 0) + n
    assert sorted(rows.values()) == sorted([100, 100, 200, 200, 200, 200])
    # backward: the interval's 600 key rows once per head, plus the image's 100
    got = {}
    for (g, hd, r0, n) in fused.bwd_items():
        got[(g, hd)] = got.get((g, hd), 0) + n
    assert sorted(got.values()) == [100, 100, 600, 600]


def test_fusion_is_all_or_nothing(Z):
    # range B uses only two of A's three chunks: fusing A would partially overlap B's chunks -> no fusion at all
    shards = [(0, 64, 0, 100, 0), (0, 64, 100, 100, 0), (0, 64, 200, 100, 0),
              (64, 64, 0, 100, 1), (64, 64, 100, 100, 1)]
    p = W.custom_placement("nofuse", 1, 64, 0, [0], shards, 128, 300)
    plain, fused = _build(Z, p), _build_fused(Z, p)
    assert fused.info.n_fused_ranges == 0
    assert (fused.info.n_tasks, fused.info.n_merge_groups, fused.info.partial_rows) == \
           (plain.info.n_tasks, plain.info.n_merge_groups, plain.info.partial_rows)
    assert fused.fwd_items() == plain.fwd_items() and fused.bwd_items() == plain.bwd_items()


def test_fusion_needs_contiguous_chunks_and_keeps_validation(Z):
    # a gap between the chunks: not fused; a single chunk: nothing to fuse
    p = W.custom_placement("gap", 1, 64, 0, [0], [(0, 64, 0, 100, 0), (0, 64, 150, 100, 0), (64, 10, 300, 20, 1)], 80, 320)
    h = _build_fused(Z, p)
    assert h.info.n_fused_ranges == 0 and h.info.n_merge_groups == 2
    # invalid input is still rejected with the same status
    bad = W.custom_placement("bad", 1, 64, 0, [0], [(0, 64, 0, 100, 0), (0, 64, 0, 100, 0)], 64, 100)
    for flags in (0, Z.BUILD_FUSE_LOCAL_CHUNKS):
        with pytest.raises(Z.ZlError) as e:
            Z.build_tasks(bad.cu_seqlens, bad.shards, bad.total_q, bad.total_kv, 1, 64, flags=flags)
        assert e.value.status == 2       # ZL_ERR_OVERLAP: duplicate (query range, key range)
    with pytest.raises(Z.ZlError) as e:
        Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, 1, 64, flags=2)
    assert e.value.status == 1           # unknown flag
