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


# --------------------------------------------------------------------------------------------------
# Per-task head ranges (zl_build_tasks_heads)
# --------------------------------------------------------------------------------------------------

def _build_heads(Z, p, flags=0):
    return Z.build_tasks_heads(p.whole_descs(), p.shards, p.shard_head_ranges(), p.total_q, p.total_kv,
                               p.n_heads, p.head_dim, flags=flags)


def test_heads_builder_with_full_ranges_equals_plain_builder(Z):
    for ci in (1, 3):
        p = W.config(ci)
        a = _build(Z, p)
        b = Z.build_tasks_heads(p.whole_descs(), p.shards, None, p.total_q, p.total_kv, p.n_heads, p.head_dim)
        assert a.fwd_items() == b.fwd_items() and a.bwd_items() == b.bwd_items()
        assert bytes(a.info) == bytes(b.info)
        assert [a.partial_slot(i) for i in range(len(p.shards))] == [b.partial_slot(i) for i in range(len(p.shards))]


def test_head_range_items_cover_each_task_on_its_heads_only(Z):
    p = W.ulysses_mix_placement(n_heads=12, head_dim=128, n_images=6, image_len=1560, seq_len=3600, degree=2)
    h = _build_heads(Z, p)
    whole = p.whole_descs()
    assert h.info.n_tasks == 8 and h.info.n_merge_groups == 0 and h.info.n_kv_groups == 8
    seen = {}
    for (t, hd, r0, rows) in h.fwd_items():
        off, ln, hb, hc = whole[t]
        assert hb <= hd < hb + hc, "work item on a head outside its task's range"
        cov = seen.setdefault((t, hd), np.zeros(ln, dtype=int))
        cov[r0:r0 + rows] += 1
    assert len(seen) == sum(w[3] for w in whole) and all((c == 1).all() for c in seen.values())
    # backward: the two sequences that share rows are two kv groups, six heads each
    per_group = {}
    for (g, hd, r0, rows) in h.bwd_items():
        per_group.setdefault(g, set()).add(hd)
    sizes = sorted(len(v) for v in per_group.values())
    assert sizes == [6, 6] + [12] * 6
    # counted work: 6 images x 12 heads + 2 sequences x 6 heads
    assert p.fwd_flops() == 4.0 * 128 * (6 * 1560 ** 2 * 12 + 2 * 3600 ** 2 * 6)


def test_head_range_shards_form_groups_per_head_range(Z):
    # one query range served on heads [0,2) by two K/V chunks and on heads [2,4) by one chunk over the same rows
    whole = [(0, 100, 0, 4)]
    shards = [(100, 100, 100, 70, 0, 0, 2), (100, 100, 170, 80, 0, 0, 2), (100, 100, 100, 150, 1, 2, 2)]
    p = W.head_range_placement("hr", 4, 64, 3, whole, shards, 200, 250)
    h = _build_heads(Z, p)
    assert h.info.n_tasks == 4 and h.info.n_merge_groups == 2 and h.info.n_kv_groups == 4
    heads_of_task = {}
    for (t, hd, r0, rows) in h.fwd_items():
        heads_of_task.setdefault(t, set()).add(hd)
    assert heads_of_task == {0: {0, 1, 2, 3}, 1: {0, 1}, 2: {0, 1}, 3: {2, 3}}
    # with chunk fusion the two-chunk range becomes one final task; the single-chunk range stays a shard
    hf = _build_heads(Z, p, flags=Z.BUILD_FUSE_LOCAL_CHUNKS)
    assert hf.info.n_fused_ranges == 1 and hf.info.n_tasks == 3 and hf.info.n_merge_groups == 1


def test_head_range_validation(Z):
    def build(whole, shards, H=4, tq=300, tkv=300):
        p = W.head_range_placement("v", H, 64, 0, whole, shards, tq, tkv)
        return _build_heads(Z, p)

    build([(0, 100, 0, 2), (0, 100, 2, 2)], [])                       # same rows, disjoint heads: fine
    build([(0, 100, 0, 4), (100, 50, 1, 2)], [])                      # different rows, nested head ranges: fine
    for whole, shards, status in [
        ([(0, 100, 0, 3), (50, 100, 2, 2)], [], 2),                   # rows overlap on head 2
        ([(0, 100, 0, 3), (0, 100, 2, 2)], [], 2),                    # identical rows, head ranges intersect but differ
        ([(0, 100, 0, 2), (0, 100, 0, 2)], [], 2),                    # the same sequence twice
        ([(0, 100, 0, 5)], [], 1),                                    # head range beyond n_heads
        ([(0, 100, 2, 0)], [], 1),                                    # empty head range
        ([(0, 100, -1, 2)], [], 1),
        ([(0, 100, 0, 4)], [(100, 50, 100, 50, 0, 0, 2), (100, 50, 150, 50, 0, 1, 2)], 2),   # one query range, head ranges intersect but differ
        ([(0, 100, 0, 4)], [(100, 50, 100, 50, 0, 0, 2), (150, 50, 100, 50, 0, 1, 2)], 2),   # one key range, same
        ([(0, 100, 0, 4)], [(50, 50, 100, 50, 0, 0, 2)], 2),          # shard inside the whole region
    ]:
        with pytest.raises(Z.ZlError) as e:
            build(whole, shards)
        assert e.value.status == status, (whole, shards, e.value.status)
    # the same token ranges on disjoint head ranges are independent tasks
    h = build([(0, 100, 0, 4)], [(100, 50, 100, 50, 0, 0, 2), (100, 50, 100, 50, 0, 2, 2)])
    assert h.info.n_tasks == 3 and h.info.n_merge_groups == 2


# ------------------------------------------------------------------------------------------------ launch phases
def _phase_placement():
    # two whole sequences + one query chunk against four K/V chunks, 2 heads
    return W.make_placement("ph", 2, 64, 0, [300, 700], [(1, 4, 500)])


def test_a_handle_starts_with_one_phase_per_direction(Z):
    h = _build(Z, _phase_placement())
    fi, bi = h.phase_info()
    assert fi == [h.info.n_fwd_items] and bi == [h.info.n_bwd_items]


def test_forward_phases_regroup_the_list_and_keep_longest_first_inside_a_phase(Z):
    p = _phase_placement()
    h = _build(Z, p)
    tasks = _tasks_of(p)
    before = sorted(h.fwd_items())
    h.set_fwd_phases([0, 0], [0, 1, 2, 3], 4)
    fi, _ = h.phase_info()
    items = h.fwd_items()
    assert sorted(items) == before and sum(fi) == len(items)
    # tasks 0,1 are the whole sequences, 2..5 the shards in the caller's order
    phase_of_task = {0: 0, 1: 0, 2: 0, 3: 1, 4: 2, 5: 3}
    pos = 0
    for ph, n in enumerate(fi):
        chunk = items[pos:pos + n]
        assert n > 0 and all(phase_of_task[t] == ph for (t, _, _, _) in chunk)
        keys = [(tasks[t][3], rows) for (t, _, _, rows) in chunk]
        assert all(keys[i] >= keys[i + 1] for i in range(len(keys) - 1))
        pos += n
    # changing the order inside the list keeps the grouping
    h.set_fwd_order(2)
    assert h.phase_info()[0] == fi
    items2 = h.fwd_items()
    assert all(phase_of_task[t] == 0 for (t, _, _, _) in items2[:fi[0]])
    # one phase again
    h.set_fwd_phases(None, None, 1)
    assert h.phase_info()[0] == [len(items)]


def test_backward_phases_follow_the_kv_group_with_the_latest_phase(Z):
    # kv range A serves two query chunks, kv range B one; an image of 200
    p = W.custom_placement("c", 1, 64, 0, [0, 200],
                           [(200, 300, 200, 256, 0), (500, 300, 200, 256, 1), (200, 300, 456, 256, 0)], 800, 712)
    h = _build(Z, p)
    n = h.info.n_bwd_items
    # the two tasks on kv range A ask for phases 0 and 1: the group runs in phase 1
    h.set_bwd_phases([1], [0, 1, 0], 2)
    _, bi = h.phase_info()
    assert sum(bi) == n
    items = h.bwd_items()
    groups_phase0 = {g for (g, _, _, _) in items[:bi[0]]}
    groups_phase1 = {g for (g, _, _, _) in items[bi[0]:]}
    assert len(groups_phase0) == 1 and len(groups_phase1) == 2 and not (groups_phase0 & groups_phase1)
    assert bi[0] == 2      # kv range B: 256 rows = two key tiles, one head


def test_phase_arguments_are_validated(Z):
    h = _build(Z, _phase_placement())
    for bad in ([0, 0], [0, 0, 0, 4]), ([0, -1], [0, 0, 0, 0]):
        with pytest.raises(Z.ZlError, match="ZL_ERR_INVALID_ARG"):
            h.set_fwd_phases(bad[0], bad[1], 4)
    for n_phases in (0, Z.MAX_PHASES + 1):
        with pytest.raises(Z.ZlError, match="ZL_ERR_INVALID_ARG"):
            h.set_bwd_phases(None, None, n_phases)
    # a failed call leaves the handle as it was
    assert h.phase_info()[0] == [h.info.n_fwd_items]


def test_a_fused_range_runs_in_the_latest_phase_of_its_chunks(Z):
    p = _phase_placement()
    h = Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, p.n_heads, p.head_dim,
                      flags=Z.BUILD_FUSE_LOCAL_CHUNKS)
    assert h.info.n_fused_ranges == 1 and h.info.n_tasks == 3
    h.set_fwd_phases(None, [0, 1, 2, 1], 3)
    fi, _ = h.phase_info()
    assert fi[1] == 0 and fi[2] > 0 and fi[0] > 0
    assert all(t == 2 for (t, _, _, _) in h.fwd_items()[fi[0]:])


@pytest.mark.parametrize("seed", range(6))
def test_random_phase_assignments_partition_both_lists(Z, seed):
    """Whatever phases the caller asks for: every forward item sits in the phase of its task, every backward item in
    the latest phase among the tasks of its kv group, nothing is lost or duplicated, and the order inside a phase is
    the order the single-phase list had."""
    rng = np.random.RandomState(100 + seed)
    p = W.random_placement(rng, int(rng.randint(1, 4)), 64, max_whole=5, max_len=700, max_groups=3)
    h = _build(Z, p)
    tasks = _tasks_of(p)
    f0, b0 = h.fwd_items(), h.bwd_items()
    n_whole, n_shards = len(p.cu_seqlens) - 1, len(p.shards)
    n_phases = int(rng.randint(1, 6))
    wp = [int(x) for x in rng.randint(0, n_phases, n_whole)]
    sp = [int(x) for x in rng.randint(0, n_phases, n_shards)]
    h.set_fwd_phases(wp, sp, n_phases)
    h.set_bwd_phases(wp, sp, n_phases)
    # task numbering: whole sequences with len > 0, then shards with q_len > 0
    task_phase = [wp[i] for i in range(n_whole) if p.cu_seqlens[i + 1] > p.cu_seqlens[i]] + \
                 [sp[j] for j in range(n_shards) if p.shards[j][1] > 0]
    assert len(task_phase) == len(tasks)
    fi, bi = h.phase_info()
    assert len(fi) == n_phases and len(bi) == n_phases
    f1, b1 = h.fwd_items(), h.bwd_items()
    assert sorted(f1) == sorted(f0) and sorted(b1) == sorted(b0)
    pos = 0
    for ph, n in enumerate(fi):
        assert all(task_phase[t] == ph for (t, _, _, _) in f1[pos:pos + n])
        assert f1[pos:pos + n] == [x for x in f0 if task_phase[x[0]] == ph]      # stable
        pos += n
    # kv groups in order of first appearance over the tasks with keys
    group_of_range, group_phase = {}, []
    for ti, t in enumerate(tasks):
        if t[3] == 0:
            continue
        g = group_of_range.setdefault((t[2], t[3]), len(group_of_range))
        if g == len(group_phase):
            group_phase.append(task_phase[ti])
        else:
            group_phase[g] = max(group_phase[g], task_phase[ti])
    pos = 0
    for ph, n in enumerate(bi):
        assert all(group_phase[g] == ph for (g, _, _, _) in b1[pos:pos + n])
        assert b1[pos:pos + n] == [x for x in b0 if group_phase[x[0]] == ph]
        pos += n
