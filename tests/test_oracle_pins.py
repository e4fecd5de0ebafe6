"""Pins the fp64 CPU oracle to facts that do not come from the oracle itself:
closed forms, a hand-worked example, invariants of softmax attention, brute force on tiny
inputs, a library routine (torch fp64 scaled_dot_product_attention + autograd) and fp64
finite differences.  Each pin is chosen so that a dropped term, a wrong sign or index, or
a transposed operand in the oracle makes it fail."""
import math
import os

import numpy as np
import pytest
import torch

import zl_workloads as W
from oracle import attention as A

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def load_fixture(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals], dtype=np.float64)
    return out


def rnd(rng, *shape):
    return rng.standard_normal(shape)


# ------------------------------------------------------------------ forward: closed forms

def test_worked_example_forward_and_backward():
    fx = load_fixture("worked_example.txt")
    q = fx["q"].reshape(1, 1); k = fx["k"].reshape(2, 1); v = fx["v"].reshape(2, 1)
    dO = fx["dO"].reshape(1, 1)
    O, lse = A.attn_fwd(q, k, v, 1.0)
    assert abs(O[0, 0] - fx["O"][0]) < 1e-14
    assert abs(lse[0] - fx["LSE"][0]) < 1e-15
    assert abs(A.bwd_delta(dO, O)[0] - fx["D"][0]) < 1e-14
    dQ, dK, dV = A.attn_bwd(q, k, v, dO, 1.0)
    np.testing.assert_allclose(dQ.ravel(), fx["dQ"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(dK.ravel(), fx["dK"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(dV.ravel(), fx["dV"], rtol=0, atol=1e-14)


def test_worked_example_split_and_merged():
    fx = load_fixture("worked_example.txt")
    q = fx["q"].reshape(1, 1); k = fx["k"].reshape(2, 1); v = fx["v"].reshape(2, 1)
    parts = [A.attn_fwd(q, k[j:j + 1], v[j:j + 1], 1.0) for j in range(2)]
    assert abs(parts[0][0][0, 0] - fx["part0_O"][0]) < 1e-15
    assert abs(parts[0][1][0] - fx["part0_LSE"][0]) < 1e-15
    assert abs(parts[1][0][0, 0] - fx["part1_O"][0]) < 1e-15
    assert abs(parts[1][1][0] - fx["part1_LSE"][0]) < 1e-15
    O, lse = A.lse_merge(parts)
    assert abs(O[0, 0] - fx["O"][0]) < 1e-14 and abs(lse[0] - fx["LSE"][0]) < 1e-15


def test_single_key_gives_value_row_and_raw_score():
    rng = np.random.RandomState(1)
    q, k, v = rnd(rng, 5, 7), rnd(rng, 1, 7), rnd(rng, 1, 7)
    O, lse = A.attn_fwd(q, k, v, 0.3)
    np.testing.assert_allclose(O, np.repeat(v, 5, 0), rtol=0, atol=1e-15)
    np.testing.assert_allclose(lse, 0.3 * (q @ k[0]), rtol=1e-14)


def test_two_keys_sigmoid_softplus_closed_form():
    rng = np.random.RandomState(2)
    q, k, v = rnd(rng, 6, 5), rnd(rng, 2, 5), rnd(rng, 2, 5)
    sc = 0.7
    O, lse = A.attn_fwd(q, k, v, sc)
    for i in range(6):
        s1 = sc * sum(q[i, c] * k[0, c] for c in range(5))
        s2 = sc * sum(q[i, c] * k[1, c] for c in range(5))
        delta = s1 - s2
        sig = 1.0 / (1.0 + math.exp(-delta))
        softplus = math.log1p(math.exp(delta))
        for c in range(5):
            assert abs(O[i, c] - (sig * v[0, c] + (1 - sig) * v[1, c])) < 1e-14
        assert abs(lse[i] - (s2 + softplus)) < 1e-13


def test_constant_value_rows_reproduce_that_row():
    rng = np.random.RandomState(3)
    q, k = rnd(rng, 9, 16), rnd(rng, 33, 16)
    vrow = rnd(rng, 1, 16)
    O, _ = A.attn_fwd(q, k, np.repeat(vrow, 33, 0), 0.25)
    assert np.max(np.abs(O - vrow) / np.abs(vrow)) < 1e-14


def test_zero_query_gives_mean_value_and_log_count():
    rng = np.random.RandomState(4)
    k, v = rnd(rng, 21, 8), rnd(rng, 21, 8)
    O, lse = A.attn_fwd(np.zeros((3, 8)), k, v, 1.0)
    np.testing.assert_allclose(O, np.repeat(v.mean(0, keepdims=True), 3, 0), atol=1e-15)
    np.testing.assert_allclose(lse, math.log(21), rtol=1e-15)


def test_key_permutation_invariance():
    rng = np.random.RandomState(5)
    q, k, v = rnd(rng, 7, 12), rnd(rng, 40, 12), rnd(rng, 40, 12)
    perm = rng.permutation(40)
    O1, l1 = A.attn_fwd(q, k, v, 0.4)
    O2, l2 = A.attn_fwd(q, k[perm], v[perm], 0.4)
    np.testing.assert_allclose(O1, O2, atol=1e-14)
    np.testing.assert_allclose(l1, l2, atol=1e-14)


def test_key_shift_moves_lse_only():
    rng = np.random.RandomState(6)
    q, k, v = rnd(rng, 7, 12), rnd(rng, 19, 12), rnd(rng, 19, 12)
    c = rnd(rng, 1, 12)
    O1, l1 = A.attn_fwd(q, k, v, 0.4)
    O2, l2 = A.attn_fwd(q, k + c, v, 0.4)
    np.testing.assert_allclose(O1, O2, atol=1e-13)
    np.testing.assert_allclose(l2 - l1, 0.4 * (q @ c[0]), atol=1e-13)


def test_empty_key_set():
    O, lse = A.attn_fwd(np.ones((3, 4)), np.zeros((0, 4)), np.zeros((0, 4)), 1.0)
    assert np.all(O == 0) and np.all(np.isneginf(lse))
    Om, lm = A.lse_merge([(O, lse), (O, lse)])
    assert np.all(Om == 0) and np.all(np.isneginf(lm))


def _brute_force(q, k, v, sc):
    """Pure-Python definition on tiny inputs."""
    nq, d = len(q), len(q[0])
    O = [[0.0] * d for _ in range(nq)]
    lse = [0.0] * nq
    for i in range(nq):
        s = [sc * sum(q[i][c] * k[j][c] for c in range(d)) for j in range(len(k))]
        z = sum(math.exp(x) for x in s)
        lse[i] = math.log(z)
        for j in range(len(k)):
            for c in range(d):
                O[i][c] += math.exp(s[j]) / z * v[j][c]
    return np.array(O), np.array(lse)


@pytest.mark.parametrize("nq,nk,d", [(1, 1, 1), (2, 3, 2), (4, 2, 3), (3, 4, 5)])
def test_brute_force_tiny(nq, nk, d):
    rng = np.random.RandomState(10 * nq + nk)
    q, k, v = rnd(rng, nq, d), rnd(rng, nk, d), rnd(rng, nk, d)
    O, lse = A.attn_fwd(q, k, v, 0.9)
    Ob, lb = _brute_force(q.tolist(), k.tolist(), v.tolist(), 0.9)
    np.testing.assert_allclose(O, Ob, atol=1e-14)
    np.testing.assert_allclose(lse, lb, atol=1e-14)


def test_row_subset_matches_full():
    rng = np.random.RandomState(7)
    q, k, v = rnd(rng, 20, 8), rnd(rng, 31, 8), rnd(rng, 31, 8)
    O, lse = A.attn_fwd(q, k, v, 0.5)
    rows = [19, 0, 7]
    Os, ls = A.attn_fwd(q, k, v, 0.5, rows=rows)
    assert np.array_equal(Os, O[rows]) and np.array_equal(ls, lse[rows])


def test_strided_head_views_accepted():
    rng = np.random.RandomState(8)
    X = rnd(rng, 30, 3, 8)
    q, k, v = X[:10, 1, :], X[10:, 2, :], X[10:, 0, :]
    O1, l1 = A.attn_fwd(q, k, v, 0.5)
    O2, l2 = A.attn_fwd(np.ascontiguousarray(q), np.ascontiguousarray(k), np.ascontiguousarray(v), 0.5)
    assert np.array_equal(O1, O2) and np.array_equal(l1, l2)


# ------------------------------------------------------------------ forward: library routine

def _torch_ref(q, k, v, sc):
    tq, tk, tv = (torch.from_numpy(np.ascontiguousarray(x)) for x in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None], scale=sc)[0]
    lse = torch.logsumexp((tq @ tk.T) * sc, -1)
    return o.numpy(), lse.numpy()


@pytest.mark.parametrize("nq,nk,d", [(17, 50, 64), (130, 33, 128), (64, 257, 16)])
def test_matches_torch_sdpa_fp64(nq, nk, d):
    rng = np.random.RandomState(nq)
    q, k, v = rnd(rng, nq, d), rnd(rng, nk, d), rnd(rng, nk, d)
    O, lse = A.attn_fwd(q, k, v, 1 / math.sqrt(d))
    Ot, lt = _torch_ref(q, k, v, 1 / math.sqrt(d))
    np.testing.assert_allclose(O, Ot, atol=1e-13)
    np.testing.assert_allclose(lse, lt, atol=1e-13)


# ------------------------------------------------------------------ merge

def test_merge_single_part_is_identity():
    rng = np.random.RandomState(11)
    O, lse = rnd(rng, 5, 4), rnd(rng, 5)
    Om, lm = A.lse_merge([(O, lse)])
    np.testing.assert_allclose(Om, O, atol=1e-15)
    np.testing.assert_allclose(lm, lse, atol=1e-15)


def test_merge_equal_lse_is_plain_average():
    rng = np.random.RandomState(12)
    parts = [(rnd(rng, 5, 4), np.full(5, 1.25)) for _ in range(3)]
    Om, lm = A.lse_merge(parts)
    np.testing.assert_allclose(Om, sum(p[0] for p in parts) / 3, atol=1e-15)
    np.testing.assert_allclose(lm, 1.25 + math.log(3), atol=1e-15)


def test_merge_is_associative():
    rng = np.random.RandomState(13)
    parts = [(rnd(rng, 6, 3), 3 * rnd(rng, 6)) for _ in range(4)]
    flat = A.lse_merge(parts)
    nested = A.lse_merge([A.lse_merge(parts[:2]), A.lse_merge(parts[2:])])
    np.testing.assert_allclose(flat[0], nested[0], atol=1e-14)
    np.testing.assert_allclose(flat[1], nested[1], atol=1e-14)


def test_merge_ignores_empty_part():
    rng = np.random.RandomState(14)
    O, lse = rnd(rng, 4, 3), rnd(rng, 4)
    Om, lm = A.lse_merge([(np.zeros((4, 3)), np.full(4, -np.inf)), (O, lse)])
    np.testing.assert_allclose(Om, O, atol=1e-15)
    np.testing.assert_allclose(lm, lse, atol=1e-15)


@pytest.mark.parametrize("chunks", [[10, 10], [5, 1, 20, 7], [3] * 8, [1, 2, 3, 4] * 4])
def test_shard_then_merge_equals_full_attention(chunks):
    rng = np.random.RandomState(len(chunks))
    n = sum(chunks)
    q, k, v = rnd(rng, 9, 8), rnd(rng, n, 8), rnd(rng, n, 8)
    O, lse = A.attn_fwd(q, k, v, 0.6)
    parts, pos = [], 0
    for c in chunks:
        parts.append(A.attn_fwd(q, k[pos:pos + c], v[pos:pos + c], 0.6))
        pos += c
    Om, lm = A.lse_merge(parts)
    np.testing.assert_allclose(Om, O, atol=1e-13)
    np.testing.assert_allclose(lm, lse, atol=1e-13)


# ------------------------------------------------------------------ backward

def test_single_key_backward():
    rng = np.random.RandomState(20)
    q, k, v, dO = rnd(rng, 4, 6), rnd(rng, 1, 6), rnd(rng, 1, 6), rnd(rng, 4, 6)
    dQ, dK, dV = A.attn_bwd(q, k, v, dO, 0.5)
    assert np.max(np.abs(dQ)) < 1e-14 and np.max(np.abs(dK)) < 1e-14
    np.testing.assert_allclose(dV[0], dO.sum(0), atol=1e-14)


def test_backward_sum_identities():
    rng = np.random.RandomState(21)
    q, k, v, dO = rnd(rng, 13, 8), rnd(rng, 29, 8), rnd(rng, 29, 8), rnd(rng, 13, 8)
    dQ, dK, dV = A.attn_bwd(q, k, v, dO, 0.35)
    np.testing.assert_allclose(dV.sum(0), dO.sum(0), atol=1e-13)   # sum_j p_ij = 1
    np.testing.assert_allclose(dK.sum(0), 0, atol=1e-13)           # sum_j dS_ij = 0
    kk = np.repeat(k[:1], 29, 0)
    dQ2, _, _ = A.attn_bwd(q, kk, v, dO, 0.35)                     # equal keys: dQ = 0
    assert np.max(np.abs(dQ2)) < 1e-13


def _loss(q, k, v, dO, sc):
    O, _ = A.attn_fwd(q, k, v, sc)
    return float(np.sum(O * dO))


@pytest.mark.parametrize("nq,nk,d", [(3, 5, 4), (16, 9, 8)])
def test_backward_finite_differences(nq, nk, d):
    rng = np.random.RandomState(22 + nq)
    q, k, v, dO = rnd(rng, nq, d), rnd(rng, nk, d), rnd(rng, nk, d), rnd(rng, nq, d)
    sc = 0.45
    grads = A.attn_bwd(q, k, v, dO, sc)
    eps = 1e-5
    for arr, g in zip((q, k, v), grads):
        fd = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            old = arr[idx]
            arr[idx] = old + eps; lp = _loss(q, k, v, dO, sc)
            arr[idx] = old - eps; lm = _loss(q, k, v, dO, sc)
            arr[idx] = old
            fd[idx] = (lp - lm) / (2 * eps)
        assert np.linalg.norm(fd - g) / np.linalg.norm(g) < 1e-7


@pytest.mark.parametrize("nq,nk,d", [(17, 50, 64), (40, 23, 128)])
def test_backward_matches_torch_autograd(nq, nk, d):
    rng = np.random.RandomState(30 + nq)
    q, k, v, dO = rnd(rng, nq, d), rnd(rng, nk, d), rnd(rng, nk, d), rnd(rng, nq, d)
    sc = 1 / math.sqrt(d)
    tq, tk, tv = (torch.from_numpy(x.copy()).requires_grad_(True) for x in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None], scale=sc)[0]
    (o * torch.from_numpy(dO)).sum().backward()
    dQ, dK, dV = A.attn_bwd(q, k, v, dO, sc)
    np.testing.assert_allclose(dQ, tq.grad.numpy(), atol=1e-13)
    np.testing.assert_allclose(dK, tk.grad.numpy(), atol=1e-13)
    np.testing.assert_allclose(dV, tv.grad.numpy(), atol=1e-13)


def test_backward_row_and_column_subsets():
    rng = np.random.RandomState(40)
    q, k, v, dO = rnd(rng, 12, 8), rnd(rng, 15, 8), rnd(rng, 15, 8), rnd(rng, 12, 8)
    O, lse = A.attn_fwd(q, k, v, 0.5)
    D = A.bwd_delta(dO, O)
    dQ = A.attn_bwd_dq(q, k, v, dO, lse, D, 0.5)
    dK, dV = A.attn_bwd_dkdv(q, k, v, dO, lse, D, 0.5)
    assert np.array_equal(A.attn_bwd_dq(q, k, v, dO, lse, D, 0.5, rows=[11, 2]), dQ[[11, 2]])
    sk, sv = A.attn_bwd_dkdv(q, k, v, dO, lse, D, 0.5, cols=[14, 0, 3])
    assert np.array_equal(sk, dK[[14, 0, 3]]) and np.array_equal(sv, dV[[14, 0, 3]])


# ------------------------------------------------------------------ placement level

def _small_placement():
    # 2 whole sequences, one long sequence as 2x2 chunk tasks, one CP shard (1 q x 3 kv)
    return W.make_placement("t", 2, 8, 123, [5, 9], [(2, 2, 6), (1, 3, 7)])


def _tensors(p, rng):
    return (rnd(rng, p.total_q, p.n_heads, p.head_dim), rnd(rng, p.total_kv, p.n_heads, p.head_dim),
            rnd(rng, p.total_kv, p.n_heads, p.head_dim), rnd(rng, p.total_q, p.n_heads, p.head_dim))


def test_placement_layout_of_small_case():
    p = _small_placement()
    assert p.cu_seqlens == (0, 5, 14)
    assert p.total_q == 14 + 12 + 7 and p.total_kv == 14 + 12 + 21
    assert p.shards[:4] == ((14, 6, 14, 6, 0), (14, 6, 20, 6, 0), (20, 6, 14, 6, 0), (20, 6, 20, 6, 0))
    assert p.shards[4:] == ((26, 7, 26, 7, 1), (26, 7, 33, 7, 1), (26, 7, 40, 7, 1))
    probs = A.logical_problems(p)
    assert [(x["q_off"], x["q_len"]) for x in probs] == [(0, 5), (5, 9), (14, 6), (20, 6), (26, 7)]
    assert probs[4]["kv_ranges"] == [(26, 7), (33, 7), (40, 7)]


def test_placement_forward_against_per_sequence_library_calls():
    p = _small_placement()
    Q, K, V, _ = _tensors(p, np.random.RandomState(50))
    out = A.placement_fwd(p, Q, K, V)
    assert out["merge_vs_direct"] < 1e-13
    for h in range(p.n_heads):
        for (qo, ql, ko, kl) in [(0, 5, 0, 5), (5, 9, 5, 9), (14, 6, 14, 12), (20, 6, 14, 12), (26, 7, 26, 21)]:
            Ot, lt = _torch_ref(Q[qo:qo + ql, h], K[ko:ko + kl, h], V[ko:ko + kl, h], p.scale)
            np.testing.assert_allclose(out["O"][qo:qo + ql, h], Ot, atol=1e-13)
            np.testing.assert_allclose(out["LSE"][h, qo:qo + ql], lt, atol=1e-13)
    # a shard task's partial is normalised within its own chunk
    Ot, lt = _torch_ref(Q[26:33, 1], K[33:40, 1], V[33:40, 1], p.scale)
    np.testing.assert_allclose(out["partials"][5][0][:, 1], Ot, atol=1e-13)
    np.testing.assert_allclose(out["partials"][5][1][1], lt, atol=1e-13)


def test_placement_isolation_between_sequences():
    p = _small_placement()
    rng = np.random.RandomState(51)
    Q, K, V, _ = _tensors(p, rng)
    a = A.placement_fwd(p, Q, K, V)
    Q2, K2, V2 = Q.copy(), K.copy(), V.copy()
    Q2[5:14] += 3.0; K2[5:14] *= -2.0; V2[5:14] += 100.0     # perturb whole sequence 1 only
    b = A.placement_fwd(p, Q2, K2, V2)
    keep = np.r_[0:5, 14:p.total_q]
    assert np.array_equal(a["O"][keep], b["O"][keep])
    assert np.array_equal(a["LSE"][:, keep], b["LSE"][:, keep])
    assert not np.array_equal(a["O"][5:14], b["O"][5:14])


def test_placement_backward_direct_equals_shard_form_and_autograd():
    p = _small_placement()
    Q, K, V, dO = _tensors(p, np.random.RandomState(52))
    g = A.placement_bwd(p, Q, K, V, dO)
    s = A.placement_bwd_shard_form(p, Q, K, V, dO)
    for name in ("dQ", "dK", "dV"):
        np.testing.assert_allclose(g[name], s[name], atol=1e-12)
    # library autograd over the same logical problems
    tQ, tK, tV = (torch.from_numpy(x.copy()).requires_grad_(True) for x in (Q, K, V))
    loss = 0
    for (qo, ql, ko, kl) in [(0, 5, 0, 5), (5, 9, 5, 9), (14, 6, 14, 12), (20, 6, 14, 12), (26, 7, 26, 21)]:
        o = torch.nn.functional.scaled_dot_product_attention(
            tQ[qo:qo + ql].transpose(0, 1), tK[ko:ko + kl].transpose(0, 1),
            tV[ko:ko + kl].transpose(0, 1), scale=p.scale)
        loss = loss + (o.transpose(0, 1) * torch.from_numpy(dO[qo:qo + ql])).sum()
    loss.backward()
    np.testing.assert_allclose(g["dQ"], tQ.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(g["dK"], tK.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(g["dV"], tV.grad.numpy(), atol=1e-12)


def test_placement_backward_finite_differences_through_shard_and_merge():
    p = W.make_placement("fd", 1, 4, 5, [3], [(1, 2, 4)])
    Q, K, V, dO = _tensors(p, np.random.RandomState(53))

    def loss():
        return float(np.sum(A.placement_fwd(p, Q, K, V, with_partials=False)["O"] * dO))

    g = A.placement_bwd(p, Q, K, V, dO)
    eps = 1e-5
    for arr, name in ((Q, "dQ"), (K, "dK"), (V, "dV")):
        fd = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            old = arr[idx]
            arr[idx] = old + eps; lp = loss()
            arr[idx] = old - eps; lm = loss()
            arr[idx] = old
            fd[idx] = (lp - lm) / (2 * eps)
        assert np.linalg.norm(fd - g[name]) / np.linalg.norm(g[name]) < 1e-7


def test_head_range_placement_against_per_head_library_calls():
    """Tasks over head ranges: each head of a row block belongs to the problems that list it, and only
    to those.  Library routine + autograd per (problem, head); (row, head) pairs no problem covers get
    no output and no gradient."""
    whole = [(0, 5, 0, 3), (5, 9, 0, 1), (5, 9, 1, 2)]          # two sequences share rows 5..13 on disjoint heads
    shards = [(14, 6, 14, 4, 0, 0, 2), (14, 6, 18, 7, 0, 0, 2), (14, 6, 14, 11, 1, 2, 1)]
    p = W.head_range_placement("hr", 3, 8, 77, whole, shards, 20, 25)
    probs = A.logical_problems(p)
    assert [(x["q_off"], x["q_len"], x["heads"]) for x in probs] == \
        [(0, 5, (0, 3)), (5, 9, (0, 1)), (5, 9, (1, 2)), (14, 6, (0, 2)), (14, 6, (2, 1))]
    assert probs[3]["kv_ranges"] == [(14, 4), (18, 7)] and probs[4]["kv_ranges"] == [(14, 11)]
    Q, K, V, dO = _tensors(p, np.random.RandomState(54))
    out = A.placement_fwd(p, Q, K, V)
    g = A.placement_bwd(p, Q, K, V, dO)
    s = A.placement_bwd_shard_form(p, Q, K, V, dO)
    tQ, tK, tV = (torch.from_numpy(x.copy()).requires_grad_(True) for x in (Q, K, V))
    loss = 0
    covered = np.zeros((p.total_q, p.n_heads), dtype=bool)
    for (qo, ql, ko, kl, hb, hc) in [(0, 5, 0, 5, 0, 3), (5, 9, 5, 9, 0, 1), (5, 9, 5, 9, 1, 2),
                                     (14, 6, 14, 11, 0, 2), (14, 6, 14, 11, 2, 1)]:
        for h in range(hb, hb + hc):
            Ot, lt = _torch_ref(Q[qo:qo + ql, h], K[ko:ko + kl, h], V[ko:ko + kl, h], p.scale)
            np.testing.assert_allclose(out["O"][qo:qo + ql, h], Ot, atol=1e-13)
            np.testing.assert_allclose(out["LSE"][h, qo:qo + ql], lt, atol=1e-13)
            covered[qo:qo + ql, h] = True
            o = torch.nn.functional.scaled_dot_product_attention(
                tQ[qo:qo + ql, h][None], tK[ko:ko + kl, h][None], tV[ko:ko + kl, h][None], scale=p.scale)[0]
            loss = loss + (o * torch.from_numpy(dO[qo:qo + ql, h])).sum()
    loss.backward()
    assert np.isnan(out["LSE"].T[~covered]).all() and not np.isnan(out["LSE"].T[covered]).any()
    for name, ref in (("dQ", tQ.grad), ("dK", tK.grad), ("dV", tV.grad)):
        np.testing.assert_allclose(g[name], ref.numpy(), atol=1e-12)
        np.testing.assert_allclose(s[name], ref.numpy(), atol=1e-12)
    assert np.all(g["dQ"][~covered] == 0)


# ------------------------------------------------------------------ config 1: generator + library

def _cfg1_tensors():
    p = W.config(1)
    T = {t: np.stack([W.head_tensor_for(p, t, h).astype(np.float64) for h in range(p.n_heads)], 1)
         for t in ("Q", "K", "V", "dO")}
    return p, T


def test_generator_sanity_values():
    p, T = _cfg1_tensors()
    assert (p.total_q, p.total_kv, p.cu_seqlens) == (3816, 3816, (0, 256, 768, 1768))
    assert p.shards == ((1768, 1024, 1768, 1024, 0), (1768, 1024, 2792, 1024, 0),
                        (2792, 1024, 1768, 1024, 0), (2792, 1024, 2792, 1024, 0))
    # the same stream through torch's own float64 -> float32 -> bfloat16 conversion
    rs = np.random.RandomState(0 * 1000003 + 0 * 10007 + 0)
    ref = torch.from_numpy(rs.standard_normal((3816, 64))).to(torch.float32).to(torch.bfloat16)
    assert np.array_equal(T["Q"][:, 0, :], ref.double().numpy())
    bits = W.f32_to_bf16_bits(W.head_tensor_for(p, "Q", 0))
    assert np.array_equal(bits.view(np.int16), ref.view(torch.int16).numpy())


def test_config1_against_library_and_stored_digests():
    p, T = _cfg1_tensors()
    out = A.placement_fwd(p, T["Q"], T["K"], T["V"])
    g = A.placement_bwd(p, T["Q"], T["K"], T["V"], T["dO"])
    # live library comparison on every logical problem
    tQ, tK, tV = (torch.from_numpy(T[t].copy()).requires_grad_(True) for t in ("Q", "K", "V"))
    loss = 0
    for pr in A.logical_problems(p):
        qo, ql = pr["q_off"], pr["q_len"]
        ko, kl = pr["kv_ranges"][0][0], sum(r[1] for r in pr["kv_ranges"])
        qh = tQ[qo:qo + ql].transpose(0, 1); kh = tK[ko:ko + kl].transpose(0, 1); vh = tV[ko:ko + kl].transpose(0, 1)
        o = torch.nn.functional.scaled_dot_product_attention(qh, kh, vh, scale=p.scale).transpose(0, 1)
        np.testing.assert_allclose(out["O"][qo:qo + ql], o.detach().numpy(), atol=1e-12)
        lse = torch.logsumexp((qh @ kh.transpose(1, 2)) * p.scale, -1)
        np.testing.assert_allclose(out["LSE"][:, qo:qo + ql], lse.detach().numpy(), atol=1e-12)
        loss = loss + (o * torch.from_numpy(T["dO"][qo:qo + ql])).sum()
    loss.backward()
    for name, t in (("dQ", tQ), ("dK", tK), ("dV", tV)):
        np.testing.assert_allclose(g[name], t.grad.numpy(), atol=1e-11)
    # digests stored by tests/golden/make_config1_digests.py (which calls only the oracle)
    fx = load_fixture("config1_digests.txt")
    for name, x in (("O", out["O"]), ("LSE", out["LSE"]), ("dQ", g["dQ"]), ("dK", g["dK"]), ("dV", g["dV"])):
        s, sa, first, last = fx[name]
        assert abs(x.sum() - s) <= 1e-9 * max(1.0, sa)
        assert abs(np.abs(x).sum() - sa) <= 1e-9 * sa
        assert abs(x.ravel()[0] - first) <= 1e-12 and abs(x.ravel()[-1] - last) <= 1e-12
