"""TEST INFRASTRUCTURE: Python front end of the fp64 CPU oracle (plain C underneath).

Nothing here is used by the product path.  Per-problem functions take ONE head as 2-D
float64 arrays [rows, d]; placement-level functions walk a placement (whole sequences
plus context-parallel shard tasks, paper Section IV-D) and evaluate each logical
attention problem by its definition.

Logical problems of a placement
  * every whole sequence i: queries = keys = rows [cu[i], cu[i+1]);
  * every merge group (shard tasks sharing one query range): queries = that range, keys =
    the union of the group's K/V chunks.  The "direct form" evaluates this as one
    problem over the concatenated keys; the "merge form" evaluates each shard task on its
    own chunk and combines the (O_t, LSE_t) pairs with the log-sum-exp merge.  Context
    parallelism computes exact attention, so both must agree to rounding.
"""
from __future__ import annotations

import ctypes
from typing import Callable, Dict, List, Optional, Sequence, Tuple, Union

import numpy as np

from . import build as _build

_lib = None
_dp = ctypes.POINTER(ctypes.c_double)
_lp = ctypes.POINTER(ctypes.c_long)


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(_build.build())
        L.orc_num_threads.restype = ctypes.c_int
        for name in ("orc_attn_fwd", "orc_lse_merge", "orc_attn_bwd_delta",
                     "orc_attn_bwd_dq", "orc_attn_bwd_dkdv"):
            getattr(L, name).restype = None
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _view(a: np.ndarray) -> Tuple[ctypes.c_void_p, int]:
    """Pointer and row stride (elements) of a 2-D float64 array with unit inner stride."""
    assert a.dtype == np.float64 and a.ndim == 2
    assert a.shape[1] == 1 or a.strides[1] == 8, "inner dimension must be contiguous"
    assert a.strides[0] % 8 == 0
    return ctypes.c_void_p(a.ctypes.data), a.strides[0] // 8


def _vec(a: np.ndarray) -> ctypes.c_void_p:
    assert a.dtype == np.float64 and a.ndim == 1 and (a.size <= 1 or a.strides[0] == 8)
    return ctypes.c_void_p(a.ctypes.data)


def _idx(rows) -> Tuple[Optional[np.ndarray], ctypes.c_void_p]:
    if rows is None:
        return None, ctypes.c_void_p(0)
    r = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    assert ctypes.sizeof(ctypes.c_long) == 8
    return r, ctypes.c_void_p(r.ctypes.data)


# --------------------------------------------------------------------------------------
# One logical problem, one head
# --------------------------------------------------------------------------------------

def attn_fwd(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float,
             rows=None) -> Tuple[np.ndarray, np.ndarray]:
    """O = softmax(scale * q k^T) v and LSE = logsumexp(scale * q k^T) for one head.

    ``rows`` restricts the computation to the listed query rows (outputs in that order).
    """
    d = q.shape[1]
    n_kv = k.shape[0]
    assert k.shape[1] == d and v.shape == k.shape
    ridx, rptr = _idx(rows)
    n_rows = q.shape[0] if ridx is None else ridx.size
    O = np.zeros((n_rows, d), dtype=np.float64)
    lse = np.zeros((n_rows,), dtype=np.float64)
    qp, ldq = _view(q)
    kp, ldk = _view(k) if n_kv else (ctypes.c_void_p(0), d)
    vp, ldv = _view(v) if n_kv else (ctypes.c_void_p(0), d)
    op, ldo = _view(O) if n_rows else (ctypes.c_void_p(0), d)
    if n_rows:
        lib().orc_attn_fwd(qp, ctypes.c_long(ldq), kp, ctypes.c_long(ldk), vp, ctypes.c_long(ldv),
                           ctypes.c_long(n_kv), ctypes.c_int(d), ctypes.c_double(scale),
                           rptr, ctypes.c_long(n_rows), op, ctypes.c_long(ldo), _vec(lse))
    return O, lse


def lse_merge(parts: Sequence[Tuple[np.ndarray, np.ndarray]]) -> Tuple[np.ndarray, np.ndarray]:
    """Combine partial (O_t, LSE_t) of the same query rows over disjoint key sets."""
    assert len(parts) >= 1
    n_rows, d = parts[0][0].shape
    Os = [np.ascontiguousarray(p[0], dtype=np.float64) for p in parts]
    Ls = [np.ascontiguousarray(p[1], dtype=np.float64) for p in parts]
    for o, l in zip(Os, Ls):
        assert o.shape == (n_rows, d) and l.shape == (n_rows,)
    O = np.zeros((n_rows, d), dtype=np.float64)
    lse = np.zeros((n_rows,), dtype=np.float64)
    n = len(parts)
    optrs = (ctypes.c_void_p * n)(*[o.ctypes.data for o in Os])
    lptrs = (ctypes.c_void_p * n)(*[l.ctypes.data for l in Ls])
    if n_rows:
        lib().orc_lse_merge(ctypes.c_int(n), optrs, ctypes.c_long(d), lptrs,
                            ctypes.c_long(n_rows), ctypes.c_int(d),
                            ctypes.c_void_p(O.ctypes.data), ctypes.c_long(d), _vec(lse))
    return O, lse


def bwd_delta(dO: np.ndarray, O: np.ndarray) -> np.ndarray:
    """D_i = sum_c dO[i,c] * O[i,c]."""
    n_q, d = dO.shape
    D = np.zeros((n_q,), dtype=np.float64)
    if n_q:
        dop, lddo = _view(dO)
        op, ldo = _view(O)
        lib().orc_attn_bwd_delta(dop, ctypes.c_long(lddo), op, ctypes.c_long(ldo),
                                 ctypes.c_long(n_q), ctypes.c_int(d), _vec(D))
    return D


def attn_bwd_dq(q, k, v, dO, lse, D, scale, rows=None) -> np.ndarray:
    """dQ rows (all, or those listed) of one problem; lse and D cover every query row."""
    d = q.shape[1]
    n_kv = k.shape[0]
    ridx, rptr = _idx(rows)
    n_rows = q.shape[0] if ridx is None else ridx.size
    dQ = np.zeros((n_rows, d), dtype=np.float64)
    lse = np.ascontiguousarray(lse, dtype=np.float64)
    D = np.ascontiguousarray(D, dtype=np.float64)
    if n_rows and n_kv:
        qp, ldq = _view(q); kp, ldk = _view(k); vp, ldv = _view(v); dop, lddo = _view(dO)
        dqp, lddq = _view(dQ)
        lib().orc_attn_bwd_dq(qp, ctypes.c_long(ldq), kp, ctypes.c_long(ldk), vp, ctypes.c_long(ldv),
                              dop, ctypes.c_long(lddo), _vec(lse),
                              _vec(D), ctypes.c_long(n_kv), ctypes.c_int(d),
                              ctypes.c_double(scale), rptr, ctypes.c_long(n_rows),
                              dqp, ctypes.c_long(lddq))
    return dQ


def attn_bwd_dkdv(q, k, v, dO, lse, D, scale, cols=None) -> Tuple[np.ndarray, np.ndarray]:
    """dK, dV rows (all keys, or those listed) of one problem."""
    d = q.shape[1]
    n_q = q.shape[0]
    cidx, cptr = _idx(cols)
    n_cols = k.shape[0] if cidx is None else cidx.size
    dK = np.zeros((n_cols, d), dtype=np.float64)
    dV = np.zeros((n_cols, d), dtype=np.float64)
    lse = np.ascontiguousarray(lse, dtype=np.float64)
    D = np.ascontiguousarray(D, dtype=np.float64)
    if n_cols and n_q:
        qp, ldq = _view(q); kp, ldk = _view(k); vp, ldv = _view(v); dop, lddo = _view(dO)
        dkp, lddk = _view(dK); dvp, lddv = _view(dV)
        lib().orc_attn_bwd_dkdv(qp, ctypes.c_long(ldq), kp, ctypes.c_long(ldk), vp, ctypes.c_long(ldv),
                                dop, ctypes.c_long(lddo), _vec(lse),
                                _vec(D), ctypes.c_long(n_q), ctypes.c_int(d),
                                ctypes.c_double(scale), cptr, ctypes.c_long(n_cols),
                                dkp, ctypes.c_long(lddk), dvp, ctypes.c_long(lddv))
    return dK, dV


def attn_bwd(q, k, v, dO, scale) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """dQ, dK, dV of one problem, one head, from the oracle's own fp64 O and LSE."""
    O, lse = attn_fwd(q, k, v, scale)
    D = bwd_delta(dO, O)
    dQ = attn_bwd_dq(q, k, v, dO, lse, D, scale)
    dK, dV = attn_bwd_dkdv(q, k, v, dO, lse, D, scale)
    return dQ, dK, dV


# --------------------------------------------------------------------------------------
# Placement level
# --------------------------------------------------------------------------------------

HeadSource = Union[np.ndarray, Callable[[int], np.ndarray]]


def _head(x: HeadSource, h: int) -> np.ndarray:
    """[rows, d] float64 block of head h from a [rows, H, d] array or a per-head callable."""
    if callable(x):
        return np.ascontiguousarray(x(h), dtype=np.float64)
    return np.ascontiguousarray(x[:, h, :], dtype=np.float64)


def logical_problems(p) -> List[dict]:
    """Direct-form problems of a placement, in placement order.

    Each entry: q_off, q_len, kv_ranges [(off, len), ...] in ascending shard order, ``shards``
    (indices into p.shards; empty for a whole sequence) and ``heads`` = (head_begin, head_count): the
    heads for which the problem exists (all heads unless the placement gives head ranges -- a
    sequence under Ulysses parallelism holds its tokens for a subset of the heads; the attention of
    each of those heads is the same definition)."""
    probs = []
    if hasattr(p, "whole_descs"):
        whole = p.whole_descs()
        shard_heads = p.shard_head_ranges()
    else:
        whole = [(p.cu_seqlens[i], p.cu_seqlens[i + 1] - p.cu_seqlens[i], 0, p.n_heads)
                 for i in range(len(p.cu_seqlens) - 1)]
        shard_heads = [(0, p.n_heads)] * len(p.shards)
    for (a, l, hb, hc) in whole:
        probs.append(dict(q_off=a, q_len=l, kv_ranges=[(a, l)], shards=[], heads=(hb, hc)))
    groups: Dict[Tuple[int, int, int, int], dict] = {}
    for si, (qo, ql, ko, kl, sid) in enumerate(p.shards):
        hb, hc = shard_heads[si]
        g = groups.get((qo, ql, hb, hc))
        if g is None:
            g = dict(q_off=qo, q_len=ql, kv_ranges=[], shards=[], heads=(hb, hc))
            groups[(qo, ql, hb, hc)] = g
            probs.append(g)
        g["kv_ranges"].append((ko, kl))
        g["shards"].append(si)
    return probs


def _has_head(pr: dict, h: int) -> bool:
    hb, hc = pr["heads"]
    return hb <= h < hb + hc


def _gather_kv(x: np.ndarray, ranges) -> np.ndarray:
    if len(ranges) == 1:
        o, l = ranges[0]
        return x[o:o + l]
    return np.concatenate([x[o:o + l] for o, l in ranges], axis=0)


def placement_fwd(p, Q: HeadSource, K: HeadSource, V: HeadSource, scale: Optional[float] = None,
                  heads: Optional[Sequence[int]] = None, with_partials: bool = True,
                  merge_check_tol: float = 1e-12):
    """Forward of a whole placement for the listed heads (default: all).

    Returns dict: O [Tq, nh, d], LSE [nh, Tq] (direct form), ``partials`` {shard index:
    (O_t [q_len, nh, d], LSE_t [nh, q_len])} with each O_t normalised within its own K/V
    chunk, ``heads``, and ``merge_vs_direct`` = largest |merge form - direct form| seen
    (asserted <= merge_check_tol, relative to max(1, |value|))."""
    scale = p.scale if scale is None else scale
    hs = list(range(p.n_heads)) if heads is None else list(heads)
    d = p.head_dim
    O = np.zeros((p.total_q, len(hs), d), dtype=np.float64)
    LSE = np.full((len(hs), p.total_q), np.nan, dtype=np.float64)
    partials = {si: (np.zeros((s[1], len(hs), d)), np.zeros((len(hs), s[1])))
                for si, s in enumerate(p.shards)} if with_partials else {}
    worst = 0.0
    probs = logical_problems(p)
    for hi, h in enumerate(hs):
        q, k, v = _head(Q, h), _head(K, h), _head(V, h)
        for pr in probs:
            if not _has_head(pr, h):
                continue
            qo, ql = pr["q_off"], pr["q_len"]
            kk = _gather_kv(k, pr["kv_ranges"])
            vv = _gather_kv(v, pr["kv_ranges"])
            o, l = attn_fwd(q[qo:qo + ql], kk, vv, scale)
            O[qo:qo + ql, hi, :] = o
            LSE[hi, qo:qo + ql] = l
            if with_partials and pr["shards"]:
                parts = []
                for si in pr["shards"]:
                    _, _, ko, kl, _ = p.shards[si]
                    ot, lt = attn_fwd(q[qo:qo + ql], k[ko:ko + kl], v[ko:ko + kl], scale)
                    partials[si][0][:, hi, :] = ot
                    partials[si][1][hi, :] = lt
                    parts.append((ot, lt))
                om, lm = lse_merge(parts)
                fin = np.isfinite(l)
                e1 = np.max(np.abs(om - o) / np.maximum(1.0, np.abs(o))) if o.size else 0.0
                e2 = np.max(np.abs(lm[fin] - l[fin]) / np.maximum(1.0, np.abs(l[fin]))) if fin.any() else 0.0
                assert np.array_equal(np.isfinite(lm), fin)
                worst = max(worst, float(e1), float(e2))
    assert worst <= merge_check_tol, f"merge form deviates from direct form by {worst}"
    return dict(O=O, LSE=LSE, partials=partials, heads=hs, merge_vs_direct=worst)


def placement_bwd(p, Q: HeadSource, K: HeadSource, V: HeadSource, dO: HeadSource,
                  scale: Optional[float] = None, heads: Optional[Sequence[int]] = None):
    """Backward of a whole placement in direct form for the listed heads.

    dK/dV rows of a K/V range that serves several query ranges receive the sum over them.
    Returns dict dQ [Tq, nh, d], dK, dV [Tkv, nh, d]."""
    scale = p.scale if scale is None else scale
    hs = list(range(p.n_heads)) if heads is None else list(heads)
    d = p.head_dim
    dQ = np.zeros((p.total_q, len(hs), d), dtype=np.float64)
    dK = np.zeros((p.total_kv, len(hs), d), dtype=np.float64)
    dV = np.zeros((p.total_kv, len(hs), d), dtype=np.float64)
    probs = logical_problems(p)
    for hi, h in enumerate(hs):
        q, k, v, do = _head(Q, h), _head(K, h), _head(V, h), _head(dO, h)
        for pr in probs:
            if not _has_head(pr, h):
                continue
            qo, ql = pr["q_off"], pr["q_len"]
            kk = _gather_kv(k, pr["kv_ranges"])
            vv = _gather_kv(v, pr["kv_ranges"])
            gq, gk, gv = attn_bwd(q[qo:qo + ql], kk, vv, do[qo:qo + ql], scale)
            dQ[qo:qo + ql, hi, :] += gq
            pos = 0
            for (ko, kl) in pr["kv_ranges"]:
                dK[ko:ko + kl, hi, :] += gk[pos:pos + kl]
                dV[ko:ko + kl, hi, :] += gv[pos:pos + kl]
                pos += kl
    return dict(dQ=dQ, dK=dK, dV=dV, heads=hs)


def placement_bwd_shard_form(p, Q, K, V, dO, scale=None, heads=None):
    """Backward evaluated task by task: each shard task uses the MERGED LSE and the D of
    the final O, and contributions are summed.  Must equal the direct form to rounding."""
    scale = p.scale if scale is None else scale
    hs = list(range(p.n_heads)) if heads is None else list(heads)
    d = p.head_dim
    fwd = placement_fwd(p, Q, K, V, scale, heads=hs, with_partials=False)
    dQ = np.zeros((p.total_q, len(hs), d)); dK = np.zeros((p.total_kv, len(hs), d)); dV = np.zeros_like(dK)
    tasks = []
    for pr in logical_problems(p):
        if pr["shards"]:
            tasks += [tuple(p.shards[si][:4]) + (pr["heads"],) for si in pr["shards"]]
        else:
            tasks.append((pr["q_off"], pr["q_len"], pr["q_off"], pr["q_len"], pr["heads"]))
    for hi, h in enumerate(hs):
        q, k, v, do = _head(Q, h), _head(K, h), _head(V, h), _head(dO, h)
        o_h = np.ascontiguousarray(fwd["O"][:, hi, :])
        D = bwd_delta(do, o_h)
        lse = np.ascontiguousarray(fwd["LSE"][hi])
        for (qo, ql, ko, kl, (hb, hc)) in tasks:
            if ql == 0 or kl == 0 or not (hb <= h < hb + hc):
                continue
            qs, ks, vs, dos = q[qo:qo + ql], k[ko:ko + kl], v[ko:ko + kl], do[qo:qo + ql]
            ls, Ds = lse[qo:qo + ql], D[qo:qo + ql]
            dQ[qo:qo + ql, hi, :] += attn_bwd_dq(qs, ks, vs, dos, ls, Ds, scale)
            gk, gv = attn_bwd_dkdv(qs, ks, vs, dos, ls, Ds, scale)
            dK[ko:ko + kl, hi, :] += gk
            dV[ko:ko + kl, hi, :] += gv
    return dict(dQ=dQ, dK=dK, dV=dV, heads=hs)
