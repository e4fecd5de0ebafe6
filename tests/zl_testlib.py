"""Shared helpers of the GPU parity tests: seeded inputs, GPU runs through the C ABI
(via the Python binding), oracle runs, and the tolerance checks."""
from __future__ import annotations

import numpy as np
import torch

import zl_workloads as W

# Graded tolerances (forward O, LSE; backward relative Frobenius error).
TOL_O_MAX, TOL_O_MEAN, TOL_LSE_MAX, TOL_GRAD_REL = 2e-2, 2e-3, 1e-3, 1e-2
# Tighter internal gates, about 3x the error of an fp32-accumulate / bf16-P emulation.
# GATE_O_MAX bounds the error in excess of the output's own bf16 rounding (2^-8 * |O|).
GATE_O_MAX, GATE_LSE_MAX, GATE_GRAD_REL = 3e-3, 2e-5, 5e-3

# Row-wise gradient gate: a relative Frobenius norm over a whole tensor cannot see one wrong row among
# tens of thousands, so every (row, head) vector g is also held to
#     ||g - ref|| <= TOL_GRAD_ROW * (||ref|| + GRAD_ROW_FLOOR * rms),   rms = root mean square row norm of ref,
# where the floor keeps rows whose own gradient is small relative to the tensor from dividing by ~0: a
# query whose softmax is nearly one-hot has a tiny dQ, yet its error is set by D = rowsum(dO o O) being
# formed from the stored bf16 O (|dO . (O_bf16 - O)| ~ 1e-2 at d = 128), which does not shrink with the
# row.  Measured: 0.04 * rms on such a row of a 2-token sequence, <= 0.01 elsewhere; a wrong row gives ~0.8.
# GRAD_ROW_ABS covers tensors that are exactly zero in the oracle (a single key: dQ = dK = 0).
TOL_GRAD_ROW, GRAD_ROW_FLOOR, GRAD_ROW_ABS = 3e-2, 0.25, 1e-3

SENTINEL = 768.0  # exactly representable in bf16


def bits(p, tensor, workers=0):
    return W.packed_bf16_bits(p, tensor, workers=workers)


def random_bits(rng, rows, H, d, scale=1.0):
    x = (rng.standard_normal((rows, H, d)) * scale).astype(np.float32)
    return W.f32_to_bf16_bits(W._bf16_round_f32(x))


def to_dev(b: np.ndarray, device="cuda"):
    return torch.from_numpy(b.view(np.int16)).to(device).view(torch.bfloat16)


def to_f64(b: np.ndarray) -> np.ndarray:
    return W.bf16_bits_to_f32(b).astype(np.float64)


def dev_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


class EngineRun:
    """Runs forward (+merge) and optionally backward for a placement through the binding."""

    def __init__(self, p, scale=None, flags=0):
        import paper_2608_01150_b200 as Z
        self.Z = Z
        self.p = p
        self.scale = p.scale if scale is None else scale
        if p.has_head_ranges:
            self.h = Z.build_tasks_heads(p.whole_descs(), p.shards, p.shard_head_ranges(), p.total_q, p.total_kv,
                                         p.n_heads, p.head_dim, flags=flags)
        else:
            self.h = Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, p.n_heads, p.head_dim, flags=flags)
        self.info = self.h.info
        # ZL_TEST_BWD_KERNEL=1|2 runs the whole suite on one of the two backward main kernels
        import os
        k = int(os.environ.get("ZL_TEST_BWD_KERNEL", "0"))
        if k == 1 or (k == 2 and p.head_dim == 128):
            self.h.set_bwd_kernel(k)

    def forward(self, Q, K, V, merge=True):
        p, H, d = self.p, self.p.n_heads, self.p.head_dim
        dev = Q.device
        O = torch.full((p.total_q, H, d), SENTINEL, dtype=torch.bfloat16, device=dev)
        LSE = torch.full((H, p.total_q), SENTINEL, dtype=torch.float32, device=dev)
        pr = int(self.info.partial_rows)
        OP = torch.full((max(pr, 1), H, d), SENTINEL, dtype=torch.float32, device=dev)
        LP = torch.full((H, max(pr, 1)), SENTINEL, dtype=torch.float32, device=dev)
        self.Z.coalesced_attn_fwd(self.h, Q, K, V, self.scale, O, LSE, OP, LP)
        if merge:
            self.Z.lse_merge(self.h, OP, LP, O, LSE)
        torch.cuda.synchronize()
        code, where = self.h.last_device_status()
        assert code == 0, f"device status {code} at {where}"
        return O, LSE, OP, LP

    def backward(self, Q, K, V, O, LSE, dO):
        p, H, d = self.p, self.p.n_heads, self.p.head_dim
        dev = Q.device
        dQ = torch.full((p.total_q, H, d), SENTINEL, dtype=torch.bfloat16, device=dev)
        dK = torch.full((p.total_kv, H, d), SENTINEL, dtype=torch.bfloat16, device=dev)
        dV = torch.full((p.total_kv, H, d), SENTINEL, dtype=torch.bfloat16, device=dev)
        ws = torch.empty(int(self.info.bwd_workspace_bytes) + 256, dtype=torch.uint8, device=dev)
        self.Z.coalesced_attn_bwd(self.h, Q, K, V, O, LSE, dO, self.scale, dQ, dK, dV, ws,
                                  int(self.info.bwd_workspace_bytes))
        torch.cuda.synchronize()
        code, where = self.h.last_device_status()
        assert code == 0, f"device status {code} at {where}"
        return dQ, dK, dV


def covered_rows(p):
    """Boolean masks [rows, H] of the (row, head) pairs of Q-space / KV-space covered by at least one task."""
    q = np.zeros((p.total_q, p.n_heads), dtype=bool)
    kv = np.zeros((p.total_kv, p.n_heads), dtype=bool)
    for (o, l, hb, hc) in p.whole_descs():
        q[o:o + l, hb:hb + hc] = True
        kv[o:o + l, hb:hb + hc] = True
    for (qo, ql, ko, kl, _), (hb, hc) in zip(p.shards, p.shard_head_ranges()):
        if ql > 0:
            q[qo:qo + ql, hb:hb + hc] = True
            if kl > 0:
                kv[ko:ko + kl, hb:hb + hc] = True
    return q, kv


def check_forward(p, O_gpu, LSE_gpu, ref, tol=(TOL_O_MAX, TOL_O_MEAN, TOL_LSE_MAX), heads=None):
    """Compare GPU O/LSE (torch tensors) with oracle dict (placement_fwd) on covered (row, head) pairs."""
    hs = list(range(p.n_heads)) if heads is None else list(heads)
    qmask = covered_rows(p)[0][:, hs]                  # [rows, nh]
    Og = dev_to_f64(O_gpu)[:, hs, :]
    Lg = dev_to_f64(LSE_gpu)[hs, :].T                  # [rows, nh]
    Lr = ref["LSE"].T
    eo = np.abs(Og[qmask] - ref["O"][qmask])
    fin = np.isfinite(Lr[qmask])
    el = np.abs(Lg[qmask][fin] - Lr[qmask][fin])
    assert np.array_equal(np.isneginf(Lg[qmask]), np.isneginf(Lr[qmask]))
    # error beyond the unavoidable bf16 rounding of the output (half an ulp = 2^-9 relative)
    excess = eo - np.abs(ref["O"][qmask]) * 2.0 ** -8
    stats = dict(o_max=float(eo.max()) if eo.size else 0.0, o_mean=float(eo.mean()) if eo.size else 0.0,
                 lse_max=float(el.max()) if el.size else 0.0,
                 o_excess=float(excess.max()) if eo.size else 0.0)
    assert stats["o_max"] <= tol[0], stats
    assert stats["o_mean"] <= tol[1], stats
    assert stats["lse_max"] <= tol[2], stats
    # (row, head) pairs outside every task keep the sentinel
    if (~qmask).any():
        assert np.all(Og[~qmask] == SENTINEL) and np.all(Lg[~qmask] == SENTINEL)
    return stats


def rel_fro(a, b):
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / nb) if nb > 0 else float(np.linalg.norm(a))


def row_rel(g, ref, rms=None):
    """Largest row-wise relative error of g [..., d] against ref, with the floor described above.
    `rms` (root mean square row norm of the whole tensor) may be given when ref is only a sample."""
    rn = np.linalg.norm(ref, axis=-1)
    if rn.size == 0:
        return 0.0
    if rms is None:
        rms = float(np.sqrt(np.mean(rn ** 2)))
    return float(np.max(np.linalg.norm(g - ref, axis=-1) / (rn + GRAD_ROW_FLOOR * rms + GRAD_ROW_ABS)))


def check_backward(p, dQ, dK, dV, ref, tol=TOL_GRAD_REL, heads=None, row_tol=TOL_GRAD_ROW):
    hs = list(range(p.n_heads)) if heads is None else list(heads)
    qmask, kvmask = covered_rows(p)
    out = {}
    for name, g, mask in (("dQ", dQ, qmask[:, hs]), ("dK", dK, kvmask[:, hs]), ("dV", dV, kvmask[:, hs])):
        gg = dev_to_f64(g)[:, hs, :]
        out[name] = rel_fro(gg[mask], ref[name][mask])
        assert out[name] <= tol, (name, out)
        out[name + "_row"] = row_rel(gg[mask], ref[name][mask])
        assert out[name + "_row"] <= row_tol, (name, "row-wise", out)
        if (~mask).any():
            assert np.all(gg[~mask] == SENTINEL), f"{name}: (row, head) pairs outside every task were written"
    return out
