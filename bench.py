#!/usr/bin/env python
"""Benchmark of the coalesced attention engine on B200.

    python bench.py --gpus N --steps K --warmup W [--config 4] [--impl reference]

A *step* is one pass of the whole hot path over one rank-local placement: the forward
launch over whole sequences and shard tasks, the LSE merge, and the backward (preprocess,
main, dQ conversion).  The task handle is built once per placement and reused, as a
training loop reuses it for every layer.  Prints ONE JSON line (rank 0).

  value     counted TFLOP/s of forward + backward (4*Lq*Lkv*d*H forward, 2.5x that
            backward), inputs resident in HBM, device-timed with CUDA events
  e2e       the same metric with pinned HOST buffers: every step copies Q, K, V, dO to the
            device and O, LSE, dQ, dK, dV back, inside the timed region
  roofline  the backward main kernel (dominant) against the measured dense bf16 peak
  cpu_baseline  the fp64 CPU oracle timed on this machine's host cores on a bounded sample

With N > 1 (torchrun) every rank runs its own rank-local placement of the same shape
(weak scaling, no data-path collective); value is the sum over ranks divided by the
slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "coalesced attention TFLOP/s fwd and fwd+bwd; % of B200 dense BF16 peak"
# DRAM traffic of one launch of the backward main kernel (dram__bytes_read.sum + dram__bytes_write.sum, a one-pass
# ncu capture; profiles/zl_bwd_pair_kernel_cfg4_dram.txt), keyed by (configuration, kernel).  It is reported only for
# the workload and kernel it was measured on; any other combination reports null.
NCU_BWD_DRAM_BYTES = {(4, "zl_bwd_pair_kernel"): 9.32e9 + 5.42e9,
                      (3, "zl_bwd_pair_kernel"): 2.384398592e9 + 1.395509248e9,
                      (3, "zl_bwd_main_kernel"): 2.647806e9 + 1.529451e9}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.path = tempfile.mktemp(prefix="zl_clocks_", suffix=".csv")
        self.proc = None
        try:
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=self.fh, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, mx, pw = [], [], []
        reasons = set()
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [x.strip() for x in line.split(",")]
                    if len(parts) < 8:
                        continue
                    try:
                        sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
                    except ValueError:
                        continue
                    for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                        "sw_power_cap"), parts[4:8]):
                        if v.lower().startswith("active"):
                            reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            # samples under load: upper half of the power readings
            thr = statistics.median(pw) if pw else 0
            under = [s for s, p in zip(sm, pw) if p >= thr] or sm
            out.update(sm_mhz=statistics.median(under), sm_max_mhz=max(mx), samples=len(sm),
                       power_w_max=max(pw) if pw else None)
        out["reasons"] = sorted(reasons)
        return out


# --------------------------------------------------------------------------------------
# multi-rank helpers (also exercised on CPU with gloo by tests/test_multirank_cpu.py)
# --------------------------------------------------------------------------------------
def reduce_max_ms(ms: float, dist, device) -> float:
    """Slowest rank's time: every rank contributes its device-timed milliseconds."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tflops(world: int, flops_per_rank: float, ms_per_step: float) -> float:
    """Whole-job throughput: every rank runs its own rank-local placement of the same shape
    (weak scaling, no data-path collective), so the job does world * flops in the slowest time."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e12


# --------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------
class Workload:
    """Device tensors + task handle of one placement."""

    def __init__(self, p, device, seed_shift=0, flags=0, bwd_kernel=0):
        import torch
        import paper_2608_01150_b200 as Z
        import zl_workloads as W
        self.Z, self.p, self.torch = Z, p, torch
        H, d = p.n_heads, p.head_dim
        mk = lambda rows, s: W.device_normal_bf16((rows, H, d), p.seed * 100 + s + seed_shift, device)
        self.Q, self.K, self.V, self.dO = mk(p.total_q, 0), mk(p.total_kv, 1), mk(p.total_kv, 2), mk(p.total_q, 3)
        t0 = time.perf_counter()
        self.h = Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, H, d, flags=flags)
        self.build_ms = (time.perf_counter() - t0) * 1e3
        if bwd_kernel and not (bwd_kernel == 2 and d != 128):
            self.h.set_bwd_kernel(bwd_kernel)
        info = self.h.info
        self.O = torch.empty_like(self.Q)
        self.LSE = torch.empty(H, p.total_q, dtype=torch.float32, device=device)
        pr = max(1, int(info.partial_rows))
        self.OP = torch.empty(pr, H, d, dtype=torch.float32, device=device)
        self.LP = torch.empty(H, pr, dtype=torch.float32, device=device)
        self.dQ, self.dK, self.dV = torch.empty_like(self.Q), torch.empty_like(self.K), torch.empty_like(self.V)
        self.ws = torch.empty(max(256, int(info.bwd_workspace_bytes)), dtype=torch.uint8, device=device)
        self.merge_bytes = (sum(s[1] for s in p.shards) * H * (d * 4 + 4)
                            + sum(g[1] for g in {(s[0], s[1]) for s in p.shards}) * H * (d * 2 + 4))

    def fwd(self):
        Z, p = self.Z, self.p
        Z.coalesced_attn_fwd(self.h, self.Q, self.K, self.V, p.scale, self.O, self.LSE, self.OP, self.LP)
        Z.lse_merge(self.h, self.OP, self.LP, self.O, self.LSE)

    def bwd(self):
        self.Z.coalesced_attn_bwd(self.h, self.Q, self.K, self.V, self.O, self.LSE, self.dO, self.p.scale,
                                  self.dQ, self.dK, self.dV, self.ws)

    def step(self):
        self.fwd()
        self.bwd()

    def time_region(self, fn, n, dist=None):
        """Device time (ms) of n calls of fn, bracketed by barrier + synchronize; max over ranks."""
        torch = self.torch
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = reduce_max_ms(e0.elapsed_time(e1), dist, self.Q.device)
        if dist is not None:
            dist.barrier()
        return ms

    def make_host_buffers(self):
        torch = self.torch
        pin = lambda t: torch.empty(t.shape, dtype=t.dtype, device="cpu", pin_memory=True).copy_(t)
        self.hQ, self.hK, self.hV, self.hdO = pin(self.Q), pin(self.K), pin(self.V), pin(self.dO)
        self.hO, self.hLSE = pin(self.O), pin(self.LSE)
        self.hdQ, self.hdK, self.hdV = pin(self.dQ), pin(self.dK), pin(self.dV)
        nb = lambda *ts: sum(t.numel() * t.element_size() for t in ts)
        self.h2d_bytes = nb(self.hQ, self.hK, self.hV, self.hdO)
        self.d2h_bytes = nb(self.hO, self.hLSE, self.hdQ, self.hdK, self.hdV)

    def e2e_step(self):
        """Serial variant: copy in, compute, copy out on one stream."""
        for dst, src in ((self.Q, self.hQ), (self.K, self.hK), (self.V, self.hV), (self.dO, self.hdO)):
            dst.copy_(src, non_blocking=True)
        self.step()
        for dst, src in ((self.hO, self.O), (self.hLSE, self.LSE), (self.hdQ, self.dQ), (self.hdK, self.dK),
                         (self.hdV, self.dV)):
            dst.copy_(src, non_blocking=True)

    def e2e_pipelined(self, n, dist=None):
        """n end-to-end steps with the host<->device copies of neighbouring steps overlapped with the
        compute: inputs and outputs are double-buffered on the device, copies run on their own
        streams.  Every step still copies all its inputs from pinned host memory and all its results
        back.  Returns device milliseconds from the first H2D copy to the last D2H copy (max over ranks)."""
        torch, Z, p = self.torch, self.Z, self.p
        dev = self.Q.device
        if not hasattr(self, "_in2"):
            self._in2 = [(self.Q, self.K, self.V, self.dO),
                         tuple(torch.empty_like(t) for t in (self.Q, self.K, self.V, self.dO))]
            self._out2 = [(self.O, self.LSE, self.dQ, self.dK, self.dV),
                          tuple(torch.empty_like(t) for t in (self.O, self.LSE, self.dQ, self.dK, self.dV))]
            self._s_in, self._s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        s_comp = torch.cuda.current_stream(dev)
        h_in = (self.hQ, self.hK, self.hV, self.hdO)
        h_out = (self.hO, self.hLSE, self.hdQ, self.hdK, self.hdV)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        ev = lambda: torch.cuda.Event(enable_timing=True)
        start, end = ev(), ev()
        in_ready, comp_done, out_done = [ev() for _ in range(n)], [ev() for _ in range(n)], [ev() for _ in range(n)]
        with torch.cuda.stream(self._s_in):
            start.record()
        for i in range(n):
            b = i & 1
            Q, K, V, dO = self._in2[b]
            O, LSE, dQ, dK, dV = self._out2[b]
            with torch.cuda.stream(self._s_in):
                if i >= 2:
                    self._s_in.wait_event(comp_done[i - 2])   # input buffers of step i-2 are free
                for dst, src in zip((Q, K, V, dO), h_in):
                    dst.copy_(src, non_blocking=True)
                in_ready[i].record()
            s_comp.wait_event(in_ready[i])
            if i >= 2:
                s_comp.wait_event(out_done[i - 2])            # output buffers of step i-2 were copied out
            Z.coalesced_attn_fwd(self.h, Q, K, V, p.scale, O, LSE, self.OP, self.LP)
            Z.lse_merge(self.h, self.OP, self.LP, O, LSE)
            Z.coalesced_attn_bwd(self.h, Q, K, V, O, LSE, dO, p.scale, dQ, dK, dV, self.ws)
            comp_done[i].record()
            with torch.cuda.stream(self._s_out):
                self._s_out.wait_event(comp_done[i])
                for dst, src in zip(h_out, (O, LSE, dQ, dK, dV)):
                    dst.copy_(src, non_blocking=True)
                out_done[i].record()
        with torch.cuda.stream(self._s_out):
            end.record()
        torch.cuda.synchronize()
        ms = reduce_max_ms(start.elapsed_time(end), dist, dev)
        if dist is not None:
            dist.barrier()
        return ms


def cpu_baseline(p, target_s=12.0):
    """Times the fp64 CPU oracle (as it stands) on a bounded sample of the placement:
    forward + backward of whole sequences / sampled query rows of the first heads."""
    import numpy as np
    import zl_workloads as W
    from oracle import attention as A
    cores = A.num_threads()
    d = p.head_dim
    rng = np.random.RandomState(0)
    # sample problem: the first whole sequence of the placement (or 1024 rows of the first
    # shard's query chunk against its full key set), head by head until the time target.
    probs = A.logical_problems(p)
    pr = probs[0]
    n_q = min(pr["q_len"], 1560)
    n_kv = sum(r[1] for r in pr["kv_ranges"])
    flops_per_head = 3.5 * 4.0 * n_q * n_kv * d
    t0 = time.perf_counter()
    heads = 0
    while True:
        q = rng.standard_normal((n_q, d)); k = rng.standard_normal((n_kv, d))
        v = rng.standard_normal((n_kv, d)); do = rng.standard_normal((n_q, d))
        A.attn_bwd(q, k, v, do, p.scale)      # runs the oracle forward, then its backward
        heads += 1
        el = time.perf_counter() - t0
        if el >= target_s or heads >= 4096:
            break
    return {"value": flops_per_head * heads / el / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
            "sample": f"{heads} head-problems of {n_q} query x {n_kv} key rows, d={d}, fwd+bwd in fp64 "
                      f"({el:.1f} s), same FLOP convention",
            "seconds": el}


def flash_attn_context(device):
    """Context only, never the reference arm: the flash_attn package of this image (an mma.sync kernel family built for
    earlier GPUs) through its varlen call on configuration 2 (whole sequences only: it has no shard tasks), same
    GPU, same FLOP convention, random bf16 inputs."""
    import torch
    import zl_workloads as W
    try:
        from flash_attn import flash_attn_varlen_func
        p = W.config(2)
        H, d, T = p.n_heads, p.head_dim, p.total_q
        q, k, v = (torch.randn(T, H, d, device=device, dtype=torch.bfloat16, requires_grad=True) for _ in range(3))
        do = torch.randn(T, H, d, device=device, dtype=torch.bfloat16)
        cu = torch.tensor(p.cu_seqlens, dtype=torch.int32, device=device)
        mx = max(b - a for a, b in zip(p.cu_seqlens[:-1], p.cu_seqlens[1:]))

        def fwd():
            return flash_attn_varlen_func(q, k, v, cu, cu, mx, mx, softmax_scale=d ** -0.5, causal=False)

        def step():
            fwd().backward(do)
            q.grad = k.grad = v.grad = None

        def timed(fn, n=10):
            for _ in range(3):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(n):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / n

        ms_step = timed(step)
        with torch.no_grad():
            ms_fwd = timed(fwd)
        return {"what": "flash_attn varlen (library, mma.sync) on cfg2_images, same GPU", "fwd_ms": ms_fwd,
                "fwd_tflops": p.fwd_flops() / ms_fwd / 1e9, "fwd_bwd_ms": ms_step,
                "fwd_bwd_tflops": (p.fwd_flops() + p.bwd_flops()) / ms_step / 1e9}
    except Exception as e:  # noqa: BLE001  (package missing or not runnable on this GPU)
        return {"what": "flash_attn varlen on cfg2_images", "unavailable": repr(e)[:200]}


def run_ours(args):
    import torch
    import zl_workloads as W
    import paper_2608_01150_b200 as Z

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_mod
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    peaks, peak_kind = load_peaks()

    p = W.config(args.config)
    wl = Workload(p, device, seed_shift=rank * 7, flags=1 if args.fuse_local_chunks else 0, bwd_kernel=args.bwd_kernel)
    K, Wm = args.steps, max(3, args.warmup)
    for _ in range(Wm):
        wl.step()
    torch.cuda.synchronize()
    code, where = wl.h.last_device_status()
    if code != 0:
        raise RuntimeError(f"device status {code} at {where}")

    uuid = str(torch.cuda.get_device_properties(device).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    launches0 = Z.launch_count()
    ms_total = wl.time_region(wl.step, K, dist)
    launches = Z.launch_count() - launches0
    ms_fwd = wl.time_region(wl.fwd, K, dist)
    clocks = sampler.stop()
    ms_step = ms_total / K
    flops = p.fwd_flops() + p.bwd_flops()
    value = aggregate_tflops(world, flops, ms_step)

    # per-kernel device time (separate pass with event brackets around every launch)
    wl.h.set_kernel_timing(True)
    for _ in range(K):
        wl.step()
    kt = wl.h.get_kernel_timing()
    wl.h.set_kernel_timing(False)
    tot = sum(v[0] for v in kt.values()) or 1.0
    kernels = {k: {"launches": v[1], "avg_ms": (v[0] / v[1] if v[1] else None), "ms_per_step": v[0] / K, "share": v[0] / tot}
               for k, v in kt.items()}
    # per step, not per launch: a placement with many short sequences runs its last key tiles in a second launch
    bm = kernels["bwd_main"]["ms_per_step"] or None
    peak_t = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
    achieved = p.bwd_flops() / (bm * 1e-3) / 1e12 if bm else None
    pair = p.head_dim == 128 and args.bwd_kernel != 1   # the library's default at head_dim 128 is the CTA-pair kernel
    bwd_name = "zl_bwd_pair_kernel" if pair else "zl_bwd_main_kernel"
    traffic = NCU_BWD_DRAM_BYTES.get((args.config, bwd_name)) if not args.fuse_local_chunks else None
    roofline = {"kernel": bwd_name, "bound": "tensor", "achieved": achieved, "peak": peak_t,
                "unit": "TFLOP/s", "frac": (achieved / peak_t if achieved else None),
                "peak_kind": f"{peak_kind} sustained bf16 (kernel timed inside a long step)",
                "frac_of_burst": (achieved / float(peaks.get("bf16_tflops", 1590.0)) if achieved else None),
                "traffic": traffic,
                "traffic_note": ("DRAM bytes of one launch of this kernel on this configuration (ncu, one pass)" if traffic
                                 else "not captured for this configuration and kernel")}
    # The same kernel against shared-memory bandwidth (128 B/clk/SM), which is what actually binds the one-CTA
    # formulation: bytes through shared memory per (128-row query tile, 128-row key tile, head) -- MMA operand
    # reads, TMA tile writes, dS stores, dQ staging writes and the reduce engine's reads of them.
    d = p.head_dim
    b_mn = 16 * d * 2                                   # B operand of one K step when N = d
    per_pair = (2 * ((d // 16) * 8192 + 8192)           # S^T and dP^T: A + B per K step, plus the augmentation step
                + 8 * b_mn + 2 * 8 * (4096 + b_mn)      # dV (A from TMEM), dK, dQ
                + 2 * 128 * d * 2 + 4096                # TMA writes of Q, dO and the augmentation tile
                + 128 * 128 * 2                         # dS^T tile written by the P/dS warps
                + 2 * 128 * d * 4)                      # dQ staged in fp32 and read back by the reduce
    tasks_qk = [(l, l) for l in p.whole_lengths()] + [(s[1], s[3]) for s in p.shards]
    n_pairs = p.n_heads * sum(-(-q // 128) * -(-k // 128) for q, k in tasks_qk)
    n_sms = torch.cuda.get_device_properties(device).multi_processor_count
    sm_hz = float(clocks.get("sm_mhz") or 0.0) * 1e6
    if bm and sm_hz and not pair:
        b_clk = per_pair * n_pairs / (n_sms * bm * 1e-3 * sm_hz)
        roofline["smem"] = {"bytes_per_tile_pair": per_pair, "tile_pairs": n_pairs, "achieved": b_clk, "peak": 128.0,
                            "unit": "B/clk/SM", "frac": b_clk / 128.0,
                            "note": "shared-memory traffic of the same launches over the sampled median SM clock"}
    fm = kernels["fwd"]["ms_per_step"] or None
    fwd_kernel_tflops = p.fwd_flops() / (fm * 1e-3) / 1e12 if fm else None
    mm = kernels["merge"]["ms_per_step"] or None
    merge_gbs = wl.merge_bytes / (mm * 1e-3) / 1e9 if mm else None

    # end to end with host buffers
    wl.make_host_buffers()
    for _ in range(2):
        wl.e2e_step()
    ms_e2e_serial = wl.time_region(wl.e2e_step, K, dist) / K
    wl.e2e_pipelined(2, dist)
    ms_e2e = wl.e2e_pipelined(K, dist) / K
    e2e = {"value": aggregate_tflops(world, flops, ms_e2e), "unit": "TFLOP/s", "ms_per_step": ms_e2e,
           "how": "every step copies Q,K,V,dO from pinned host memory and O,LSE,dQ,dK,dV back; copies of "
                  "neighbouring steps overlap the compute (double-buffered, separate streams)",
           "serial_value": aggregate_tflops(world, flops, ms_e2e_serial), "serial_ms_per_step": ms_e2e_serial,
           "h2d_bytes_per_step": wl.h2d_bytes, "d2h_bytes_per_step": wl.d2h_bytes}
    code, where = wl.h.last_device_status()
    if code != 0:
        raise RuntimeError(f"device status {code} at {where}")

    result = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": p.name, "n_heads": p.n_heads, "head_dim": p.head_dim, "total_q": p.total_q,
                   "total_kv": p.total_kv, "tasks": int(wl.h.info.n_tasks),
                   "step": "fwd launch + lse merge + bwd (pre, main, post)",
                   "fuse_local_chunks": bool(args.fuse_local_chunks),
                   "l2": "inputs larger than L2 (K+V alone exceed 126 MB); no flush",
                   "parallelism": f"{world} independent rank-local placements"},
        "fwd_tflops": aggregate_tflops(world, p.fwd_flops(), ms_fwd / K),
        "fwd_ms": ms_fwd / K,
        # with activation checkpointing (the paper's training setting, Section V-A) a layer costs two forwards and one
        # backward; the forward is counted twice in both the time and the FLOPs
        "step_equivalent": {"what": "2 x fwd + bwd (recompute)", "ms": ms_step + ms_fwd / K,
                            "tflops": aggregate_tflops(world, 2 * p.fwd_flops() + p.bwd_flops(), ms_step + ms_fwd / K)},
        # the datasheet dense BF16 figure first: that is the peak the metric names (its 60 % mark is 1350 TFLOP/s)
        "frac_of_peak": {"datasheet_2250": value / world / 2250.0,
                         "measured_burst": value / world / float(peaks.get("bf16_tflops", 1590.0)),
                         "measured_sustained": value / world / peak_t},
        "build_tasks_ms": wl.build_ms,
        "gpu_launches": int(launches),
        "e2e": e2e, "roofline": roofline, "kernels": kernels,
        "fwd_kernel_tflops": fwd_kernel_tflops, "merge_gbs": merge_gbs,
        "merge_frac_of_hbm": (merge_gbs / float(peaks.get("hbm_gbs", 6650.0)) if merge_gbs else None),
        "clocks": clocks,
    }

    if world == 1 and args.context_flash_attn:
        result["context"] = flash_attn_context(device)
    if world == 1 and args.extra_configs:
        extra = {}
        del wl
        torch.cuda.empty_cache()
        for ci in [int(x) for x in args.extra_configs.split(",") if x]:
            try:
                pe = W.config(ci)
                we = Workload(pe, device, bwd_kernel=args.bwd_kernel)
                n = 3 if ci == 5 else 5
                for _ in range(3):
                    we.step()
                tf = we.time_region(we.fwd, n) / n
                tb = we.time_region(we.bwd, n) / n
                extra[pe.name] = {"fwd_ms": tf, "bwd_ms": tb, "fwd_tflops": pe.fwd_flops() / tf / 1e9,
                                  "bwd_tflops": pe.bwd_flops() / tb / 1e9,
                                  "fwd_bwd_tflops": (pe.fwd_flops() + pe.bwd_flops()) / (tf + tb) / 1e9}
                code, where = we.h.last_device_status()
                if code != 0:
                    extra[pe.name]["device_status"] = [code, where]
                del we
                torch.cuda.empty_cache()
            except Exception as e:  # noqa: BLE001
                extra[f"cfg{ci}"] = {"error": repr(e)}
        result["per_config"] = extra
        if not args.fuse_local_chunks and p.shards:
            # the same workload with ZL_BUILD_FUSE_LOCAL_CHUNKS (one final task per query range whose chunks are
            # contiguous: no partials, nothing to merge) -- reported beside the headline, never instead of it
            try:
                wf = Workload(p, device, flags=1)
                for _ in range(3):
                    wf.step()
                tf = wf.time_region(wf.fwd, 5) / 5
                ts = wf.time_region(wf.step, 5) / 5
                result["fused_local_chunks"] = {
                    "value": (p.fwd_flops() + p.bwd_flops()) / ts / 1e9, "unit": "TFLOP/s", "ms_per_step": ts,
                    "fwd_ms": tf, "fwd_tflops": p.fwd_flops() / tf / 1e9,
                    "fused_ranges": int(wf.h.info.n_fused_ranges), "tasks": int(wf.h.info.n_tasks),
                    "note": "optional schedule (bench.py --fuse-local-chunks); the headline value keeps the merge step"}
                del wf
                torch.cuda.empty_cache()
            except Exception as e:  # noqa: BLE001
                result["fused_local_chunks"] = {"error": repr(e)}

    if world == 1 and rank == 0 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(p)
    if rank == 0:
        print(json.dumps(result), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------
# reference arm: the fp64 CPU oracle on host cores
# --------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import zl_workloads as W
    p = W.config(args.config)
    K, Wm = args.steps, max(1, min(args.warmup, 2))
    per_step = max(1.0, min(8.0, 120.0 / (K + Wm)))
    for _ in range(Wm):
        cpu_baseline(p, target_s=per_step)
    vals, secs, last = [], 0.0, None
    for _ in range(K):
        last = cpu_baseline(p, target_s=per_step)
        vals.append(last["value"]); secs += last["seconds"]
    v = sum(vals) / len(vals)
    out = {"impl": "reference", "metric": METRIC, "value": v, "unit": "TFLOP/s",
           "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": K, "warmup": Wm,
           "ms_per_step": secs / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f64", "data": "synthetic",
           "config": {"workload": p.name, "n_heads": p.n_heads, "head_dim": p.head_dim,
                      "note": "each step is a bounded sample of the workload run by the fp64 CPU oracle"},
           "cpu_baseline": {"value": v, "unit": "TFLOP/s", "kind": "oracle", "cores": last["cores"],
                            "sample": last["sample"]},
           "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def run_ablation(args):
    """Extra measurements that evidence design choices (printed as one JSON line, not the headline):
    'straggler' -- config 3's images next to one WHOLE 32,760-token video (the naive data-parallel
    placement): forward time with the work list longest-first, in placement order and shortest-first;
    'coalescing' -- config 2 as one coalesced launch vs one launch per sequence."""
    import torch
    import zl_workloads as W
    import paper_2608_01150_b200 as Z
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    out = {"ablation": args.ablation}
    if args.ablation == "straggler":
        p = W.straggler_placement()
        wl = Workload(p, device)
        for name, mode in (("longest_first", 0), ("placement_order", 1), ("shortest_first", 2)):
            wl.h.set_fwd_order(mode)
            for _ in range(3):
                wl.fwd()
            ms = wl.time_region(wl.fwd, 10) / 10
            out[name] = {"fwd_ms": ms, "fwd_tflops": p.fwd_flops() / ms / 1e9}
        wl.h.set_fwd_order(0)
    else:
        p = W.config(2)
        wl = Workload(p, device)
        for _ in range(3):
            wl.fwd()
        ms = wl.time_region(wl.fwd, 10) / 10
        out["coalesced"] = {"launches": 1, "fwd_ms": ms, "fwd_tflops": p.fwd_flops() / ms / 1e9}
        # the same sequences, one launch each (handles built beforehand)
        H, d = p.n_heads, p.head_dim
        hs = []
        for i in range(p.n_whole):
            a, b = p.cu_seqlens[i], p.cu_seqlens[i + 1]
            hs.append((a, b, Z.build_tasks([0, b - a], [], b - a, b - a, H, d)))

        def per_sequence():
            for a, b, h in hs:
                Z.coalesced_attn_fwd(h, wl.Q[a:b], wl.K[a:b], wl.V[a:b], p.scale, wl.O[a:b], wl.LSE, None, None)
        # LSE is [H, total_q]: a per-sequence handle writes rows [0, len) of each head's line; only timing matters here
        for _ in range(3):
            per_sequence()
        ms = wl.time_region(per_sequence, 10) / 10
        out["per_sequence"] = {"launches": len(hs), "fwd_ms": ms, "fwd_tflops": p.fwd_flops() / ms / 1e9}
    print(json.dumps(out), flush=True)


def run_cp(args):
    """Context-parallel mode (not the headline): all N ranks share one 75,600-token video under N-way all-gather
    context parallelism (Table II, configuration (q,1,1)) and each also runs six whole 1560-token images; one
    layer forward + backward through the executor (K/V all-gather into local buffers -> one coalesced launch +
    merge -> backward -> dK/dV reduce-scatter).  value = counted FLOPs of the whole job / slowest rank's time."""
    import torch
    import torch.distributed as dist
    from paper_2608_01150_b200 import executor as E
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    else:
        dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{29500 + os.getpid() % 2000}", rank=0, world_size=1)
    H, d, L = 40, 128, 75600
    segs = [E.Segment(0, L, (world, 1, 1), tuple(range(world)))] if world > 1 else [E.Segment(0, L // 8, (1, 1, 1), (0,))]
    sid = 1
    for r in range(world):
        for _ in range(6):
            segs.append(E.Segment(sid, 1560, (1, 1, 1), (r,)))
            sid += 1
    ex = E.CPExecutor(segs, H, d)
    eng = E.EngineAttention(d, sm_margin=(8 if world > 1 else 0))   # NCCL's kernels need SMs beside a launch phase
    T = ex.schedule.own_tokens
    g = torch.Generator(device=device); g.manual_seed(7 + rank)
    q, k, v, do = (torch.randn((T, H, d), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16) for _ in range(4))

    def timed(fwd_step, bwd_step):
        def step():
            ex.forward(q, k, v, fwd_step)
            ex.backward(do, bwd_step)
        for _ in range(max(3, args.warmup)):
            step()
        torch.cuda.synchronize(); dist.barrier(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record(); torch.cuda.synchronize()
        return reduce_max_ms(e0.elapsed_time(e1), dist, device) / args.steps

    # launch phases under the collectives (the engine object itself), then one launch after all collectives
    ms = timed(eng, eng)
    ms_single = timed(eng.fwd, eng.bwd)
    video_len = L if world > 1 else L // 8
    pairs = video_len * video_len + world * 6 * 1560 * 1560
    flops = 3.5 * 4.0 * pairs * d * H
    if rank == 0:
        print(json.dumps({"mode": "cp", "metric": METRIC, "value": flops / (ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                          "n_gpus": world, "steps": args.steps, "ms_per_step": ms, "scaling": "strong (video) + weak (images)",
                          "overlap": {"how": "tasks with local K/V launched first, collectives on a second stream, the rest released on "
                                             "arrival; gradients of remote chunks reduce-scattered under the second backward phase",
                                      "fwd_phases": ex.schedule.n_fwd_phases, "bwd_phases": ex.schedule.n_bwd_phases,
                                      "ms_per_step_one_launch_after_collectives": ms_single,
                                      "value_one_launch_after_collectives": flops / (ms_single * 1e-3) / 1e12},
                          "config": {"workload": f"one {video_len}-token video under {world}-way all-gather CP + 6 images per rank",
                                     "n_heads": H, "head_dim": d, "collectives": [list(map(str, e)) for e in ex.log]}}), flush=True)
    dist.barrier()
    dist.destroy_process_group()


def run_profile(args):
    """Hardware-profiler record (paper Section IV-B / V-B): the price table of the paper's catalog on this GPU, the
    catalog cut it implies, and the additive model checked on the covering plans; one JSON line."""
    import torch
    from paper_2608_01150_b200 import profiler
    torch.cuda.set_device(0)
    rep = profiler.catalog_report(args.profile_heads, 128, steps=3)
    rep = {"mode": "profile", **rep}
    print(json.dumps(rep), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4, help="named configuration 1..5 (default: Wan-14B-shaped rank)")
    ap.add_argument("--extra-configs", default="2,3,5", help="also time these configurations (N=1 only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fuse-local-chunks", action="store_true",
                    help="build the handle with ZL_BUILD_FUSE_LOCAL_CHUNKS: query ranges whose chunks are contiguous run "
                         "as one final task (no partials, nothing to merge); off by default")
    ap.add_argument("--profile", action="store_true",
                    help="print the hardware profiler's record (price table of the paper's catalog, catalog cut, additivity) "
                         "instead of the benchmark line")
    ap.add_argument("--profile-heads", type=int, default=12)
    ap.add_argument("--cp", action="store_true",
                    help="context-parallel mode: one video under N-way all-gather CP across the N ranks + images per rank, "
                         "through the executor (printed as its own JSON line, not the headline)")
    ap.add_argument("--context-flash-attn", action="store_true",
                    help="also time the image's flash_attn package on configuration 2 (context line, N=1)")
    ap.add_argument("--bwd-kernel", type=int, default=0, choices=[0, 1, 2],
                    help="backward main kernel: 0 library default, 1 one CTA per key tile, 2 CTA pairs")
    ap.add_argument("--ablation", default="", choices=["", "straggler", "coalescing"],
                    help="print an extra measurement instead of the benchmark line")
    args = ap.parse_args()

    if args.ablation:
        run_ablation(args)
        return
    if args.profile:
        run_profile(args)
        return

    if args.impl == "reference":
        run_reference(args)
        return
    if args.cp and (args.gpus == 1 or "WORLD_SIZE" in os.environ):
        run_cp(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        port = 29500 + (os.getpid() % 2000)
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if args.cp:
        run_cp(args)
        return
    run_ours(args)


if __name__ == "__main__":
    main()
