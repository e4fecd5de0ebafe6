"""Hardware profiler for the coalesced attention engine (paper Section IV-B).

The planner of the paper works with an additive price table: the per-rank time ``P[b, theta]`` of one
sequence of catalog bucket ``b`` run under parallelism configuration ``theta``, measured once per
setup "after removing a placement-independent step cost"; a rank's load is then the sum of the
prices of the segments placed on it (Eq. for the makespan, Section IV-B), and Section V-B reports how
well that additive model predicts measured steps (3.4 % MAPE on the paper's testbed).

This module measures that table on the engine of this repository and checks the additive model
against mixed placements, for the attention part of a step (forward launch, LSE merge, backward).
On one GPU a configuration is a context-parallel degree k: the rank owns one query chunk of
``L / k`` tokens and attends to all k key/value chunks, which are local inputs (what the all-gather
variant of Table II leaves on the rank).  It uses the public binding only.

    python -m paper_2608_01150_b200.profiler --out prices.json

Everything here is measurement glue: the arithmetic of the method stays in the kernels.
"""
from __future__ import annotations

import argparse
import json
import sys
from dataclasses import dataclass
from typing import Callable, Dict, List, Optional, Sequence, Tuple

# Wan latent token counts (21 latent frames; 480p and 720p frames of 1,560 and 3,600 tokens) and one image
BUCKETS: Dict[str, int] = {"image_480p": 1560, "video_480p": 32760, "video_720p": 75600}
DEGREES: Tuple[int, ...] = (1, 2, 4, 8)

# The catalog of the paper's evaluation (Section V-A: 256p-1080p images, 480p-1080p videos of 5, 10 and 15
# seconds): tokens per latent frame x latent frames.  A 1080p frame is 8,160 tokens and a 15-second clip has 61
# latent frames, which gives the 497,760-token sequence of the paper's introduction; 10 s = 41 frames, 5 s = 21.
FRAME_TOKENS = {"256p": 256, "480p": 1560, "720p": 3600, "1080p": 8160}
LATENT_FRAMES = {"5s": 21, "10s": 41, "15s": 61}
CATALOG: Dict[str, int] = {f"image_{r}": t for r, t in FRAME_TOKENS.items()}
CATALOG.update({f"video_{r}_{d}": FRAME_TOKENS[r] * n for r in ("480p", "720p", "1080p") for d, n in LATENT_FRAMES.items()})
CATALOG_DEGREES: Tuple[int, ...] = (1, 2, 4, 8, 16)
# a (bucket, degree) pair is profiled when the rank's share is at most this many score pairs per head
# (a whole 15-second 1080p video on one rank is 2.5e11 pairs: seconds per step, and no planner would place it so)
MAX_PAIRS_PER_HEAD = 3.2e10
# small buckets are priced from a batch with at least this many query rows (a few waves of 256-row work items on
# 148 SMs at 12 heads)
FILL_ROWS = 16384


@dataclass(frozen=True)
class Segment:
    """One sequence of `tokens` tokens run at context-parallel degree `degree` on this rank."""
    bucket: str
    tokens: int
    degree: int

    def chunk(self) -> int:
        return -(-self.tokens // self.degree)


def placement_of(segments: Sequence[Segment]):
    """cu_seqlens, shard descriptors and row totals of the rank-local placement of `segments`:
    degree-1 segments are whole sequences, the others one query chunk against `degree` K/V chunks."""
    cu = [0]
    for s in segments:
        if s.degree == 1:
            cu.append(cu[-1] + s.tokens)
    q_pos = kv_pos = cu[-1]
    shards = []
    sid = 0
    for s in segments:
        if s.degree == 1:
            continue
        c = s.chunk()
        for k in range(s.degree):
            shards.append((q_pos, c, kv_pos + k * c, c, sid))
        q_pos += c
        kv_pos += s.degree * c
        sid += 1
    return cu, shards, q_pos, kv_pos


def predict_ms(prices: Dict[str, float], step_cost_ms: float, segments: Sequence[Segment]) -> float:
    """The additive model: the placement-independent cost plus the sum of the segments' prices."""
    return step_cost_ms + sum(prices[f"{s.bucket}@{s.degree}"] for s in segments)


def mape(pairs: Sequence[Tuple[float, float]]) -> float:
    """Mean absolute percentage error of (predicted, measured) pairs, in percent."""
    return 100.0 * sum(abs(p - m) / m for p, m in pairs) / max(1, len(pairs))


def gpu_timer(n_heads: int, head_dim: int, steps: int = 5, warmup: int = 2) -> Callable[[Sequence[Segment]], float]:
    """Returns measure(segments) -> milliseconds per step (forward launch + merge + backward) on cuda:0,
    timed with CUDA events after warm-up, synthetic N(0,1) bf16 inputs."""
    import torch
    from . import binding as Z

    def measure(segments: Sequence[Segment]) -> float:
        cu, shards, tq, tkv = placement_of(segments)
        h = Z.build_tasks(cu, shards, tq, tkv, n_heads, head_dim)
        dev = torch.device("cuda", 0)
        mk = lambda rows, seed: torch.randn((rows, n_heads, head_dim), device=dev, dtype=torch.float32,
                                            generator=torch.Generator(device=dev).manual_seed(seed)).to(torch.bfloat16)
        q, k, v, d_o = mk(tq, 1), mk(tkv, 2), mk(tkv, 3), mk(tq, 4)
        o = torch.empty_like(q)
        lse = torch.empty((n_heads, tq), device=dev, dtype=torch.float32)
        pr = max(1, int(h.info.partial_rows))
        op = torch.empty((pr, n_heads, head_dim), device=dev, dtype=torch.float32)
        lp = torch.empty((n_heads, pr), device=dev, dtype=torch.float32)
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        ws = torch.empty(max(256, int(h.info.bwd_workspace_bytes)), device=dev, dtype=torch.uint8)
        scale = head_dim ** -0.5

        def step():
            Z.coalesced_attn_fwd(h, q, k, v, scale, o, lse, op, lp)
            Z.lse_merge(h, op, lp, o, lse)
            Z.coalesced_attn_bwd(h, q, k, v, o, lse, d_o, scale, dq, dk, dv, ws)

        for _ in range(warmup):
            step()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            step()
        b.record()
        torch.cuda.synchronize()
        code, where = h.last_device_status()
        if code != 0:
            raise RuntimeError(f"device status {code} at {where}")
        return a.elapsed_time(b) / steps

    return measure


def profile_prices(measure: Callable[[Sequence[Segment]], float], buckets: Dict[str, int] = BUCKETS,
                   degrees: Sequence[int] = DEGREES, max_pairs: float = float("inf"),
                   fill_rows: int = 0) -> Tuple[Dict[str, float], float]:
    """Measures every bucket x degree.  The placement-independent step cost is the time of a step over one
    128-token sequence (five launches that do next to nothing); it is removed from every price.  Pairs whose
    chunks would be shorter than one tile, or whose rank share exceeds `max_pairs` score pairs per head, are
    not profiled.  A bucket too small to fill the GPU on its own is measured as a batch of identical sequences
    with at least `fill_rows` query rows in total and priced per sequence: one image alone leaves most SMs
    idle, which is not what it costs inside a batch (the paper's measurements include packing)."""
    step_cost = measure([Segment("floor", 128, 1)])
    prices = {}
    for name, tokens in buckets.items():
        for k in degrees:
            if tokens // k < 128 or (tokens / k) * tokens > max_pairs:
                continue
            seg = Segment(name, tokens, k)
            n = max(1, -(-fill_rows // seg.chunk())) if fill_rows else 1
            # a sequence that costs no more than the placement-independent floor gets the timer's resolution
            # (1 us): prices enter the catalog cut through their logarithm
            prices[f"{name}@{k}"] = max(1e-3, (measure([seg] * n) - step_cost) / n)
    return prices, step_cost


def whole_prices(prices: Dict[str, float], buckets: Dict[str, int]) -> Dict[str, float]:
    """Price of every bucket run as ONE sequence on one rank, the quantity the catalog cut (Eq. 3) orders the
    buckets by: the degree-1 price where it was measured, else k times the price of the smallest profiled
    degree k (the k chunks of a sequence cost the same on every rank, and together they are the sequence)."""
    out = {}
    for name in buckets:
        ks = sorted(int(key.split("@")[1]) for key in prices if key.split("@")[0] == name)
        if ks:
            out[name] = ks[0] * prices[f"{name}@{ks[0]}"]
    return out


def covering_plans(prices: Dict[str, float], buckets: Dict[str, int], n_images: int = 50,
                   image: str = "image_480p", duration: str = "5s") -> List[List[Segment]]:
    """Mixed plans in the manner of Section V-B: every plan holds one 480p, one 720p and one 1080p video of
    `duration` plus a fixed set of images, and the profiled degrees rotate over the resolutions so that every
    (resolution, degree) pair that was profiled occurs; then the all-whole corner plans (images only; three
    480p videos + images; three 720p videos + images)."""
    videos = [f"video_{r}_{duration}" for r in ("480p", "720p", "1080p") if f"video_{r}_{duration}" in buckets]
    img = [Segment(image, buckets[image], 1)] * n_images
    degs = {v: sorted(int(k.split("@")[1]) for k in prices if k.split("@")[0] == v) for v in videos}
    n = max(len(d) for d in degs.values())
    plans = []
    for r in range(n):
        plan = [Segment(v, buckets[v], degs[v][(r + i) % len(degs[v])]) for i, v in enumerate(videos)]
        plans.append(plan + img)
    plans.append(list(img))
    for v in videos[:2]:
        if 1 in degs[v]:
            plans.append([Segment(v, buckets[v], 1)] * 3 + img)
    return plans


def rotation_plans(buckets: Dict[str, int] = BUCKETS, degrees: Sequence[int] = DEGREES,
                   n_images: int = 16) -> List[List[Segment]]:
    """Mixed plans in the manner of Section V-B: every plan holds one sequence of each video bucket plus a
    fixed set of images, and the degrees rotate over the buckets so that each (bucket, degree) pair
    occurs; then all-whole corner plans."""
    videos = [n for n in buckets if not n.startswith("image")]
    images = [n for n in buckets if n.startswith("image")]
    img = [Segment(images[0], buckets[images[0]], 1)] * n_images if images else []
    plans = []
    for r in range(len(degrees)):
        plan = [Segment(v, buckets[v], degrees[(r + i) % len(degrees)]) for i, v in enumerate(videos)]
        plans.append(plan + img)
    plans.append(list(img))
    for v in videos[:1]:
        plans.append([Segment(v, buckets[v], 1)] * 2 + img)
    return [p for p in plans if p]


def check_additivity(measure, prices, step_cost, plans) -> Dict:
    rows = []
    for plan in plans:
        pred, meas = predict_ms(prices, step_cost, plan), measure(plan)
        rows.append({"plan": [f"{s.bucket}@{s.degree}" for s in plan], "predicted_ms": pred, "measured_ms": meas,
                     "error_pct": 100.0 * (pred - meas) / meas})
    return {"plans": rows, "mape_pct": mape([(r["predicted_ms"], r["measured_ms"]) for r in rows]),
            "mae_ms": sum(abs(r["predicted_ms"] - r["measured_ms"]) for r in rows) / max(1, len(rows))}


def catalog_report(n_heads: int, head_dim: int, steps: int = 3, n_images: int = 50, duration: str = "5s") -> Dict:
    """Profiles the paper's catalog on cuda:0 and checks the additive model on the covering plans; also applies
    the catalog cut (Eq. 3) to the whole-sequence prices.  Returns a JSON-ready dict."""
    from . import planner
    measure = gpu_timer(n_heads, head_dim, steps=steps, warmup=1)
    prices, step_cost = profile_prices(measure, CATALOG, CATALOG_DEGREES, MAX_PAIRS_PER_HEAD, fill_rows=FILL_ROWS)
    whole = whole_prices(prices, CATALOG)
    fillers, anchors = planner.split_catalog(whole)
    plans = covering_plans(prices, CATALOG, n_images=n_images, duration=duration)
    return {"n_heads": n_heads, "head_dim": head_dim, "step_cost_ms": step_cost, "prices_ms": prices,
            "whole_prices_ms": whole, "catalog_cut": {"fillers": fillers, "anchors": anchors},
            "additivity": check_additivity(measure, prices, step_cost, plans)}


def main(argv: Optional[Sequence[str]] = None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--heads", type=int, default=12)
    ap.add_argument("--head-dim", type=int, default=128)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--images", type=int, default=16)
    ap.add_argument("--catalog", action="store_true",
                    help="profile the paper's catalog (256p-1080p images, 480p-1080p videos of 5/10/15 s, degrees 1-16) "
                         "and check the additive model on the covering plans of its Section V-B")
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    if args.catalog:
        report = catalog_report(args.heads, args.head_dim, steps=min(args.steps, 3), n_images=max(args.images, 50))
        text = json.dumps(report, indent=1)
        if args.out:
            with open(args.out, "w") as f:
                f.write(text)
        print(text)
        return 0
    measure = gpu_timer(args.heads, args.head_dim, steps=args.steps)
    prices, step_cost = profile_prices(measure)
    report = {"n_heads": args.heads, "head_dim": args.head_dim, "step_cost_ms": step_cost, "prices_ms": prices,
              "additivity": check_additivity(measure, prices, step_cost, rotation_plans(n_images=args.images))}
    text = json.dumps(report, indent=1)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)
    print(text)
    return 0


if __name__ == "__main__":
    sys.exit(main())
