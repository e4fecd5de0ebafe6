"""N > 1 host logic on CPU: two gloo ranks build their rank-local schedules independently (the
path has no data-path collective) and the benchmark's timing reduction takes the slowest rank."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import zl_workloads as W
    import paper_2608_01150_b200 as Z

    p = W.config(3)
    h = Z.build_tasks(p.cu_seqlens, p.shards, p.total_q, p.total_kv, p.n_heads, p.head_dim)
    # every rank lowers the same-shaped placement to the same schedule, without talking to anyone
    items = torch.tensor(h.fwd_items()[:64], dtype=torch.int64).flatten()
    gathered = [torch.zeros_like(items) for _ in range(world)]
    dist.all_gather(gathered, items)
    assert all(torch.equal(g, items) for g in gathered)
    # slowest rank decides the step time; throughput is the sum over ranks
    local_ms = 10.0 + 5.0 * rank
    ms = bench.reduce_max_ms(local_ms, dist, torch.device("cpu"))
    assert ms == 10.0 + 5.0 * (world - 1)
    flops = p.fwd_flops() + p.bwd_flops()
    v = bench.aggregate_tflops(world, flops, ms)
    assert abs(v - world * flops / (ms * 1e-3) / 1e12) < 1e-9
    dist.barrier()
    with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
        f.write(f"{ms} {v}")
    dist.destroy_process_group()


def test_two_gloo_ranks(tmp_path):
    from paper_2608_01150_b200 import build
    build.build()
    port = 29600 + os.getpid() % 300
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    vals = [open(tmp_path / f"ok{r}").read() for r in range(2)]
    assert vals[0] == vals[1]
