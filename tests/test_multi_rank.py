"""The N > 1 benchmark path on CPU: two gloo ranks, each with its own seeded workload, no
data-path exchange, timing reduced with MAX over ranks (the aggregation bench.py uses)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from hx_synth import make_workload
    wl = make_workload("sweep", seed=bench.rank_seed(rank), scale=1 / 256)
    total_ms, e2e_s = bench.reduce_times(dist, 10.0 * (rank + 1), 0.5 * (rank + 1), device="cpu")
    digest = float(wl.calls["prompt_tokens"].sum())
    gathered = [None] * world
    dist.all_gather_object(gathered, digest)
    if rank == 0:
        out.put((total_ms, e2e_s, gathered, bench.job_value(world, 1000, total_ms / 5)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_by_seed_and_reduce_with_max():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    total_ms, e2e_s, digests, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert total_ms == 20.0 and e2e_s == 1.0              # the slowest rank decides
    assert digests[0] != digests[1]                       # each rank schedules its own workload
    assert value == pytest.approx(2 * 1000 / (20.0 / 5 * 1e-3))
