"""The N > 1 path of the benchmark on CPU: replicas only, no data-path collective.  Two gloo
ranks check the max-over-ranks timing, the aggregate throughput and that replicas draw
different images."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    import bench
    import vitgen
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow replica
    ms = bench.max_over_ranks(local_ms, dist)
    value = bench.aggregate_images_per_s(world, 128, ms)
    shape = vitgen.preset("tiny16")
    pix = vitgen.make_pixels(shape, 1, seed=bench.rank_pixel_seed(rank))
    digest = torch.tensor([float(np.abs(pix).sum())], dtype=torch.float64)
    both = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(both, digest)                     # test-side check only, not the data path
    q.put((rank, ms, value, [float(b.item()) for b in both]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_slowest_time_and_aggregate_throughput():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value, digests in res:
        assert ms == 15.0                             # the max over ranks, on every rank
        assert abs(value - 2 * 128 / 0.015) < 1e-6
        assert digests[0] != digests[1]               # replicas process different images


def test_single_process_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(7.5) == 7.5
    assert bench.aggregate_images_per_s(1, 64, 8.0) == 8000.0
