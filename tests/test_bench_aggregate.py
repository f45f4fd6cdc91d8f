"""Whole-job aggregation of the benchmark over ranks (replicas): tokens add up, time is the slowest
rank's.  Two gloo ranks on CPU."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    tokens, seconds = bench.aggregate(100.0 * (rank + 1), 2.0 + rank, dist)
    out.put((rank, tokens, seconds))
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_sums_tokens_and_takes_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29731, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, 300.0, 3.0), (1, 300.0, 3.0)]


def test_aggregate_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(5.0, 2.0, None) == (5.0, 2.0)
