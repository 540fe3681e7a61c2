"""The benchmark's multi-GPU arm runs independent replicas (the SpMM path has no exchange
step) and reports total work over the slowest rank's time.  This checks that aggregation
with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 2.0 + rank                       # rank 1 is the slow one: 3 ms
    ms, value = bench.aggregate_over_ranks(ms_local, 6.0e9, world, dist, "cpu")
    out.put((rank, ms, value))
    dist.destroy_process_group()


def test_two_rank_replica_aggregation():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, ms, value in results:
        assert ms == 3.0                                       # max over ranks
        assert abs(value - 2 * 6.0e9 / 3.0e-3 / 1e9) < 1e-6    # both replicas' work over that time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    ms, value = bench.aggregate_over_ranks(0.5, 1.0e9, 1)
    assert ms == 0.5 and abs(value - 2000.0) < 1e-9
