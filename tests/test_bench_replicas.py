"""The multi-GPU arm of bench.py runs independent replicas (the path has no exchange step); only its
timing reduction talks across ranks.  This covers that reduction with two gloo ranks on the CPU."""
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
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))     # rank 1 is the slower replica
    total = bench.whole_job(1.0e12, world, ms)
    out.put((rank, ms, total))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_weak_scaling_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, total in res:
        assert ms == 15.0                                  # the max over ranks, on every rank
        assert abs(total - 2 * 1.0e12 / 15.0e-3) < 1.0     # both replicas' units over the slower time


def test_single_process_path_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, torch.device("cpu")) == 3.5
    assert bench.whole_job(2.0, 1, 1000.0) == 2.0
