"""The N > 1 path of bench.py is "replicas only": every rank decodes its own sequence, the
only exchanges are a barrier and a MAX over the ranks' times.  Two gloo ranks on the CPU
exercise exactly that arithmetic (no GPU, no data-path collective exists to test)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    my_ms = 100.0 + 50.0 * rank          # rank 1 is the slow replica
    dist.barrier()
    worst = bench.max_over_ranks(my_ms, dist, "cpu")
    value = bench.job_tokens_per_s(world, steps=2, new_tokens=256, total_ms=worst)
    out[rank] = (worst, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_are_timed_by_the_slowest_and_counted_twice():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    worst, value = res[0]
    assert worst == 150.0
    assert abs(value - 2 * 2 * 256 / 0.150) < 1e-6


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(12.5, None, "cpu") == 12.5
    assert bench.job_tokens_per_s(1, 5, 256, 1000.0) == 1280.0
