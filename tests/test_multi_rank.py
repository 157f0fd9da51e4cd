"""The N > 1 path of bench.py ("replicas only": no data-path collective, max-over-ranks timing) on two gloo ranks."""
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
    try:
        # rank r "measured" (10 + 5 r) ms for its own replica of 1000 frames
        local_ms = 10.0 + 5.0 * rank
        slowest = bench.max_over_ranks(local_ms, world, "cpu")
        value = bench.whole_job_frames_per_sec(1000.0, world, slowest * 1e-3)
        dist.barrier()
        out[rank] = (slowest, value)
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_summed_frames():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in range(world):
        slowest, value = res[rank]
        assert slowest == 15.0  # every rank sees the max
        assert abs(value - 2 * 1000.0 / 15e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.whole_job_frames_per_sec(100.0, 1, 0.5) == 200.0
