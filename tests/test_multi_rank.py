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


def _grad_worker(rank, world, port, out):
    """Rank r takes envs [r*B/2, (r+1)*B/2) of one recorded batch, computes the checker's gradient on its shard and
    sums it with the exchange function the replicated driver uses."""
    sys.path.insert(0, ROOT)
    import numpy as np

    from oracle import binding as orc
    from paper_2104_06272_b200 import replicas

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, N, H, T, seed = 8, 5, 32, 6, 5
        walls, start, goal = orc.env_init(seed, B, N)
        theta = orc.param_init(seed, N, H)
        pos, tep = start.copy(), np.zeros(B, np.uint8)
        tr = orc.rollout(N, H, 0, T, 50, theta, walls, start, goal, pos, tep, seed, 0)
        adv, ret = orc.gae(0.99, 0.95, tr.reward, tr.value, tr.done)
        full, _ = orc.learn(N, H, 0, theta, walls, goal, tr.pos, tr.action, adv, ret)
        off, bl = replicas.shard_of(B, rank, world)
        sl = slice(off, off + bl)
        mine, _ = orc.learn(N, H, 0, theta, walls[sl], goal[sl], np.ascontiguousarray(tr.pos[:, sl]),
                            np.ascontiguousarray(tr.action[:, sl]), np.ascontiguousarray(adv[:, sl]), np.ascontiguousarray(ret[:, sl]))
        g = torch.from_numpy(mine.copy())
        n = replicas.sum_over_replicas_(g)
        assert n == world
        out[rank] = (g.numpy().copy() / np.float32(n), full, mine)  # the library divides inside its Adam kernel
    finally:
        dist.destroy_process_group()


def test_gradient_mean_over_two_replicas_equals_the_full_batch_gradient():
    import numpy as np

    world = 2
    port = 31500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_grad_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    g0, full, mine0 = res[0]
    g1, _, mine1 = res[1]
    assert np.array_equal(g0, g1)  # every replica applies the same gradient
    assert not np.allclose(mine0, mine1)  # the shards really differ
    scale = np.abs(full).max()
    assert np.abs(g0 - full).max() <= 2e-6 * scale  # mean of the two shard means = full-batch mean (fp32 rounding)


def test_shards_partition_the_batch():
    sys.path.insert(0, ROOT)
    import pytest

    from paper_2104_06272_b200 import replicas

    assert [replicas.shard_of(12, r, 4) for r in range(4)] == [(0, 3), (3, 3), (6, 3), (9, 3)]
    with pytest.raises(ValueError):
        replicas.shard_of(10, 0, 4)
