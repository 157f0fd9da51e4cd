"""Replicated Anakin on one GPU: G handles with B/G envs each and env offsets 0, B/G, ... are run one after the other
(no kernel waits on another) and must hold exactly the envs of one B-env handle; the mean of their gradients must be
the full-batch gradient; and the split update (gradient, then Adam) must equal the fused one."""
import numpy as np
import pytest
import torch

from paper_2104_06272_b200.workloads import WORKLOADS

pytestmark = pytest.mark.gpu

CASES = {
    "mma_h64": WORKLOADS["tiny"].scaled(name="mma_h64", B=256, T=16),
    "ffma_h96": WORKLOADS["tiny"].scaled(name="ffma_h96", B=192, H=96, T=8),
    "wide_bf16": WORKLOADS["tensor_core"].scaled(name="wide_bf16", B=256, H=512, T=4),
    # the kernels the large workloads run: the warp-level tensor rollout at H = 128 and the CTA-pair tcgen05 rollout at
    # H = 256, each with a shard boundary (env_offset) that is not a multiple of its envs per CTA
    "mma_h128": WORKLOADS["memory_bound"].scaled(name="mma_h128", B=2 * 176, T=12),
    "pair_h256": WORKLOADS["throughput"].scaled(name="pair_h256", B=2 * 208, T=10),
}


@pytest.fixture(scope="module")
def bnd():
    from paper_2104_06272_b200 import binding

    return binding


def make(bnd, w, env_offset=0):
    return bnd.Anakin(bnd.cfg_from_workload(w, debug_logits=0, env_offset=env_offset))


@pytest.mark.parametrize("name", list(CASES))
def test_split_update_equals_the_fused_update_bitwise(bnd, name):
    w = CASES[name]
    a, b = make(bnd, w), make(bnd, w)
    for an in (a, b):
        an.reset(3)
        an.rollout()
    a.learn()
    b.grads()
    assert np.array_equal(b.get(bnd.PARAMS), bnd_params_after_reset(bnd, w, 3))  # grads() leaves the parameters alone
    assert int(b.get(bnd.ADAM_STEP)) == 0
    b.apply_grads()
    for which in (bnd.GRADS, bnd.PARAMS, bnd.ADAM_M, bnd.ADAM_V):
        assert np.array_equal(a.get(which), b.get(which)), which
    assert int(b.get(bnd.ADAM_STEP)) == 1
    # and the next iteration starts from the same state on both
    a.run(1)
    b.rollout()
    b.grads()
    b.apply_grads()
    assert np.array_equal(a.get(bnd.PARAMS), b.get(bnd.PARAMS))
    assert a.status() == 0 and b.status() == 0


def bnd_params_after_reset(bnd, w, seed):
    an = make(bnd, w)
    an.reset(seed)
    return an.get(bnd.PARAMS)


@pytest.mark.parametrize("name", list(CASES))
def test_two_shards_hold_the_envs_of_one_handle_and_their_mean_gradient_is_the_full_one(bnd, name):
    w = CASES[name]
    G = 2
    full = make(bnd, w)
    shards = [make(bnd, w.scaled(B=w.B // G), env_offset=r * (w.B // G)) for r in range(G)]
    for an in [full] + shards:
        an.reset(7)
        an.rollout()
    bl = w.B // G
    for r, sh in enumerate(shards):
        sl = slice(r * bl, (r + 1) * bl)
        assert np.array_equal(sh.get(bnd.PARAMS), full.get(bnd.PARAMS))  # parameters depend on the seed alone
        for which in (bnd.ENV_WALLS, bnd.ENV_START, bnd.ENV_GOAL, bnd.ENV_POS, bnd.ENV_TEP):
            got, want = sh.get(which), full.get(which)
            assert np.array_equal(got.reshape(bl, -1), want.reshape(w.B, -1)[sl]), which
        for which in (bnd.TRAJ_POS, bnd.TRAJ_ACTION, bnd.TRAJ_DONE, bnd.TRAJ_REWARD, bnd.TRAJ_LOGP):
            got, want = sh.get(which), full.get(which)
            assert np.array_equal(got.reshape(w.T, bl), want.reshape(w.T, w.B)[:, sl]), which
        assert np.array_equal(sh.get(bnd.TRAJ_VALUE).reshape(w.T + 1, bl), full.get(bnd.TRAJ_VALUE).reshape(w.T + 1, w.B)[:, sl])
    full.grads()
    for sh in shards:
        sh.grads()
    gfull = full.get(bnd.GRADS).astype(np.float64)
    gmean = np.mean([sh.get(bnd.GRADS).astype(np.float64) for sh in shards], axis=0)
    rtol = 1e-5 if w.precision == 0 else 2e-3  # summation order only (bf16 workload: plus the split of the bf16-rounded sums)
    rms = np.sqrt((gfull**2).mean())
    assert (np.abs(gmean - gfull) <= rtol * (np.abs(gfull) + rms)).all()
    # the exchange: every shard receives the SUM (what the all-reduce leaves), the Adam kernel divides by the number of
    # replicas, and the replicas stay identical
    total = torch.from_numpy(shards[0].get(bnd.GRADS)).cuda() + torch.from_numpy(shards[1].get(bnd.GRADS)).cuda()
    for sh in shards:
        sh.set(bnd.GRADS, total)
        sh.apply_grads(G)
        assert np.array_equal(sh.get(bnd.GRADS), (total / G).cpu().numpy())  # GRADS now reads as the mean
    assert np.array_equal(shards[0].get(bnd.PARAMS), shards[1].get(bnd.PARAMS))
    full.apply_grads()
    p_full, p_sh = full.get(bnd.PARAMS).astype(np.float64), shards[0].get(bnd.PARAMS).astype(np.float64)
    # a first Adam step is +-lr for any gradient well above eps, so the parameters agree far better than the gradients
    assert np.abs(p_full - p_sh).max() <= 1.01 * w.lr
    assert np.mean(np.abs(p_full - p_sh) > 1e-6) < 1e-2
    for an in [full] + shards:
        assert an.status() == 0


def test_replicated_driver_with_one_rank_matches_run(bnd):
    """ReplicatedAnakin with world = 1 (no process group) walks the same states as anakin_run."""
    from paper_2104_06272_b200 import replicas

    w = CASES["mma_h64"]
    a = make(bnd, w)
    a.reset(11)
    a.run(3)
    r = replicas.ReplicatedAnakin(w, rank=0, world=1)
    r.reset(11)
    r.run(3)
    assert np.array_equal(a.get(bnd.PARAMS), r.an.get(bnd.PARAMS))
    assert np.array_equal(a.get(bnd.ENV_POS), r.an.get(bnd.ENV_POS))


def test_exchange_through_nccl_in_a_group_of_one(bnd):
    """The copy / all-reduce / copy / Adam sequence on the handle's stream with the NCCL backend (one rank: the mean of
    one gradient is that gradient, so the states must equal anakin_run's)."""
    import os

    import torch.distributed as dist

    from paper_2104_06272_b200 import replicas

    w = CASES["mma_h64"]
    a = make(bnd, w)
    a.reset(13)
    a.run(2)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(28500 + os.getpid() % 1000)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        stream = torch.cuda.Stream()
        r = replicas.ReplicatedAnakin(w, rank=0, world=1, stream=stream, always_exchange=True)
        r.reset(13)
        r.run(2)
        assert np.array_equal(a.get(bnd.PARAMS), r.an.get(bnd.PARAMS))
        assert r.an.status() == 0
    finally:
        dist.destroy_process_group()
