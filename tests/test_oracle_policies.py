"""Pins for the oracle's many-policies functions (CPU only): K independent networks, policy p on its own envs.

Nothing couples the policies, so the functions must equal K separate calls of the single-policy functions (which have
pins of their own) on the policy's slice of the inputs, bit for bit, and K = 1 must be the single-policy path itself.
"""
import math

import numpy as np
import pytest

from oracle import binding as orc
from paper_2104_06272_b200.workloads import random_params


def setup(seed, B, N, H, K):
    walls, start, goal = orc.env_init(seed, B, N)
    theta = np.stack([random_params(100 + p, orc.Dims(N, H).P, 0.25) for p in range(K)])
    return walls, start, goal, theta


def test_policy_env_ranges_partition_the_batch():
    for B, K in ((10, 3), (64, 1), (64, 64), (100, 7), (192, 3)):
        spans = [orc.policy_envs(B, K, p) for p in range(K)]
        assert spans[0][0] == 0 and all(n >= 1 for _, n in spans)
        assert all(spans[p][0] + spans[p][1] == spans[p + 1][0] for p in range(K - 1))
        assert spans[-1][0] + spans[-1][1] == B
        assert len({n for _, n in spans[:-1]}) <= 1  # all but the last policy have ceil(B/K) envs


def test_env_offset_draws_what_the_whole_batch_draws():
    """A slice of a batch run with env0 = its first global env index records exactly the columns of the full run."""
    B, N, H, T, seed = 12, 5, 16, 7, 3
    walls, start, goal, theta = setup(seed, B, N, H, 1)
    pos, tep = start.copy(), np.zeros(B, np.uint8)
    full = orc.rollout(N, H, 0, T, 6, theta[0], walls, start, goal, pos, tep, seed, 40)
    e0, n = 5, 4
    sl = slice(e0, e0 + n)
    p2, t2 = start[sl].copy(), np.zeros(n, np.uint8)
    part = orc.rollout(N, H, 0, T, 6, theta[0], np.ascontiguousarray(walls[sl]), start[sl].copy(), goal[sl].copy(), p2, t2, seed, 40, env0=e0)
    for name in ("pos", "action", "done", "reward", "value", "logp", "near"):
        assert np.array_equal(getattr(part, name), getattr(full, name)[:, sl]), name
    assert np.array_equal(p2, pos[sl]) and np.array_equal(t2, tep[sl])
    # without the offset the slice draws other uniforms: some action differs
    p3, t3 = start[sl].copy(), np.zeros(n, np.uint8)
    other = orc.rollout(N, H, 0, T, 6, theta[0], np.ascontiguousarray(walls[sl]), start[sl].copy(), goal[sl].copy(), p3, t3, seed, 40)
    assert not np.array_equal(other.action, part.action)


@pytest.mark.parametrize("B,K", [(9, 1), (10, 3), (24, 4)])
def test_policies_equal_separate_single_policy_runs(B, K):
    N, H, T, seed, cap = 5, 16, 6, 8, 5
    walls, start, goal, theta = setup(seed, B, N, H, K)
    pos, tep = start.copy(), np.zeros(B, np.uint8)
    tr = orc.rollout_policies(K, N, H, 0, T, cap, theta, walls, start, goal, pos, tep, seed, 17)
    adv, ret = orc.gae_policies(K, B, T, 0.99, 0.95, tr.reward, tr.value, tr.done)
    grads, loss = orc.learn_policies(K, N, H, 0, T, theta, walls, goal, tr.pos, tr.action, adv, ret)
    for p in range(K):
        e0, n = orc.policy_envs(B, K, p)
        sl = slice(e0, e0 + n)
        p1, t1 = start[sl].copy(), np.zeros(n, np.uint8)
        one = orc.rollout(N, H, 0, T, cap, theta[p], np.ascontiguousarray(walls[sl]), start[sl].copy(), goal[sl].copy(), p1, t1,
                          seed, 17, env0=e0)
        for name in ("pos", "action", "done", "reward", "logp", "near"):
            assert np.array_equal(orc.block(getattr(tr, name), B, K, p, T), getattr(one, name)), (p, name)
        assert np.array_equal(orc.block(tr.value, B, K, p, T + 1), one.value)
        assert np.array_equal(orc.block(tr.logits, B, K, p, T, 4), one.logits)
        assert np.array_equal(pos[sl], p1) and np.array_equal(tep[sl], t1)
        a1, r1 = orc.gae(0.99, 0.95, one.reward, one.value, one.done)
        assert np.array_equal(orc.block(adv, B, K, p, T), a1) and np.array_equal(orc.block(ret, B, K, p, T), r1)
        g1, l1 = orc.learn(N, H, 0, theta[p], np.ascontiguousarray(walls[sl]), goal[sl].copy(), one.pos, one.action, a1, r1)
        assert np.array_equal(grads[p], g1) and np.array_equal(loss[p], l1)
    if K > 1:  # different parameters: the policies really act and learn differently
        assert not np.array_equal(grads[0], grads[1])


def test_policy_parameter_init_draws_counter_i_p():
    N, H, seed = 5, 16, (3 << 32) | 77
    d = orc.Dims(N, H)
    assert np.array_equal(orc.param_init_policy(seed, N, H, 0), orc.param_init(seed, N, H))
    th = [orc.param_init_policy(seed, N, H, p) for p in range(3)]
    assert not np.array_equal(th[1], th[0]) and not np.array_equal(th[2], th[1])
    s = d.slices()
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for p in (1, 2):
        for i in (0, 7, s["W2"].start + 5, s["Wh"].start + 3, s["Wh"].start + 4):
            u = orc.uniform24(int(orc.philox4x32_10([i, p, 0, 2], key)[0]))
            if i < s["b1"].start:
                bound = math.sqrt(6.0 / (d.D + H))
            elif i < s["b2"].start:
                bound = math.sqrt(6.0 / (H + H))
            else:
                bound = math.sqrt(6.0 / (H + (4 if (i - s["Wh"].start) % 5 < 4 else 1)))
            assert th[p][i] == np.float32((2.0 * u - 1.0) * bound)
        for k in ("b1", "b2", "bh"):
            assert not th[p][s[k]].any()
