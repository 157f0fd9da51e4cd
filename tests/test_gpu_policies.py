"""Many policies on the GPU (needs a B200): K independent networks side by side, each on its own envs, against the
oracle policy by policy (the same staged, teacher-forced comparison as for one policy) and against the oracle's
many-policies functions."""
import numpy as np
import pytest
import torch

from oracle import binding as orc
from paper_2104_06272_b200.workloads import WORKLOADS, Workload, forced_actions, random_params
from tests import parity as par

pytestmark = pytest.mark.gpu

CASES = {
    # K, ragged B/K (the last policy has fewer envs), several CTA tiles per policy, the three hidden widths
    "k1_h64": Workload("k1_h64", B=70, N=5, H=64, T=6, iters=1, episode_cap=7, n_policies=1),
    "k3_h64_ragged": Workload("k3_h64_ragged", B=100, N=5, H=64, T=9, iters=1, episode_cap=7, n_policies=3),
    "k64_h64": Workload("k64_h64", B=64 * 40 - 13, N=6, H=64, T=8, iters=1, episode_cap=9, n_policies=64),
    "k3_h128_ragged": Workload("k3_h128_ragged", B=230, N=8, H=128, T=7, iters=1, episode_cap=9, n_policies=3),
    "k5_h128": Workload("k5_h128", B=5 * 96, N=10, H=128, T=12, iters=1, episode_cap=9, n_policies=5),
}


@pytest.fixture(scope="module")
def bnd():
    from paper_2104_06272_b200 import binding

    return binding


def make(bnd, w, debug=1):
    return bnd.Anakin(bnd.cfg_from_workload(w, debug_logits=debug))


def policy_thetas(w, K, seed=5):
    return np.stack([random_params(seed + 17 * p, w.P, 0.15) for p in range(K)])


def policy_state(an, bnd, p):
    """Host copy of policy p's state, as tests/parity.py's comparisons expect it."""
    e0, n = an.policy_envs(p)
    sl = slice(e0, e0 + n)
    P = an.P
    W = (an.N * an.N + 31) // 32
    return dict(theta=an.get(bnd.PARAMS).reshape(an.K, P)[p].copy(), m=an.get(bnd.ADAM_M).reshape(an.K, P)[p].copy(),
                v=an.get(bnd.ADAM_V).reshape(an.K, P)[p].copy(), k=int(an.get(bnd.ADAM_STEP)),
                walls=np.ascontiguousarray(an.get(bnd.ENV_WALLS).reshape(an.B, W)[sl]), start=an.get(bnd.ENV_START)[sl].copy(),
                goal=an.get(bnd.ENV_GOAL)[sl].copy(), pos=an.get(bnd.ENV_POS)[sl].copy(), tep=an.get(bnd.ENV_TEP)[sl].copy(),
                gstep=int(an.get(bnd.GLOBAL_STEP)))


def policy_traj(an, bnd, p, T):
    blk = lambda which, rows=T, width=1: np.ascontiguousarray(an.policy_block(an.get(which), p, rows, width))
    return dict(pos=blk(bnd.TRAJ_POS), action=blk(bnd.TRAJ_ACTION), done=blk(bnd.TRAJ_DONE), reward=blk(bnd.TRAJ_REWARD),
                value=blk(bnd.TRAJ_VALUE, T + 1), logp=blk(bnd.TRAJ_LOGP), logits=blk(bnd.DEBUG_LOGITS, T, 4))


@pytest.mark.parametrize("name", list(CASES))
def test_policies_reset_is_bit_exact(bnd, name):
    w = CASES[name]
    seed = (9 << 32) | 4242
    an = make(bnd, w)
    an.reset(seed)
    walls, start, goal = orc.env_init(seed, w.B, w.N, w.wall_density)
    assert (an.get(bnd.ENV_WALLS).reshape(w.B, -1) == walls).all()
    assert (an.get(bnd.ENV_START) == start).all() and (an.get(bnd.ENV_GOAL) == goal).all() and (an.get(bnd.ENV_POS) == start).all()
    theta = an.get(bnd.PARAMS).reshape(an.K, an.P)
    for p in range(an.K):
        assert (theta[p].view(np.uint32) == orc.param_init_policy(seed, w.N, w.H, p).view(np.uint32)).all(), p
    if an.K > 1:
        assert not np.array_equal(theta[0], theta[1])
    assert not an.get(bnd.ADAM_M).any() and an.status() == 0


@pytest.mark.parametrize("name", list(CASES))
def test_policies_env_transitions_bit_exact_under_forced_actions(bnd, name):
    w = CASES[name]
    an = make(bnd, w)
    an.reset(3)
    T = w.T
    # one [T][B_p] block of forced actions per policy
    blocks = [forced_actions(50 + p, T, an.policy_envs(p)[1]) for p in range(an.K)]
    sts = [policy_state(an, bnd, p) for p in range(an.K)]
    an.rollout_forced(torch.from_numpy(np.concatenate([b.ravel() for b in blocks])).cuda().reshape(T, w.B))
    assert an.status() == 0
    for p in range(an.K):
        e0, n = an.policy_envs(p)
        par.compare_rollout(w, 3, sts[p], policy_traj(an, bnd, p, T), T, an.get(bnd.ENV_POS)[e0:e0 + n], an.get(bnd.ENV_TEP)[e0:e0 + n],
                            forced=blocks[p], env0=e0)


@pytest.mark.parametrize("name", list(CASES))
def test_policies_one_iteration_stage_by_stage(bnd, name):
    """Each policy of the handle against the single-policy oracle functions on its slice of the state."""
    w = CASES[name]
    seed = 11
    an = make(bnd, w)
    an.reset(seed)
    an.set(bnd.PARAMS, policy_thetas(w, an.K))
    T = w.T
    for it in range(2):  # the second pass starts from the updated parameters, Adam state and env state
        sts = [policy_state(an, bnd, p) for p in range(an.K)]
        an.rollout()
        assert an.status() == 0 and int(an.get(bnd.GLOBAL_STEP)) == sts[0]["gstep"] + T
        trajs = [policy_traj(an, bnd, p, T) for p in range(an.K)]
        near = 0
        for p in range(an.K):
            e0, n = an.policy_envs(p)
            near += par.compare_rollout(w, seed, sts[p], trajs[p], T, an.get(bnd.ENV_POS)[e0:e0 + n], an.get(bnd.ENV_TEP)[e0:e0 + n],
                                        env0=e0)["near"]
        an.gae()
        adv_all, ret_all = an.get(bnd.ADV), an.get(bnd.RET)
        an.learn()
        grads = an.get(bnd.GRADS).reshape(an.K, an.P)
        gates_all = an.get(bnd.DEBUG_GATES)
        stats = an.stats() if an.K > 1 else [an.stats()]
        k_new, m_new, v_new, th_new = int(an.get(bnd.ADAM_STEP)), an.get(bnd.ADAM_M).reshape(an.K, an.P), an.get(bnd.ADAM_V).reshape(
            an.K, an.P), an.get(bnd.PARAMS).reshape(an.K, an.P)
        GW = w.H // 32
        worst = {}
        goff = 0  # the gate blob holds, per policy, [2][R_p][H/32] words
        for p in range(an.K):
            e0, n = an.policy_envs(p)
            g = trajs[p]
            oadv, oret = orc.gae(np.float32(w.gamma), np.float32(w.gae_lambda), g["reward"], g["value"], g["done"])
            gadv, gret = an.policy_block(adv_all, p, T), an.policy_block(ret_all, p, T)
            par.assert_close(gadv, oadv, par.RTOL_FP32, "advantages")
            par.assert_close(gret, oret, par.RTOL_FP32, "returns")
            R = n * T
            gates = gates_all[goff:goff + 2 * R * GW].reshape(2, R, GW)
            goff += 2 * R * GW
            s = stats[p]
            par.compare_learn(w, sts[p], g, np.ascontiguousarray(gadv), np.ascontiguousarray(gret), grads[p], gates,
                              [s.loss_total, s.loss_pg, s.loss_value, s.entropy], dict(k=k_new, m=m_new[p], v=v_new[p], theta=th_new[p]))
            assert s.frames == (it + 1) * R
            for kk, vv in par.MARGINS.items():
                worst[kk] = max(worst.get(kk, 0.0), vv)
        assert goff == gates_all.size
        print(name, "iteration", it, "near-boundary samples", near, "worst error / bound:", {k: round(v, 3) for k, v in worst.items() if k.startswith("grad")})


def test_policies_match_the_oracles_many_policies_functions(bnd):
    """The whole handle against the oracle's own K-policy loop (blob layouts included): transitions bit-exact when the
    oracle replays the library's actions is covered above; here both sides run the update on the library's trajectory."""
    w = CASES["k3_h64_ragged"]
    an = make(bnd, w)
    an.reset(21)
    thetas = policy_thetas(w, an.K, seed=31)
    an.set(bnd.PARAMS, thetas)
    an.rollout()
    T, K = w.T, an.K
    walls, goal = an.get(bnd.ENV_WALLS).reshape(w.B, -1), an.get(bnd.ENV_GOAL)
    oadv, oret = orc.gae_policies(K, w.B, T, np.float32(w.gamma), np.float32(w.gae_lambda), an.get(bnd.TRAJ_REWARD), an.get(bnd.TRAJ_VALUE),
                                  an.get(bnd.TRAJ_DONE))
    an.gae()
    par.assert_close(an.get(bnd.ADV), oadv, par.RTOL_FP32, "advantages, all policies")
    an.learn()
    ograds, oloss, reps = orc.learn_policies(K, w.N, w.H, 0, T, thetas, walls, goal, an.get(bnd.TRAJ_POS), an.get(bnd.TRAJ_ACTION),
                                             an.get(bnd.ADV), an.get(bnd.RET), np.float32(w.value_coef), np.float32(w.entropy_coef),
                                             gates=split_gates(an, bnd, w))
    grads = an.get(bnd.GRADS).reshape(K, an.P)
    for p in range(K):
        assert reps[p]["layer1"]["mismatched"] + reps[p]["layer2"]["mismatched"] <= 10
        for nm, sl in orc.Dims(w.N, w.H).slices().items():
            par.assert_close(grads[p][sl], ograds[p][sl], par.RTOL_FP32, f"policy {p} grad {nm}")
        s = an.stats()[p]
        assert abs(s.loss_total - oloss[p][0]) <= 1e-4 * (abs(oloss[p][0]) + 1e-3)


def split_gates(an, bnd, w):
    """The library's gate blob is per policy [2][R_p][H/32]; the oracle wants (layer-1 blocks, layer-2 blocks)."""
    allg, GW, g1, g2, off = an.get(bnd.DEBUG_GATES), w.H // 32, [], [], 0
    for p in range(an.K):
        R = an.policy_envs(p)[1] * w.T
        g1.append(allg[off:off + R * GW])
        g2.append(allg[off + R * GW:off + 2 * R * GW])
        off += 2 * R * GW
    return np.concatenate(g1), np.concatenate(g2)


def test_a_policy_of_a_group_equals_a_single_policy_handle_on_its_envs(bnd):
    """Nothing couples the policies: policy p of a K-policy handle walks the states of a one-policy handle created with
    env_offset = p*Bp, the same parameters and the same seed (trajectories bit for bit: the same rollout kernel)."""
    w = CASES["k3_h64_ragged"]
    an = make(bnd, w, debug=0)
    an.reset(8)
    thetas = policy_thetas(w, an.K, seed=3)
    an.set(bnd.PARAMS, thetas)
    an.rollout()
    ones = {}
    for p in (0, 2):  # a full policy and the ragged last one
        e0, n = an.policy_envs(p)
        one = bnd.Anakin(bnd.cfg_from_workload(w.scaled(B=n, n_policies=0), env_offset=e0))
        one.reset(8)
        one.set(bnd.PARAMS, thetas[p])
        one.rollout()
        for which in (bnd.TRAJ_POS, bnd.TRAJ_ACTION, bnd.TRAJ_REWARD, bnd.TRAJ_VALUE, bnd.TRAJ_LOGP):
            rows = w.T + 1 if which == bnd.TRAJ_VALUE else w.T
            assert np.array_equal(an.policy_block(an.get(which), p, rows), one.get(which).reshape(rows, n)), (p, which)
        ones[p] = one
    an.learn()
    for p, one in ones.items():
        one.learn()
        # the update runs on other kernels there (tcgen05 GEMMs), which sum in another order
        gp, g1 = an.get(bnd.GRADS).reshape(an.K, an.P)[p].astype(np.float64), one.get(bnd.GRADS).astype(np.float64)
        assert np.abs(gp - g1).max() <= 2e-5 * (np.abs(g1).max())
        tp, t1 = an.get(bnd.PARAMS).reshape(an.K, an.P)[p].astype(np.float64), one.get(bnd.PARAMS).astype(np.float64)
        assert np.abs(tp - t1).max() <= 2.01 * w.lr and np.mean(np.abs(tp - t1) > 1e-6) < 1e-2
        assert one.status() == 0
    assert an.status() == 0


def test_policies_runs_are_bitwise_deterministic_and_limits_are_refused(bnd):
    w = CASES["k64_h64"]
    outs = []
    for _ in range(2):
        an = make(bnd, w, debug=0)
        an.reset(5)
        an.run(3)
        outs.append((an.get(bnd.PARAMS), an.get(bnd.TRAJ_ACTION), an.get(bnd.ADV)))
        assert an.status() == 0
        st = an.stats()
        assert len(st) == 64 and all(s.frames == 3 * an.policy_envs(p)[1] * w.T for p, s in enumerate(st))
        assert all(np.isfinite(s.loss_total) for s in st)
    for a, b in zip(*outs):
        assert (a.view(np.uint8) == b.view(np.uint8)).all()
    an = make(bnd, CASES["k3_h64_ragged"], debug=0)
    an.reset(1)
    an.rollout()
    with pytest.raises(bnd.AnakinError) as e:
        an.learn_ppo(2, 0.2)
    assert e.value.code == bnd.E_UNSUPPORTED_CFG
    with pytest.raises(bnd.AnakinError) as e:
        an.learn_vtrace(1)
    assert e.value.code == bnd.E_UNSUPPORTED_CFG
    for kw, code in ((dict(precision=1), bnd.E_UNSUPPORTED_CFG), (dict(H=96), bnd.E_UNSUPPORTED_CFG), (dict(H=256), bnd.E_UNSUPPORTED_CFG), (dict(B=2), bnd.E_INVALID_ARG),
                     (dict(B=9, n_policies=4), bnd.E_INVALID_ARG)):  # 9 envs over 4 policies of 3 would leave the last one empty
        args = dict(B=100, N=5, H=64, T_max=4, n_policies=3)
        args.update(kw)
        with pytest.raises(bnd.AnakinError) as e:
            bnd.workspace_bytes(bnd.make_cfg(**args))
        assert e.value.code == code, kw
