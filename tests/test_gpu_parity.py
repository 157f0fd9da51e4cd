"""GPU-vs-oracle parity through the C ABI (needs a B200).

Stages are teacher-forced: one flipped action would send a free-running comparison down a different
trajectory, so each stage of the library is fed to the oracle and compared there.
"""
import numpy as np
import pytest
import torch

from oracle import binding as orc
from paper_2104_06272_b200.workloads import WORKLOADS, Workload, forced_actions, random_params
from tests import parity as par

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bnd():
    from paper_2104_06272_b200 import binding

    return binding


def make(bnd, w, T_max=None, debug=1):
    return bnd.Anakin(bnd.cfg_from_workload(w, debug_logits=debug, T_max=T_max))


# Reduced-batch versions of the large workloads (same grid, network, T and precision) whose oracle run takes
# seconds; they still span several CTA tiles and a ragged tail.
SMALL = {
    "tiny": WORKLOADS["tiny"],
    "memory_bound_s": WORKLOADS["memory_bound"].scaled(name="memory_bound_s", B=2048 + 37),
    "large_batch_s": WORKLOADS["large_batch"].scaled(name="large_batch_s", B=1024 + 19),
    "tensor_core_s": WORKLOADS["tensor_core"].scaled(name="tensor_core_s", B=256 + 5),
    "ragged": Workload("ragged", B=77, N=7, H=96, T=5, iters=1, episode_cap=6),
    "one_env": Workload("one_env", B=1, N=2, H=32, T=1, iters=1, episode_cap=1, wall_density=0.0),
    "dense_walls": Workload("dense_walls", B=130, N=16, H=32, T=9, iters=1, episode_cap=255, wall_density=0.9),
    "ragged_bf16": Workload("ragged_bf16", B=45, N=6, H=192, T=7, iters=1, precision=1, episode_cap=4),
    # ragged shapes on the tensor-pipe path (H in {64, 128, 256}): batch tails, T not a multiple of the t-slices,
    # grids whose cell count is not a multiple of 32, the bf16 operand format
    "tp_ragged_128": Workload("tp_ragged_128", B=333, N=9, H=128, T=11, iters=1, episode_cap=7),
    "tp_ragged_256": Workload("tp_ragged_256", B=150, N=12, H=256, T=7, iters=1, episode_cap=9, wall_density=0.35),
    "tp_ragged_64": Workload("tp_ragged_64", B=97, N=3, H=64, T=3, iters=1, episode_cap=2),
    "tp_bf16_128": Workload("tp_bf16_128", B=210, N=7, H=128, T=6, iters=1, precision=1, episode_cap=5),
    "tp_bf16_256": Workload("tp_bf16_256", B=131, N=16, H=256, T=5, iters=1, precision=1),
    # the second env (torus: moves wrap around the edges) on every rollout path: persistent tensor-pipe kernel,
    # FFMA kernel, wide bf16 path
    "torus_tp_256": Workload("torus_tp_256", B=140, N=6, H=256, T=12, iters=1, episode_cap=9, env_kind=1),
    "torus_ffma_96": Workload("torus_ffma_96", B=77, N=5, H=96, T=12, iters=1, episode_cap=9, env_kind=1),
    "torus_wide_512": Workload("torus_wide_512", B=70, N=8, H=512, T=6, iters=1, precision=1, episode_cap=9, env_kind=1),
    # the two-group tcgen05 rollout (H = 128) takes batches of at least one 128-env CTA per SM: a second, ragged wave of
    # CTAs whose last one has a full first group and 13 envs in the second
    "tc128_two_groups": Workload("tc128_two_groups", B=148 * 128 + 77, N=8, H=128, T=5, iters=1, episode_cap=4),
    # the two-group CTA-pair rollout (H = 256) takes batches of at least 74 clusters of 128 envs: a ragged second wave whose
    # last cluster has a full first group and 21 envs (all in its first CTA) in the second
    "pair2_two_groups": Workload("pair2_two_groups", B=74 * 128 + 85, N=10, H=256, T=4, iters=1, episode_cap=3),
    "tc128_torus": Workload("tc128_torus", B=148 * 128 + 3, N=6, H=128, T=6, iters=1, episode_cap=5, env_kind=1, wall_density=0.3),
}


@pytest.mark.parametrize("name", list(SMALL))
def test_reset_is_bit_exact(bnd, name):
    w = SMALL[name]
    seed = (7 << 32) | 12345
    an = make(bnd, w)
    an.reset(seed)
    walls, start, goal = orc.env_init(seed, w.B, w.N, w.wall_density)
    assert (an.get(bnd.ENV_WALLS).reshape(w.B, -1) == walls).all()
    assert (an.get(bnd.ENV_START) == start).all() and (an.get(bnd.ENV_GOAL) == goal).all()
    assert (an.get(bnd.ENV_POS) == start).all() and not an.get(bnd.ENV_TEP).any()
    theta = orc.param_init(seed, w.N, w.H)
    assert (an.get(bnd.PARAMS).view(np.uint32) == theta.view(np.uint32)).all()
    assert not an.get(bnd.ADAM_M).any() and not an.get(bnd.ADAM_V).any()
    assert int(an.get(bnd.ADAM_STEP)) == 0 and int(an.get(bnd.GLOBAL_STEP)) == 0
    s = an.stats()
    assert (s.frames, s.episodes, s.goals, s.episode_steps) == (0, 0, 0, 0)
    assert an.status() == 0


@pytest.mark.parametrize("name", list(SMALL))
def test_env_transitions_bit_exact_under_forced_actions(bnd, name):
    w = SMALL[name]
    an = make(bnd, w)
    an.reset(3)
    for it in range(2):  # the second pass continues from the first pass's env state
        st = par.gpu_state(an, bnd)
        f = forced_actions(100 + it, w.T, w.B)
        g, _ = par.check_rollout(an, bnd, w, 3, st, w.T, forced=f)
    s = an.stats()
    assert s.frames == 2 * w.T * w.B


@pytest.mark.parametrize("name", list(SMALL))
def test_one_iteration_stage_by_stage(bnd, name):
    w = SMALL[name]
    an = make(bnd, w)
    an.reset(11)
    # start from parameters with non-zero biases so every term of the network is exercised
    an.set(bnd.PARAMS, random_params(5, w.P, 0.15))
    par.MARGINS.clear()
    try:
        counts = par.check_iteration(an, bnd, w, 11)
        # and a second iteration from the updated parameters and Adam state
        counts2 = par.check_iteration(an, bnd, w, 11)
        print(name, "near-boundary samples:", counts, counts2)
    finally:
        print(name, "worst error / bound (last comparison of each tensor):", {k: round(v, 3) for k, v in par.MARGINS.items()})


@pytest.mark.parametrize("name", ["tp_ragged_128", "tp_ragged_256", "large_batch_s", "tp_bf16_256"])
def test_an_iteration_shorter_than_t_max(bnd, name):
    """A rollout of fewer steps than the handle was sized for, then the update: the launch plans (partial counts, grids)
    are made for T_max, so some CTAs of the update kernels find no rows (the fused heads + dW2 kernel then contributes a
    zero partial) and the t-slices of the dh1 kernel are cut from fewer steps."""
    w = SMALL[name]
    an = make(bnd, w)
    an.reset(13)
    an.set(bnd.PARAMS, random_params(6, w.P, 0.15))
    par.check_iteration(an, bnd, w, 13, T=2)
    par.check_iteration(an, bnd, w, 13, T=1)


def free_running_seed(ag, iters, learn=True):
    """First seed for which the ORACLE's own free run draws no uniform within 1e-5 of a CDF boundary (about one sample in
    17,000 does): on such a run the library has no excuse for a different action, so nothing needs to be skipped."""
    for seed in range(1, 50):
        ag.reset(seed)
        clean = True
        for _ in range(iters):
            clean = clean and not ag.rollout().near.any()
            if learn:
                ag.learn()
        if clean:
            return seed
    raise AssertionError("no seed without near-boundary samples")


def test_tiny_free_running_end_to_end(bnd):
    """The tiny workload, both sides run freely for its 2 iterations from one seed: same actions, same
    trajectories, parameters within tolerance."""
    w = WORKLOADS["tiny"]
    an = make(bnd, w)
    ag = orc.Agent(w.B, w.N, w.H, w.T, w.precision, w.episode_cap, w.wall_density, np.float32(w.gamma),
                   np.float32(w.gae_lambda), np.float32(w.entropy_coef), np.float32(w.value_coef), np.float32(w.lr),
                   np.float32(w.adam_b1), np.float32(w.adam_b2), np.float32(w.adam_eps))
    seed = free_running_seed(ag, w.iters)
    an.reset(seed)
    ag.reset(seed)
    for it in range(w.iters):
        an.rollout()
        tr = ag.rollout()
        g = par.gpu_traj(an, bnd, w.T)
        assert not tr.near.any()
        assert (g["action"] == tr.action).all()  # no sample of this run is near a CDF boundary: every action must agree
        assert (g["pos"] == tr.pos).all() and (g["reward"] == tr.reward).all() and (g["done"] == tr.done).all()
        par.assert_close(g["value"], tr.value, 1e-4, "values")
        an.learn()
        ag.learn()
        par.assert_close(an.get(bnd.ADV), ag.adv, 1e-4, "adv")
        par.assert_close(an.get(bnd.GRADS), ag.grads, 1e-4, "grads")
    # Adam's first steps are ~lr*sign(g): compare parameters where the gradient is not within rounding of zero
    gt, ot = an.get(bnd.PARAMS), ag.theta
    assert np.abs(gt - ot).max() <= 2.1 * w.iters * w.lr
    big = np.abs(ag.grads) > 1e-3 * np.sqrt((ag.grads.astype(np.float64) ** 2).mean())
    par.assert_close(gt[big], ot[big], 1e-4, "params")
    s = an.stats()
    assert s.frames == w.B * w.T * w.iters and abs(s.loss_total - ag.loss[0]) < 1e-4 * (abs(ag.loss[0]) + 1e-2)


def test_throughput_workload_full_size(bnd):
    """The benchmarked configuration at full size (B=4096, 10x10, 300-256-256, T=32), two iterations."""
    w = WORKLOADS["throughput"]
    an = make(bnd, w)
    an.reset(1)
    for _ in range(2):
        print("throughput near-boundary:", par.check_iteration(an, bnd, w, 1))


@pytest.mark.parametrize("name", ["memory_bound", "large_batch", "tensor_core"])
def test_full_size_workloads_on_sampled_envs(bnd, name):
    """Full-size launches of the three large workloads.  The oracle replays a sample of envs for the acting
    stage and for GAE; the learner's full-batch gradient is checked through properties that hold at any size
    (it is compared element by element on the reduced-batch versions above and, at full size, in
    test_full_size_learner_element_by_element)."""
    w = WORKLOADS[name]
    an = make(bnd, w)
    an.reset(2)
    rng = np.random.default_rng(0)
    sel = np.unique(np.concatenate([[0, 1, 31, 32, w.B - 1], rng.integers(0, w.B, 59)]))
    st = par.gpu_state(an, bnd)
    g, counts = par.check_rollout(an, bnd, w, 2, st, w.T, envs=sel)
    an.gae()
    adv, ret = orc.gae(np.float32(w.gamma), np.float32(w.gae_lambda), np.ascontiguousarray(g["reward"][:, sel]),
                       np.ascontiguousarray(g["value"][:, sel]), np.ascontiguousarray(g["done"][:, sel]))
    gadv = an.get(bnd.ADV).reshape(w.T, w.B)
    par.assert_close(gadv[:, sel], adv, 1e-4, "advantages")
    par.assert_close(an.get(bnd.RET).reshape(w.T, w.B)[:, sel], ret, 1e-4, "returns")
    an.learn()
    grads = an.get(bnd.GRADS)
    assert np.isfinite(grads).all() and np.abs(grads).max() > 0
    sl = orc.Dims(w.N, w.H).slices()
    bh = grads[sl["bh"]]
    # softmax gradients sum to zero in every row; in the bf16 workload each of the four is rounded to bf16 (2^-9) before
    # the batch sum, so the cancellation is only as good as that rounding
    assert abs(bh[:4].sum()) <= (1e-3 if w.precision == 0 else 1e-2) * np.abs(bh[:4]).max() + 1e-9
    # loss terms from the recorded data alone: policy term = -mean(A * logp), entropy <= ln 4
    s = an.stats()
    rt = par.rtol_of(w.precision)
    want_pg = -(gadv.astype(np.float64) * g["logp"]).mean()
    assert abs(s.loss_pg - want_pg) <= max(rt, 1e-3) * (abs(want_pg) + np.abs(gadv).mean() * 1e-2)
    assert 0 < s.entropy <= np.log(4) + 1e-5
    assert abs(s.loss_total - (s.loss_pg + w.value_coef * s.loss_value - w.entropy_coef * s.entropy)) < 1e-5
    assert s.frames == w.B * w.T
    # first Adam step moves every parameter with a non-zero gradient by at most lr (plus rounding)
    step = an.get(bnd.PARAMS).astype(np.float64) - st["theta"]
    assert np.abs(step).max() <= w.lr * 1.01 and (step[grads == 0] == 0).all()
    assert an.status() == 0
    print(name, counts)


@pytest.mark.parametrize("name", ["memory_bound", "large_batch", "tensor_core"])
def test_full_size_learner_element_by_element(bnd, name):
    """The three large workloads at their full sizes, in the launch configuration the benchmark times: one whole
    update (gradient of every parameter block, loss terms, Adam moments, parameters, step) against the oracle run on
    the library's full trajectory.  The split-K counts, wave counts and partial-buffer sizes the update takes at these
    sizes occur nowhere else.  The oracle needs about 0.5-2.5 minutes of all host cores per case."""
    w = WORKLOADS[name]
    an = make(bnd, w)
    an.reset(2)
    an.set(bnd.PARAMS, random_params(5, w.P, 0.15 if w.H <= 256 else 0.05))  # non-zero biases
    st = par.gpu_state(an, bnd)
    an.rollout()
    T = w.T
    g = dict(pos=an.get(bnd.TRAJ_POS).reshape(T, w.B), action=an.get(bnd.TRAJ_ACTION).reshape(T, w.B),
             done=an.get(bnd.TRAJ_DONE).reshape(T, w.B), reward=an.get(bnd.TRAJ_REWARD).reshape(T, w.B),
             value=an.get(bnd.TRAJ_VALUE).reshape(T + 1, w.B))
    gadv, gret = par.check_gae(an, bnd, w, g, T)  # the whole batch: the scan is cheap on the CPU too
    par.MARGINS.clear()
    try:
        par.check_learn(an, bnd, w, st, g, gadv, gret)
    finally:
        print(name, "worst error / bound:", {k: round(v, 3) for k, v in par.MARGINS.items()})
    assert an.status() == 0


def test_bounded_device_wait_runs_out_and_reports(bnd):
    """A device-side wait that cannot end must give up, raise the 'bounded wait gave up' bit and return; the context
    stays usable and a reset clears the word.  The wait here is on a barrier nothing arrives on, with a short limit."""
    w = SMALL["tp_ragged_256"]
    an = make(bnd, w, debug=0)
    an.reset(1)
    an.rollout()
    assert an.status() == 0
    an.selftest_wait_timeout(2_000_000)  # about a millisecond of SM clock
    assert an.status() == 4
    an.learn()  # the context and the handle still work ...
    assert np.isfinite(an.get(bnd.PARAMS)).all()
    assert an.status() == 4  # ... and the word is sticky
    an.reset(1)
    assert an.status() == 0
    with pytest.raises(bnd.AnakinError):
        an.selftest_wait_timeout(0)


def test_profiler_brackets_replay_launches(bnd):
    """Per-kernel event timing around a PPO update of two epochs: the second epoch replays the forward pass once, and
    its launch must be bracketed like every other (one 'replay' record, a finite duration)."""
    w = SMALL["tp_ragged_128"]
    an = make(bnd, w, debug=0)
    an.reset(3)
    an.rollout()
    an.profile_enable(True)
    an.learn_ppo(2, 0.2)
    prof = an.profile_read()
    an.profile_enable(False)
    assert prof["replay"][1] == 1 and 0 < prof["replay"][0] < 100.0
    assert prof["heads_bwd"][1] == 2
    assert an.status() == 0


def test_runs_are_bitwise_deterministic(bnd):
    w = WORKLOADS["throughput"].scaled(B=1500, iters=3)
    outs = []
    for _ in range(2):
        an = make(bnd, w, debug=0)
        an.reset(9)
        an.run(3)
        outs.append((an.get(bnd.PARAMS), an.get(bnd.TRAJ_ACTION), an.get(bnd.TRAJ_VALUE), an.get(bnd.ENV_POS),
                     an.get(bnd.GRADS)))
    for a, b in zip(*outs):
        assert (a.view(np.uint8) == b.view(np.uint8)).all()
    an2 = make(bnd, w, debug=0)
    an2.reset(10)
    an2.run(3)
    assert (an2.get(bnd.PARAMS) != outs[0][0]).any()


def test_long_runs_of_the_benchmarked_workload_are_bitwise_reproducible(bnd):
    """The CTA pairs of the tcgen05 rollout hand operand tiles, accumulators and head partials to each other through
    mbarriers only; a missed ordering would show as a run that differs from its twin.  100 passes of the full-size
    throughput workload (3,300 rollout steps on 64 pairs), twice."""
    w = WORKLOADS["throughput"]
    outs = []
    for _ in range(2):
        an = make(bnd, w, debug=0)
        an.reset(2)
        an.run(100)
        outs.append((an.get(bnd.PARAMS), an.get(bnd.TRAJ_ACTION), an.get(bnd.TRAJ_VALUE), an.get(bnd.ADV)))
        assert an.status() == 0
    for a, b in zip(*outs):
        assert (a.view(np.uint8) == b.view(np.uint8)).all()
    assert np.isfinite(outs[0][0]).all()


@pytest.mark.parametrize("name", ["tc128_two_groups", "pair2_two_groups"])
def test_runs_of_the_large_batch_kernels_are_bitwise_reproducible(bnd, name):
    """The same for the kernels large batches take: the two-group rollouts, and the fused dh1 kernel walking several
    env tiles per CTA (one CTA per SM at H = 128, CTA pairs at H = 256) with its accumulators, operand tiles and gate
    tiles handed over through mbarriers.  20 passes, twice."""
    w = SMALL[name]
    outs = []
    for _ in range(2):
        an = make(bnd, w, debug=0)
        an.reset(6)
        an.run(20)
        outs.append((an.get(bnd.PARAMS), an.get(bnd.GRADS), an.get(bnd.TRAJ_ACTION), an.get(bnd.ADV)))
        assert an.status() == 0
    for a, b in zip(*outs):
        assert (a.view(np.uint8) == b.view(np.uint8)).all()
    assert np.isfinite(outs[0][0]).all()


def test_checkpoint_resume_is_bitwise(bnd):
    w = SMALL["large_batch_s"].scaled(B=300, T=8)
    a = make(bnd, w, debug=0)
    a.reset(4)
    a.run(4)
    b = make(bnd, w, debug=0)
    b.reset(4)
    b.run(2)
    # the Philox key is the seed: a resumed handle needs the same one, so resume = reset(seed) + state
    d = make(bnd, w, debug=0)
    d.reset(4)
    for blob in (bnd.PARAMS, bnd.ADAM_M, bnd.ADAM_V, bnd.ENV_POS, bnd.ENV_TEP):
        d.set(blob, b.get(blob))
    d.set(bnd.ADAM_STEP, b.get(bnd.ADAM_STEP))
    d.set(bnd.GLOBAL_STEP, b.get(bnd.GLOBAL_STEP))
    d.run(2)
    assert (d.get(bnd.PARAMS).view(np.uint32) == a.get(bnd.PARAMS).view(np.uint32)).all()
    assert (d.get(bnd.ENV_POS) == a.get(bnd.ENV_POS)).all()
    assert (d.get(bnd.ADAM_V).view(np.uint32) == a.get(bnd.ADAM_V).view(np.uint32)).all()


def test_run_equals_rollout_then_learn_and_enqueues_only(bnd):
    w = SMALL["ragged"]
    a = make(bnd, w, debug=0)
    b = make(bnd, w, debug=0)
    a.reset(6)
    b.reset(6)
    n0 = a.launch_count()
    a.run(3)
    per_iter = (a.launch_count() - n0) / 3
    assert per_iter == int(per_iter) and per_iter >= 3
    for _ in range(3):
        b.rollout()
        b.learn()
    assert (a.get(bnd.PARAMS) == b.get(bnd.PARAMS)).all() and (a.get(bnd.ENV_POS) == b.get(bnd.ENV_POS)).all()
    s = a.stats()
    assert s.frames == 3 * w.B * w.T and s.episodes > 0 and s.episode_steps >= s.episodes
    assert s.goals <= s.episodes


def test_state_errors(bnd):
    w = SMALL["ragged"]
    an = make(bnd, w)
    with pytest.raises(bnd.AnakinError) as e:
        an.rollout()
    assert e.value.code == bnd.E_BAD_STATE
    an.reset(1)
    with pytest.raises(bnd.AnakinError) as e:
        an.learn()
    assert e.value.code == bnd.E_BAD_STATE
    for T in (0, w.T + 1):
        with pytest.raises(bnd.AnakinError) as e:
            an.rollout(T)
        assert e.value.code == bnd.E_INVALID_ARG
    an.rollout(2)  # shorter than T_max is fine
    assert an.blob_bytes(bnd.TRAJ_REWARD) == 2 * w.B * 4
    an.learn()
    with pytest.raises(bnd.AnakinError):
        an.learn()  # the rollout was consumed
    with pytest.raises(bnd.AnakinError):
        an.set(bnd.STATS, torch.zeros(an.blob_bytes(bnd.STATS), dtype=torch.uint8))  # read-only blob
    with pytest.raises(bnd.AnakinError):
        an.set(bnd.PARAMS, np.zeros(an.P - 1, np.float32))  # wrong size
    # a forced action outside 0..3 sets the sticky device status instead of faulting
    bad = torch.full((w.T, w.B), 7, dtype=torch.int8, device="cuda")
    an.rollout_forced(bad)
    assert an.status() == 1


def test_on_policy_forward_reuse(bnd):
    """The update may reuse the policy's forward pass (Section 3.1): with unchanged parameters the learner's
    policy term -mean(A log pi) computed from ITS recomputed forward equals the one from the recorded logp."""
    w = SMALL["large_batch_s"]
    an = make(bnd, w)
    an.reset(8)
    an.rollout()
    logp = an.get(bnd.TRAJ_LOGP).astype(np.float64)
    an.learn()
    adv = an.get(bnd.ADV).astype(np.float64)
    s = an.stats()
    assert abs(s.loss_pg + (adv * logp).mean()) <= 1e-4 * (np.abs(adv * logp).mean() + 1e-6)


def test_update_from_set_trajectory_recomputes_the_forward_pass(bnd):
    """The learner reuses the activations the rollout saved (Section 3.1: the update may reuse the policy's forward
    pass).  A trajectory written with anakin_set has no saved activations: the library must recompute them, and the
    update must come out bitwise the same."""
    w = SMALL["large_batch_s"].scaled(B=200, T=9)
    a = make(bnd, w, debug=0)
    b = make(bnd, w, debug=0)
    for an in (a, b):
        an.reset(12)
        an.set(bnd.PARAMS, random_params(2, w.P, 0.15))
        an.rollout()
    b.set(bnd.TRAJ_POS, b.get(bnd.TRAJ_POS))  # same data, but it invalidates what the rollout saved
    n0 = b.launch_count()
    a.learn()
    b.learn()
    assert b.launch_count() - n0 > 0
    for blob in (bnd.GRADS, bnd.PARAMS, bnd.ADAM_V):
        assert (a.get(blob).view(np.uint32) == b.get(blob).view(np.uint32)).all()
    # and a trajectory built entirely from another handle's blobs
    c = make(bnd, w, debug=0)
    c.reset(12)
    c.set(bnd.PARAMS, random_params(2, w.P, 0.15))
    d = make(bnd, w, debug=0)
    d.reset(12)
    d.set(bnd.PARAMS, random_params(2, w.P, 0.15))
    c.rollout()
    d.rollout(1)  # fixes nothing but the blob sizes; every trajectory blob is overwritten below
    d.rollout()
    for blob in (bnd.TRAJ_POS, bnd.TRAJ_ACTION, bnd.TRAJ_DONE, bnd.TRAJ_REWARD, bnd.TRAJ_VALUE, bnd.TRAJ_LOGP):
        d.set(blob, c.get(blob))
    c.learn()
    d.learn()
    assert (c.get(bnd.GRADS).view(np.uint32) == d.get(bnd.GRADS).view(np.uint32)).all()


@pytest.mark.parametrize("name", ["tc128_two_groups", "pair2_two_groups"])
def test_two_group_rollout_replays_set_trajectories_bitwise(bnd, name):
    """The replay mode of the two-group tcgen05 rollouts (H = 128 and H = 256, large batch): an update from a trajectory
    written with anakin_set recomputes the activations with the same kernel and must equal the update from the rollout's own."""
    w = SMALL[name]
    a = make(bnd, w, debug=0)
    b = make(bnd, w, debug=0)
    for an in (a, b):
        an.reset(12)
        an.set(bnd.PARAMS, random_params(2, w.P, 0.15))
        an.rollout()
    b.set(bnd.TRAJ_POS, b.get(bnd.TRAJ_POS))  # same data, but it invalidates what the rollout saved
    a.learn()
    b.learn()
    for blob in (bnd.GRADS, bnd.PARAMS):
        assert (a.get(blob).view(np.uint32) == b.get(blob).view(np.uint32)).all()
    # and two runs of the kernel give the same bits (its groups meet through mbarriers only)
    c = make(bnd, w, debug=0)
    c.reset(12)
    c.set(bnd.PARAMS, random_params(2, w.P, 0.15))
    c.rollout()
    c.learn()
    assert (a.get(bnd.PARAMS).view(np.uint32) == c.get(bnd.PARAMS).view(np.uint32)).all()
    assert a.status() == 0 and b.status() == 0


def test_torus_env_free_running_and_different_from_the_grid(bnd):
    """The second env kind: the library and the oracle agent, both running freely from one seed, record the same
    trajectory; and the same seed under the grid rule gives a different one (some move crosses an edge)."""
    w = WORKLOADS["tiny"].scaled(name="tiny_torus", B=96, T=24, env_kind=1)
    an = make(bnd, w)
    ag = orc.Agent(w.B, w.N, w.H, w.T, w.precision, w.episode_cap, w.wall_density, np.float32(w.gamma),
                   np.float32(w.gae_lambda), np.float32(w.entropy_coef), np.float32(w.value_coef), np.float32(w.lr),
                   np.float32(w.adam_b1), np.float32(w.adam_b2), np.float32(w.adam_eps), kind=orc.TORUS)
    seed = free_running_seed(ag, 1, learn=False)
    an.reset(seed)
    ag.reset(seed)
    an.rollout()
    tr = ag.rollout()
    g = par.gpu_traj(an, bnd, w.T)
    assert not tr.near.any() and (g["action"] == tr.action).all()
    assert (g["pos"] == tr.pos).all() and (g["reward"] == tr.reward).all() and (g["done"] == tr.done).all()
    # a wrap really happened: some recorded step changes the column by N-1 or the row by N-1
    pos = np.concatenate([tr.pos, an.get(bnd.ENV_POS)[None, :]], axis=0).astype(np.int64)
    dr, dc = np.abs(np.diff(pos // w.N, axis=0)), np.abs(np.diff(pos % w.N, axis=0))
    moved_by_wrap = ((dr == w.N - 1) | (dc == w.N - 1)) & (tr.done == 0)
    assert moved_by_wrap.any()
    grid = make(bnd, w.scaled(env_kind=0))
    grid.reset(seed)
    grid.rollout()
    assert not (par.gpu_traj(grid, bnd, w.T)["pos"] == g["pos"]).all()
    an.learn()
    ag.learn()
    par.assert_close(an.get(bnd.GRADS), ag.grads, 1e-4, "grads")
    assert an.status() == 0


def test_asynchronous_copies_through_page_locked_host_memory(bnd):
    """ptr_is_device = 2: blobs move to and from pinned host buffers in stream order without a synchronisation per call;
    after one synchronising call the data is what the synchronous copies give."""
    import torch

    w = WORKLOADS["tiny"]
    an = make(bnd, w, debug=0)
    an.reset(4)
    an.rollout()
    an.learn()
    want = {b: an.get(b) for b in (bnd.PARAMS, bnd.ENV_POS, bnd.TRAJ_VALUE)}
    bufs = {b: torch.empty(v.size, dtype=torch.from_numpy(v).dtype).pin_memory() for b, v in want.items()}
    for b, t in bufs.items():
        an.get_into(b, t, wait=False)
    assert an.status() == 0  # synchronises
    for b, t in bufs.items():
        assert np.array_equal(t.numpy(), want[b])
    # and the other way: a pinned source, enqueued, then read back
    src = torch.from_numpy(want[bnd.PARAMS] * np.float32(0.5)).pin_memory()
    an.set(bnd.PARAMS, src)
    assert np.array_equal(an.get(bnd.PARAMS), src.numpy())
    with pytest.raises(bnd.AnakinError):
        an._ck(bnd._lib.anakin_get(an._h, bnd.PARAMS, bufs[bnd.PARAMS].data_ptr(), bufs[bnd.PARAMS].numel() * 4, 3))
