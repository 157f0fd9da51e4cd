"""anakin_learn_ppo (clipped-surrogate objective over the recorded trajectory) against the oracle, epoch by epoch,
on each learner path; and its reductions: one epoch = the A2C step, E epochs in one call = E single-epoch calls."""
import numpy as np
import pytest

from oracle import binding as orc
from paper_2104_06272_b200.workloads import WORKLOADS, Workload
from tests import parity as par

pytestmark = pytest.mark.gpu

CLIP = 0.2
CASES = {
    "mma_h64": WORKLOADS["tiny"].scaled(name="mma_h64", B=200, T=12),
    "mma_h256": Workload("mma_h256", B=150, N=9, H=256, T=7, iters=1, episode_cap=9),
    "ffma_h96": Workload("ffma_h96", B=77, N=7, H=96, T=5, iters=1, episode_cap=6),
    "wide_bf16": Workload("wide_bf16", B=140, N=8, H=512, T=5, iters=1, precision=1, episode_cap=9),
}


@pytest.fixture(scope="module")
def bnd():
    from paper_2104_06272_b200 import binding

    return binding


def make(bnd, w):
    return bnd.Anakin(bnd.cfg_from_workload(w, debug_logits=1))


TRAJ = ("TRAJ_POS", "TRAJ_ACTION", "TRAJ_DONE", "TRAJ_REWARD", "TRAJ_VALUE", "TRAJ_LOGP")


def rearm(an, bnd, blobs):
    """Writes the recorded trajectory back: it is pending again, and its forward pass will be recomputed."""
    for name in TRAJ:
        an.set(getattr(bnd, name), blobs[name])


@pytest.mark.parametrize("name", list(CASES))
def test_ppo_epochs_match_the_oracle_one_by_one(bnd, name):
    w = CASES[name]
    rtol = par.rtol_of(w.precision)
    # a larger learning rate, so that the ratios leave 1 +- clip within a few epochs and both branches are taken
    w = w.scaled(lr=0.02)
    an = make(bnd, w)
    an.reset(5)
    an.rollout()
    g = par.gpu_traj(an, bnd, w.T)
    blobs = {n: an.get(getattr(bnd, n)) for n in TRAJ}
    adv, ret = orc.gae(np.float32(w.gamma), np.float32(w.gae_lambda), g["reward"], g["value"], g["done"])
    R = g["pos"].size
    for epoch in range(4):
        st = par.gpu_state(an, bnd)
        if epoch > 0:
            rearm(an, bnd, blobs)
        an.learn_ppo(1, CLIP)
        gates = an.get(bnd.DEBUG_GATES).reshape(2, R, w.H // 32)
        ograds, oloss, rep = orc.learn(w.N, w.H, w.precision, st["theta"], st["walls"], st["goal"], g["pos"], g["action"], adv, ret,
                                       np.float32(w.value_coef), np.float32(w.entropy_coef), gates=(gates[0], gates[1]),
                                       logp_old=g["logp"], clip=CLIP)
        for layer, r in rep.items():
            assert r["max_abs_z"] <= 10 * rtol * r["rms_z"], (epoch, layer, r)
        ggrads = an.get(bnd.GRADS)
        for pname, sl in orc.Dims(w.N, w.H).slices().items():
            par.assert_close(ggrads[sl], ograds[sl], rtol, f"epoch {epoch} grad {pname}")
        s = an.stats()
        gl = np.array([s.loss_pg, s.loss_value, s.entropy], dtype=np.float64)
        assert (np.abs(gl - oloss[1:]) <= max(rtol, 1e-4) * (np.abs(oloss[1:]) + 1e-3 * np.abs(oloss).max()) + 1e-7).all(), (epoch, gl, oloss)
        assert int(an.get(bnd.ADAM_STEP)) == st["k"] + 1
    # the policy has moved: the last epoch's policy loss differs from the plain -mean(A) of ratio one
    assert abs(an.stats().loss_pg + adv.mean()) > 1e-6
    assert an.status() == 0


@pytest.mark.parametrize("name", ["mma_h64", "mma_h256", "wide_bf16"])
def test_one_ppo_epoch_is_the_a2c_step_bitwise_on_the_paths_that_reuse_the_forward_pass(bnd, name):
    """The recorded log-probability and the learner's come from the same saved head outputs with the same arithmetic,
    so the ratio is exactly one."""
    w = CASES[name]
    a, b = make(bnd, w), make(bnd, w)
    for an in (a, b):
        an.reset(8)
        an.rollout()
    a.learn()
    b.learn_ppo(1, CLIP)
    for which in (bnd.GRADS, bnd.PARAMS, bnd.ADAM_M, bnd.ADAM_V):
        assert np.array_equal(a.get(which), b.get(which)), which
    assert b.stats().loss_pg == pytest.approx(-float(b.get(bnd.ADV).astype(np.float64).mean()), rel=1e-5, abs=1e-7)


@pytest.mark.parametrize("name", list(CASES))
def test_epochs_in_one_call_equal_single_epoch_calls(bnd, name):
    w = CASES[name]
    a, b = make(bnd, w), make(bnd, w)
    for an in (a, b):
        an.reset(6)
        an.rollout()
    blobs = {n: b.get(getattr(bnd, n)) for n in TRAJ}
    a.learn_ppo(3, CLIP)
    for epoch in range(3):
        if epoch > 0:
            rearm(b, bnd, blobs)
        b.learn_ppo(1, CLIP)
    assert np.array_equal(a.get(bnd.PARAMS), b.get(bnd.PARAMS))
    assert np.array_equal(a.get(bnd.GRADS), b.get(bnd.GRADS))
    with pytest.raises(bnd.AnakinError):
        a.learn_ppo(1, CLIP)  # consumed
    assert a.status() == 0 and b.status() == 0


def test_ppo_argument_errors(bnd):
    w = CASES["mma_h64"]
    an = make(bnd, w)
    an.reset(1)
    with pytest.raises(bnd.AnakinError) as e:
        an.learn_ppo(1, CLIP)
    assert e.value.code == bnd.E_BAD_STATE
    an.rollout()
    for epochs, clip in ((0, CLIP), (1, 0.0), (1, -0.1)):
        with pytest.raises(bnd.AnakinError) as e:
            an.learn_ppo(epochs, clip)
        assert e.value.code == bnd.E_INVALID_ARG
