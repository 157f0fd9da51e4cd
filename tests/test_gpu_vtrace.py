"""anakin_learn_vtrace (V-trace targets over the recorded trajectory, then the A2C update) against the oracle on each
tensor path, off-policy (the parameters are changed between acting and learning) and in its reductions."""
import numpy as np
import pytest

from oracle import binding as orc
from paper_2104_06272_b200.workloads import WORKLOADS, Workload, random_params
from tests import parity as par

pytestmark = pytest.mark.gpu

CASES = {
    "mma_h64": WORKLOADS["tiny"].scaled(name="mma_h64", B=200, T=12),
    "pair_h256": Workload("pair_h256", B=150, N=9, H=256, T=7, iters=1, episode_cap=9),
    "wide_bf16": Workload("wide_bf16", B=140, N=8, H=512, T=5, iters=1, precision=1, episode_cap=9),
}
TRAJ = ("TRAJ_POS", "TRAJ_ACTION", "TRAJ_DONE", "TRAJ_REWARD", "TRAJ_VALUE", "TRAJ_LOGP")


@pytest.fixture(scope="module")
def bnd():
    from paper_2104_06272_b200 import binding

    return binding


def make(bnd, w):
    return bnd.Anakin(bnd.cfg_from_workload(w, debug_logits=1))


def oracle_heads(w, theta, walls, goal, pos_rows):
    """Oracle forward of the states `pos_rows` [n][B] (observation rebuilt from the state) -> out [n][B][5]."""
    n, B = pos_rows.shape
    x = np.stack([orc.observe(w.N, walls[b], int(pos_rows[t, b]), int(goal[b])) for t in range(n) for b in range(B)])
    return orc.forward(w.N, w.H, w.precision, theta, x).reshape(n, B, 5)


def logp_of(logits, action):
    l = logits.astype(np.float64)
    l = l - l.max(axis=-1, keepdims=True)
    lp = l - np.log(np.exp(l).sum(axis=-1, keepdims=True))
    return np.take_along_axis(lp, action.astype(np.int64)[..., None], axis=-1)[..., 0].astype(np.float32)


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("levels", [(1.0, 1.0), (1.1, 0.9)])
def test_off_policy_vtrace_step_matches_the_oracle(bnd, name, levels):
    w = CASES[name]
    rtol = par.rtol_of(w.precision)
    rho_bar, c_bar = levels
    an = make(bnd, w)
    an.reset(5)
    an.set(bnd.PARAMS, random_params(2, w.P, 0.15))
    an.rollout()
    g = par.gpu_traj(an, bnd, w.T)
    # the policy moves before it learns: importance ratios on both sides of the truncation levels
    theta0 = an.get(bnd.PARAMS)
    rng = np.random.default_rng(11)
    an.set(bnd.PARAMS, (theta0 + 0.03 * rng.standard_normal(theta0.size)).astype(np.float32))
    st = par.gpu_state(an, bnd)
    an.learn_vtrace(1, rho_bar, c_bar)
    # oracle: current-policy logits and values of the recorded states and of the state after the last step
    rows = np.concatenate([g["pos"], st["pos"][None, :]], axis=0)
    out = oracle_heads(w, st["theta"], st["walls"], st["goal"], rows)
    lpi = logp_of(out[:-1, :, :4], g["action"])
    ratio = np.exp(lpi.astype(np.float64) - g["logp"])
    assert (ratio > rho_bar).mean() > 0.02 and (ratio < min(rho_bar, c_bar)).mean() > 0.02  # both branches are exercised
    adv, ret = orc.vtrace(np.float32(w.gamma), rho_bar, c_bar, g["reward"], out[:, :, 4], g["done"], lpi, g["logp"])
    gadv, gret = an.get(bnd.ADV).reshape(w.T, w.B), an.get(bnd.RET).reshape(w.T, w.B)
    par.assert_close(gadv, adv, rtol, "vtrace advantages")
    par.assert_close(gret, ret, rtol, "vtrace value targets")
    # the update itself, from the library's own targets
    R = g["pos"].size
    gates = an.get(bnd.DEBUG_GATES).reshape(2, R, w.H // 32)
    ograds, oloss, rep = orc.learn(w.N, w.H, w.precision, st["theta"], st["walls"], st["goal"], g["pos"], g["action"], gadv, gret,
                                   np.float32(w.value_coef), np.float32(w.entropy_coef), gates=(gates[0], gates[1]))
    for layer, r in rep.items():
        assert r["max_abs_z"] <= 10 * rtol * r["rms_z"], (layer, r)
    ggrads = an.get(bnd.GRADS)
    for pname, sl in orc.Dims(w.N, w.H).slices().items():
        par.assert_close(ggrads[sl], ograds[sl], rtol, f"grad {pname}")
    assert int(an.get(bnd.ADAM_STEP)) == st["k"] + 1
    assert an.status() == 0


@pytest.mark.parametrize("name", list(CASES))
def test_on_policy_vtrace_is_the_a2c_step_with_lambda_one(bnd, name):
    w = CASES[name].scaled(gae_lambda=1.0)
    a, b = make(bnd, w), make(bnd, w)
    for an in (a, b):
        an.reset(8)
        an.rollout()
    a.learn()
    b.learn_vtrace(1, 1.0, 1.0)
    for which, label in ((bnd.ADV, "adv"), (bnd.RET, "ret"), (bnd.GRADS, "grads"), (bnd.ADAM_M, "m")):
        par.assert_close(b.get(which), a.get(which), par.RTOL_FP32, label)


@pytest.mark.parametrize("name", list(CASES))
def test_epochs_in_one_call_equal_single_epoch_calls(bnd, name):
    w = CASES[name].scaled(lr=0.01)
    a, b = make(bnd, w), make(bnd, w)
    for an in (a, b):
        an.reset(6)
        an.rollout()
    blobs = {n: b.get(getattr(bnd, n)) for n in TRAJ}
    a.learn_vtrace(3, 1.0, 1.0)
    for epoch in range(3):
        if epoch > 0:
            for n in TRAJ:  # pending again; its forward pass will be recomputed with the moved parameters
                b.set(getattr(bnd, n), blobs[n])
        b.learn_vtrace(1, 1.0, 1.0)
    assert np.array_equal(a.get(bnd.PARAMS), b.get(bnd.PARAMS))
    assert np.array_equal(a.get(bnd.ADV), b.get(bnd.ADV))
    # the later epochs were off-policy: their targets differ from the first epoch's
    c = make(bnd, w)
    c.reset(6)
    c.rollout()
    c.learn_vtrace(1, 1.0, 1.0)
    assert not np.array_equal(c.get(bnd.ADV), a.get(bnd.ADV))
    with pytest.raises(bnd.AnakinError):
        a.learn_vtrace(1, 1.0, 1.0)  # consumed
    assert a.status() == 0 and b.status() == 0


def test_vtrace_argument_errors_and_unsupported_path(bnd):
    an = make(bnd, CASES["mma_h64"])
    an.reset(1)
    with pytest.raises(bnd.AnakinError) as e:
        an.learn_vtrace(1, 1.0, 1.0)
    assert e.value.code == bnd.E_BAD_STATE
    an.rollout()
    for epochs, rb, cb in ((0, 1.0, 1.0), (1, -1.0, 1.0), (1, 1.0, -0.5)):
        with pytest.raises(bnd.AnakinError) as e:
            an.learn_vtrace(epochs, rb, cb)
        assert e.value.code == bnd.E_INVALID_ARG
    ff = make(bnd, Workload("ffma_h96", B=77, N=7, H=96, T=5, iters=1, episode_cap=6))
    ff.reset(1)
    ff.rollout()
    with pytest.raises(bnd.AnakinError) as e:
        ff.learn_vtrace(1, 1.0, 1.0)
    assert e.value.code == bnd.E_UNSUPPORTED_CFG
    ff.learn()  # the rollout is still pending and the generic update still works
