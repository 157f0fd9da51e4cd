"""Helpers for the GPU-vs-oracle parity tests: the tolerance metric and the staged, teacher-forced
comparison of one act+learn iteration."""
from __future__ import annotations

import numpy as np

from oracle import binding as orc

RTOL_FP32 = 1e-4
RTOL_BF16 = 2e-2
MARGINS: dict = {}  # name of the last compared tensors -> worst |error| / bound (printed by the full-size tests)


def rtol_of(prec: int) -> float:
    return RTOL_BF16 if prec == 1 else RTOL_FP32


def assert_close(got, want, rtol, name):
    """Per tensor: |g - o| <= rtol * (|o| + rms(o)) for every element (a purely element-wise relative
    error is meaningless at zero crossings)."""
    got = np.asarray(got, dtype=np.float64).ravel()
    want = np.asarray(want, dtype=np.float64).ravel()
    assert got.shape == want.shape, (name, got.shape, want.shape)
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    rms = np.sqrt((want**2).mean()) if want.size else 0.0
    err = np.abs(got - want)
    bound = rtol * (np.abs(want) + rms)
    bad = err > bound
    if want.size:
        MARGINS[name] = float((err / np.maximum(bound, 1e-300)).max())  # worst error as a fraction of its bound
    if bad.any():
        i = int(np.argmax(err - bound))
        raise AssertionError(f"{name}: {int(bad.sum())}/{got.size} outside rtol={rtol}; worst at {i}: got {got[i]!r} "
                             f"want {want[i]!r} (rms {rms:.3e})")


def gpu_state(an, bnd):
    """Host copies of everything the oracle needs to shadow the library."""
    return dict(theta=an.get(bnd.PARAMS), m=an.get(bnd.ADAM_M), v=an.get(bnd.ADAM_V), k=int(an.get(bnd.ADAM_STEP)),
                walls=an.get(bnd.ENV_WALLS).reshape(an.B, -1), start=an.get(bnd.ENV_START), goal=an.get(bnd.ENV_GOAL),
                pos=an.get(bnd.ENV_POS), tep=an.get(bnd.ENV_TEP), gstep=int(an.get(bnd.GLOBAL_STEP)))


def gpu_traj(an, bnd, T):
    B = an.B
    return dict(pos=an.get(bnd.TRAJ_POS).reshape(T, B), action=an.get(bnd.TRAJ_ACTION).reshape(T, B),
                done=an.get(bnd.TRAJ_DONE).reshape(T, B), reward=an.get(bnd.TRAJ_REWARD).reshape(T, B),
                value=an.get(bnd.TRAJ_VALUE).reshape(T + 1, B), logp=an.get(bnd.TRAJ_LOGP).reshape(T, B),
                logits=an.get(bnd.DEBUG_LOGITS).reshape(T, B, 4))


def check_rollout(an, bnd, w, seed, st, T, forced=None, envs=None):
    """Stage 1+2: acts on the GPU, then the oracle replays the GPU's action sequence from the same
    state.  Transitions are bit-exact; logits/values/logp within tolerance; the GPU's actions equal the
    oracle's samples from the GPU's own logits except where the uniform is within 1e-5 of a CDF
    boundary.  `envs` restricts the oracle's replay to a subset of env indices (full-size workloads)."""
    if forced is None:
        an.rollout(T)
    else:
        import torch

        an.rollout_forced(torch.from_numpy(forced).cuda())
    g = gpu_traj(an, bnd, T)
    assert an.status() == 0
    assert int(an.get(bnd.GLOBAL_STEP)) == st["gstep"] + T
    counts = compare_rollout(w, seed, st, g, T, an.get(bnd.ENV_POS), an.get(bnd.ENV_TEP), forced=forced, envs=envs)
    return g, counts


def compare_rollout(w, seed, st, g, T, final_pos, final_tep, forced=None, envs=None, env0=0):
    """The comparisons of check_rollout on arrays already read from the library: st = state before the rollout, g = the
    recorded trajectory, final_pos / final_tep = env state after it.  env0 = global index of the batch's first env."""
    rtol = rtol_of(w.precision)
    B = g["pos"].shape[1]
    sel = np.arange(B) if envs is None else np.asarray(envs)
    pos, tep = st["pos"][sel].copy(), st["tep"][sel].copy()
    tr = orc.rollout(w.N, w.H, w.precision, T, w.episode_cap, st["theta"], np.ascontiguousarray(st["walls"][sel]),
                     st["start"][sel].copy(), st["goal"][sel].copy(), pos, tep, seed, st["gstep"],
                     forced=np.ascontiguousarray(g["action"][:, sel]), kind=w.env_kind)
    if forced is not None:
        assert (g["action"] == forced).all()
    assert (g["pos"][:, sel] == tr.pos).all(), "recorded positions differ"
    assert (g["reward"][:, sel] == tr.reward).all(), "rewards differ"
    assert (g["done"][:, sel] == tr.done).all(), "done flags differ"
    assert (final_pos[sel] == pos).all() and (final_tep[sel] == tep).all(), "final env state differs"
    assert_close(g["logits"][:, sel], tr.logits, rtol, "logits")
    assert_close(g["value"][:, sel], tr.value, rtol, "values")
    assert_close(g["logp"][:, sel], tr.logp, rtol, "logp")
    n_near = n_mis = 0
    if forced is None:
        # sample from the GPU's own logits with the same uniforms
        if envs is None and env0 == 0:
            act, logp, near = orc.sample_from_logits(seed, st["gstep"], g["logits"])
        else:
            act = np.zeros((T, len(sel)), np.int8)
            logp = np.zeros((T, len(sel)), np.float32)
            near = np.zeros((T, len(sel)), np.uint8)
            for t in range(T):
                for j, b in enumerate(sel):
                    a, lp, nr = orc.sample_one(g["logits"][t, b], orc.act_uniform(seed, env0 + int(b), st["gstep"] + t))
                    act[t, j], logp[t, j], near[t, j] = a, lp, nr
        mism = act != g["action"][:, sel]
        n_near, n_mis = int(near.sum()), int(mism.sum())
        assert not (mism & (near == 0)).any(), "an action differs away from any CDF boundary"
        assert n_mis <= max(1, int(1e-4 * mism.size)), f"{n_mis} action mismatches in {mism.size} samples"
        ok = ~mism
        assert_close(g["logp"][:, sel][ok], logp[ok], 1e-4 if w.precision == 0 else 1e-4, "logp of sampled action")
    return dict(near=n_near, mismatched=n_mis)


def check_gae(an, bnd, w, g, T):
    an.gae()
    adv, ret = orc.gae(np.float32(w.gamma), np.float32(w.gae_lambda), g["reward"], g["value"], g["done"])
    gadv, gret = an.get(bnd.ADV).reshape(T, an.B), an.get(bnd.RET).reshape(T, an.B)
    assert_close(gadv, adv, RTOL_FP32, "advantages")
    assert_close(gret, ret, RTOL_FP32, "returns")
    return gadv, gret


def check_learn(an, bnd, w, st, g, gadv, gret):
    """Stage 4: the oracle learns from the GPU's trajectory, advantages/returns and pre-update
    parameters.  Gradients and loss terms are compared directly; Adam is compared on the GPU's own
    gradient (its early steps are close to lr*sign(g), which would otherwise turn a 1e-7 gradient
    difference on a near-zero element into a full-size parameter difference)."""
    an.learn()
    R = g["pos"].size
    gates = an.get(bnd.DEBUG_GATES).reshape(2, R, w.H // 32)
    s = an.stats()
    new = dict(k=int(an.get(bnd.ADAM_STEP)), m=an.get(bnd.ADAM_M), v=an.get(bnd.ADAM_V), theta=an.get(bnd.PARAMS))
    return compare_learn(w, st, g, gadv, gret, an.get(bnd.GRADS), gates, [s.loss_total, s.loss_pg, s.loss_value, s.entropy], new)


def compare_learn(w, st, g, gadv, gret, ggrads, gates, gloss, new):
    """The comparisons of check_learn on arrays already read from the library: ggrads = GRADS, gates = the recorded ReLU
    gates [2][R][H/32], gloss = (total, pg, value, entropy), new = Adam step count, moments and parameters after it."""
    rtol = rtol_of(w.precision)
    # ReLU gates are floating-point decisions: the oracle's backward pass takes them as the library recorded
    # them (the kernel's precision), and reports where they differ from its own
    R = g["pos"].size
    ograds, oloss, rep = orc.learn(w.N, w.H, w.precision, st["theta"], st["walls"], st["goal"], g["pos"], g["action"], gadv,
                                   gret, np.float32(w.value_coef), np.float32(w.entropy_coef), gates=(gates[0], gates[1]))
    for layer, r in rep.items():
        # a gate may differ only where the pre-activation is within rounding of zero, and only rarely: fp32 and fp64 sums
        # of O(1) terms differ by ~1e-7, so about 1e-7 of the gates can fall on the other side; 1e-5 of them (plus a floor
        # for tiny cases) leaves two orders of margin and is far below one CTA tile of mis-gated units on any workload
        assert r["max_abs_z"] <= 10 * rtol * r["rms_z"], (layer, r)
        assert r["mismatched"] <= 10 + 1e-5 * R * w.H, (layer, r)
    print(f"{w.name}: gate decisions differing from the oracle's own: layer1 {rep['layer1']['mismatched']}, "
          f"layer2 {rep['layer2']['mismatched']} of {R * w.H} each")
    d = orc.Dims(w.N, w.H)
    for name, sl in d.slices().items():
        assert_close(ggrads[sl], ograds[sl], rtol, f"grad {name}")
    gl = np.array(gloss, dtype=np.float64)
    lt = max(rtol, 1e-4)
    scale = np.abs(oloss).max()
    assert (np.abs(gl - oloss) <= lt * (np.abs(oloss) + 1e-3 * scale) + 1e-7).all(), (gl, oloss)
    theta, m, v = st["theta"].copy(), st["m"].copy(), st["v"].copy()
    orc.adam(theta, ggrads, m, v, st["k"] + 1, np.float32(w.lr), np.float32(w.adam_b1), np.float32(w.adam_b2),
             np.float32(w.adam_eps))
    assert new["k"] == st["k"] + 1
    assert_close(new["m"], m, RTOL_FP32, "adam m")
    assert_close(new["v"], v, RTOL_FP32, "adam v")
    gtheta = new["theta"]
    assert_close(gtheta, theta, RTOL_FP32, "updated params")
    # The step is only observable through the fp32 parameter it was added to: one unit in the last place of theta
    # (which can exceed rtol * step for a large weight with a small step) is rounding of the storage format, not error.
    gstep = gtheta.astype(np.float64) - st["theta"]
    ostep = theta.astype(np.float64) - st["theta"]
    bound = RTOL_FP32 * (np.abs(ostep) + np.sqrt((ostep**2).mean())) + np.spacing(np.abs(theta).astype(np.float32))
    bad = np.abs(gstep - ostep) > bound
    assert not bad.any(), f"param step: {int(bad.sum())}/{bad.size} outside tolerance; first at {int(np.argmax(bad))}"
    return ograds, oloss, rep


def check_iteration(an, bnd, w, seed, T=None):
    T = w.T if T is None else T
    st = gpu_state(an, bnd)
    g, counts = check_rollout(an, bnd, w, seed, st, T)
    gadv, gret = check_gae(an, bnd, w, g, T)
    rep = check_learn(an, bnd, w, st, g, gadv, gret)[2]
    counts["gate_mismatches"] = (rep["layer1"]["mismatched"], rep["layer2"]["mismatched"])
    return counts
