"""Pins for the oracle's network, sampling, GAE, loss/gradient and Adam (CPU only).

Library routines (numpy fp64 matmul, torch's bf16 cast), closed forms, finite differences and
invariants stand on the other side of every comparison.
"""
import math

import numpy as np
import pytest
import torch

from oracle import binding as orc
from paper_2104_06272_b200.workloads import random_params


def unpack(theta, N, H):
    d = orc.Dims(N, H)
    s = d.slices()
    return (theta[s["W1"]].reshape(d.D, H), theta[s["b1"]], theta[s["W2"]].reshape(H, H), theta[s["b2"]],
            theta[s["Wh"]].reshape(H, 5), theta[s["bh"]])


def numpy_forward64(theta, N, H, x):
    W1, b1, W2, b2, Wh, bh = [a.astype(np.float64) for a in unpack(theta, N, H)]
    z1 = x.astype(np.float64) @ W1 + b1
    h1 = np.maximum(z1, 0)
    z2 = h1 @ W2 + b2
    h2 = np.maximum(z2, 0)
    return h2 @ Wh + bh, z1, z2


def random_rows(seed, N, n):
    """n observation rows from n random envs in random positions (dense 0/1)."""
    walls, start, goal = orc.env_init(seed, n, N, 0.2)
    return np.stack([orc.observe(N, walls[b], int(start[b]), int(goal[b])) for b in range(n)])


# ------------------------------------------------------------------------------------------------
# parameters and network
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,H", [(5, 64), (10, 256)])
def test_param_init_bounds_variance_and_layout(N, H):
    theta = orc.param_init(9, N, H)
    d = orc.Dims(N, H)
    assert theta.size == d.P == orc.param_count(N, H)
    W1, b1, W2, b2, Wh, bh = unpack(theta, N, H)
    assert not b1.any() and not b2.any() and not bh.any()
    for w, fan_in, fan_out in ((W1, d.D, H), (W2, H, H), (Wh[:, :4], H, 4), (Wh[:, 4:], H, 1)):
        bound = math.sqrt(6.0 / (fan_in + fan_out))
        assert np.abs(w).max() <= bound
        n = w.size
        # uniform(-b, b): variance b^2/3, its sampling sd = b^2 sqrt(4/45/n); mean 0 with sd b/sqrt(3n)
        assert abs(w.astype(np.float64).var() - bound**2 / 3) < 4 * bound**2 * math.sqrt(4 / 45 / n) + 1e-9
        assert abs(w.astype(np.float64).mean()) < 4 * bound / math.sqrt(3 * n)
        assert np.abs(w).max() > 0.9 * bound if n > 200 else True


def test_param_init_draws_one_word_per_index():
    from tests.test_oracle_rng_env import philox_bigint

    N, H, seed = 5, 64, (2 << 32) | 17
    theta = orc.param_init(seed, N, H)
    d = orc.Dims(N, H)
    s = d.slices()
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for i, fan in ((0, d.D + H), (d.D * H - 1, d.D + H), (s["W2"].start + 5, 2 * H), (s["Wh"].start + 3, H + 4),
                   (s["Wh"].start + 4, H + 1), (s["Wh"].start + 9, H + 1)):
        u = (philox_bigint([i, 0, 0, 2], key)[0] >> 8) / 2**24
        assert theta[i] == np.float32((2 * u - 1) * math.sqrt(6 / fan))


@pytest.mark.parametrize("N,H", [(5, 64), (8, 128)])
def test_forward_matches_library_matmul(N, H):
    d = orc.Dims(N, H)
    theta = random_params(3, d.P, 0.2)
    x = random_rows(4, N, 64)
    out, h1, h2 = orc.forward(N, H, 0, theta, x, want_hidden=True)
    ref, z1, z2 = numpy_forward64(theta, N, H, x)
    # double accumulation with one fp32 rounding per layer: a few ulp of fp32
    assert np.allclose(out, ref, rtol=2e-6, atol=2e-6)
    assert np.allclose(h1, np.maximum(z1, 0), rtol=1e-6, atol=1e-7)
    # dense random (non one-hot) inputs exercise every weight row
    xr = np.random.default_rng(0).standard_normal((16, d.D)).astype(np.float32)
    assert np.allclose(orc.forward(N, H, 0, theta, xr), numpy_forward64(theta, N, H, xr)[0], rtol=2e-6, atol=5e-6)
    # fp64 instantiation agrees to fp64 rounding
    out64 = orc.forward_f64(N, H, theta.astype(np.float64), xr.astype(np.float64))
    assert np.allclose(out64, numpy_forward64(theta, N, H, xr)[0], rtol=1e-12, atol=1e-12)


def test_bf16_rounding_matches_torch_cast():
    rng = np.random.default_rng(2)
    a = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 10.0 ** rng.integers(-20, 20, 20000),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40], np.float32)])
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    got = orc.round_bf16(a)
    assert (got.view(np.uint32) == want.view(np.uint32)).all()


def test_bf16_forward_rounds_weights_and_hidden():
    N, H = 5, 64
    d = orc.Dims(N, H)
    theta = random_params(5, d.P, 0.2)
    x = random_rows(6, N, 32)
    out, h1, h2 = orc.forward(N, H, 1, theta, x, want_hidden=True)
    s = d.slices()
    th = theta.copy()
    for k in ("W1", "W2", "Wh"):
        th[s[k]] = orc.round_bf16(theta[s[k]])
    W1, b1, W2, b2, Wh, bh = [a.astype(np.float64) for a in unpack(th, N, H)]
    r1 = orc.round_bf16(np.maximum((x @ W1 + b1).astype(np.float32), 0))
    assert (h1 == r1).all()
    z2 = (r1.astype(np.float64) @ W2 + b2).astype(np.float32)
    r2 = orc.round_bf16(np.maximum(z2, 0))
    # an fp64-sum that lands within an fp32 ulp of a bf16 tie may round the other way: allow 1 bf16 ulp, rarely
    assert np.mean(h2 != r2) < 1e-3 and np.allclose(h2, r2, rtol=2**-7, atol=1e-30)
    assert np.allclose(out, h2.astype(np.float64) @ Wh + bh, rtol=2e-6, atol=2e-6)
    assert (orc.round_bf16(h1) == h1).all() and (orc.round_bf16(h2) == h2).all()


# ------------------------------------------------------------------------------------------------
# sampling
# ------------------------------------------------------------------------------------------------
def test_sampling_uniform_logits_closed_form():
    for c in (0.0, 3.5, -120.0):
        logits = np.full(4, c, np.float32)
        for u in [0.0, 0.1, 0.24999, 0.25, 0.49, 0.5, 0.74, 0.75, 0.999999]:
            a, logp, near = orc.sample_one(logits, u)
            assert a == int(math.floor(4 * u))
            assert abs(logp + math.log(4)) < 1e-7
            assert near == (min(abs(u - 0.25), abs(u - 0.5), abs(u - 0.75)) < 1e-5)


def test_sampling_deterministic_limits_and_ordering():
    # a dominant logit takes everything; cdf order is action 0,1,2,3
    assert orc.sample_one([50, 0, 0, 0], 0.999)[0] == 0
    assert orc.sample_one([0, 0, 0, 50], 0.001)[0] == 3
    p = np.exp([0.0, 1.0, 2.0, 3.0])
    p /= p.sum()
    cdf = np.cumsum(p)
    for u in np.linspace(0.001, 0.999, 97):
        a, logp, _ = orc.sample_one([0.0, 1.0, 2.0, 3.0], float(u))
        assert a == int(np.searchsorted(cdf[:3], u, side="right"))
        assert abs(logp - math.log(p[a])) < 1e-6


def test_sampling_frequencies_match_softmax():
    logits = np.array([0.3, -1.2, 0.9, 0.1], np.float32)
    p = np.exp(logits.astype(np.float64))
    p /= p.sum()
    T, B = 64, 1024
    act, logp, near = orc.sample_from_logits(123, 1000, np.broadcast_to(logits, (T, B, 4)).copy())
    n = T * B
    counts = np.bincount(act.ravel(), minlength=4)
    assert (np.abs(counts - n * p) < 4 * np.sqrt(n * p * (1 - p))).all()
    assert np.allclose(logp, np.log(p)[act], atol=1e-6)
    # batch sampler == single sampler fed the documented uniform
    for t, b in ((0, 0), (5, 77), (63, 1023)):
        a1, lp1, nr1 = orc.sample_one(logits, orc.act_uniform(123, b, 1000 + t))
        assert (a1, nr1) == (act[t, b], near[t, b]) and lp1 == logp[t, b]
    assert near.mean() < 5e-4  # expected about 6e-5


# ------------------------------------------------------------------------------------------------
# GAE
# ------------------------------------------------------------------------------------------------
def direct_gae(r, v, done, gamma, lam):
    """A_t = sum_l (gamma lam)^l (prod_{j<l} d_{t+j}) delta_{t+l}, written out in fp64."""
    T, B = r.shape
    r, v = r.astype(np.float64), v.astype(np.float64)
    d = 1.0 - done.astype(np.float64)
    delta = r + gamma * d * v[1:] - v[:-1]
    A = np.zeros((T, B))
    for t in range(T):
        for b in range(B):
            w = 1.0
            for l in range(T - t):
                A[t, b] += (gamma * lam) ** l * w * delta[t + l, b]
                w *= d[t + l, b]
    return A


def gae_inputs(seed, T, B, p_done=0.15):
    rng = np.random.default_rng(seed)
    r = (rng.random((T, B)) < 0.2).astype(np.float32)
    v = rng.standard_normal((T + 1, B)).astype(np.float32)
    done = (rng.random((T, B)) < p_done).astype(np.uint8)
    return r, v, done


def test_gae_matches_direct_sum():
    r, v, done = gae_inputs(0, 9, 7)
    adv, ret = orc.gae(0.99, 0.95, r, v, done)
    A = direct_gae(r, v, done, 0.99, 0.95)
    assert np.allclose(adv, A, rtol=1e-6, atol=1e-6)
    assert np.allclose(ret, A + v[:-1], rtol=1e-6, atol=1e-6)


def test_gae_special_cases():
    T, B, g = 12, 5, 0.9
    r, v, done = gae_inputs(1, T, B)
    d = 1.0 - done.astype(np.float64)
    # lambda = 0: one-step TD error
    adv, _ = orc.gae(g, 0.0, r, v, done)
    assert np.allclose(adv, r + g * d * v[1:] - v[:-1], atol=1e-6)
    # lambda = 1, no dones: discounted return-to-go plus bootstrap, minus V_t
    nod = np.zeros_like(done)
    adv, ret = orc.gae(g, 1.0, r, v, nod)
    G = np.zeros((T + 1, B))
    G[T] = v[T]
    for t in range(T - 1, -1, -1):
        G[t] = r[t] + g * G[t + 1]
    assert np.allclose(adv, G[:-1] - v[:-1], atol=1e-5) and np.allclose(ret, G[:-1], atol=1e-5)
    # every step terminal: A_t = r_t - V_t
    adv, ret = orc.gae(g, 0.95, r, v, np.ones_like(done))
    assert np.allclose(adv, r - v[:-1], atol=1e-6) and np.allclose(ret, r, atol=1e-6)
    # constant r and V, no dones: geometric series
    lam, rc, vc = 0.8, 0.5, 2.0
    adv, _ = orc.gae(g, lam, np.full((T, B), rc, np.float32), np.full((T + 1, B), vc, np.float32), nod)
    t = np.arange(T)[:, None]
    want = (rc + (g - 1) * vc) * (1 - (g * lam) ** (T - t)) / (1 - g * lam)
    assert np.allclose(adv, np.broadcast_to(want, (T, B)), rtol=1e-5)
    # a terminal step blocks everything after it
    done2 = np.zeros((T, B), np.uint8)
    done2[4] = 1
    a1, _ = orc.gae(g, 0.95, r, v, done2)
    v2 = v.copy()
    v2[6:] += 10.0
    r2 = r.copy()
    r2[5:] += 3.0
    a2, _ = orc.gae(g, 0.95, r2, v2, done2)
    assert np.allclose(a1[:5], a2[:5])


# ------------------------------------------------------------------------------------------------
# loss and gradients
# ------------------------------------------------------------------------------------------------
def tiny_batch(seed, N=5, H=16, B=4, T=3):
    walls, start, goal = orc.env_init(seed, B, N, 0.2)
    rng = np.random.default_rng(seed)
    free = [[c for c in range(N * N) if not (walls[b, c // 32] >> np.uint32(c % 32)) & 1 and c != goal[b]] for b in range(B)]
    tpos = np.array([[rng.choice(free[b]) for b in range(B)] for _ in range(T)], np.uint8)
    tact = rng.integers(0, 4, (T, B)).astype(np.int8)
    adv = rng.standard_normal((T, B))
    ret = rng.standard_normal((T, B))
    return walls, goal, tpos, tact, adv, ret


def test_entropy_of_uniform_logits_is_ln4_and_loss_terms():
    N, H = 5, 16
    walls, goal, tpos, tact, adv, ret = tiny_batch(1)
    theta = np.zeros(orc.Dims(N, H).P)  # all-zero network: logits 0, value 0
    _, loss = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, 0.5, 0.01, want_grads=False)
    assert abs(loss[3] - math.log(4)) < 1e-14
    assert abs(loss[1] - (adv.mean() * math.log(4))) < 1e-12  # -mean(A * log(1/4))
    assert abs(loss[2] - (ret**2).mean()) < 1e-12
    assert abs(loss[0] - (loss[1] + 0.5 * loss[2] - 0.01 * loss[3])) < 1e-14


def test_loss_matches_numpy_restatement():
    N, H = 5, 16
    d = orc.Dims(N, H)
    walls, goal, tpos, tact, adv, ret = tiny_batch(2)
    theta = random_params(7, d.P, 0.3).astype(np.float64)
    _, loss = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, 0.5, 0.01, want_grads=False)
    T, B = tpos.shape
    x = np.stack([orc.observe(N, walls[b], int(tpos[t, b]), int(goal[b])) for t in range(T) for b in range(B)])
    out = numpy_forward64(theta, N, H, x)[0]
    lg = torch.log_softmax(torch.from_numpy(out[:, :4]), dim=1).numpy()
    a = tact.ravel().astype(int)
    pg = -(adv.ravel() * lg[np.arange(T * B), a]).mean()
    vl = ((out[:, 4] - ret.ravel()) ** 2).mean()
    ent = -(np.exp(lg) * lg).sum(1).mean()
    assert np.allclose(loss, [pg + 0.5 * vl - 0.01 * ent, pg, vl, ent], rtol=1e-12)


def test_gradient_matches_central_finite_differences_fp64():
    N, H, c_v, c_e = 5, 16, 0.5, 0.01
    d = orc.Dims(N, H)
    # find a draw with no pre-activation near a ReLU kink (a perturbation of 1e-5 must not cross it)
    for seed in range(50):
        walls, goal, tpos, tact, adv, ret = tiny_batch(seed)
        theta = random_params(100 + seed, d.P, 0.3).astype(np.float64)
        T, B = tpos.shape
        x = np.stack([orc.observe(N, walls[b], int(tpos[t, b]), int(goal[b])) for t in range(T) for b in range(B)])
        _, z1, z2 = numpy_forward64(theta, N, H, x)
        if min(np.abs(z1).min(), np.abs(z2).min()) > 1e-3:
            break
    else:
        pytest.fail("no kink-free draw found")
    grads, loss = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, c_v, c_e)
    h = 1e-5
    rng = np.random.default_rng(0)
    s = d.slices()
    # every bias and head weight, and a random sample of the large matrices
    idx = list(range(s["b1"].start, s["b1"].stop)) + list(range(s["b2"].start, s["b2"].stop))
    idx += list(range(s["Wh"].start, s["bh"].stop))
    idx += list(rng.choice(np.arange(s["W1"].start, s["W1"].stop), 200, replace=False))
    idx += list(rng.choice(np.arange(s["W2"].start, s["W2"].stop), 150, replace=False))
    scale = np.sqrt((grads**2).mean())
    for i in idx:
        tp, tm = theta.copy(), theta.copy()
        tp[i] += h
        tm[i] -= h
        lp = orc.learn_f64(N, H, tp, walls, goal, tpos, tact, adv, ret, c_v, c_e, want_grads=False)[1][0]
        lm = orc.learn_f64(N, H, tm, walls, goal, tpos, tact, adv, ret, c_v, c_e, want_grads=False)[1][0]
        fd = (lp - lm) / (2 * h)
        assert abs(fd - grads[i]) <= 1e-6 * (abs(fd) + scale), (i, fd, grads[i])
    # W1 rows of features that are never 1 in the batch get exactly zero gradient
    W1g = grads[s["W1"]].reshape(d.D, H)
    assert not W1g[x.sum(0) == 0].any() and W1g[x.sum(0) > 0].any()


def torch_bf16(a):
    """Round to bf16 and back with torch's cast (the library routine on the other side of the pin)."""
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def numpy_backward_bf16(theta, N, H, x, h1, h2, out, act, adv, ret, c_v, c_e, round_at=("dout", "dh2", "dh1")):
    """The backward pass of the bf16 workload written out with matrix products in fp64: weights rounded to bf16, and the
    three gradient-side GEMM inputs (output gradients, dh2, dh1) rounded to bf16 where `round_at` names them.  h1, h2
    (already bf16 values) and the fp32 head outputs come from the forward pass."""
    d = orc.Dims(N, H)
    s = d.slices()
    th = theta.copy()
    for k in ("W1", "W2", "Wh"):
        th[s[k]] = torch_bf16(theta[s[k]])
    W1, b1, W2, b2, Wh, bh = [a.astype(np.float64) for a in unpack(th, N, H)]
    R = x.shape[0]
    rnd = lambda a, name: torch_bf16(a.astype(np.float32)).astype(np.float64) if name in round_at else a.astype(np.float32).astype(np.float64)
    lg = torch.log_softmax(torch.from_numpy(out[:, :4].astype(np.float64)), dim=1).numpy()
    p = np.exp(lg)
    ent = -(p * lg).sum(1)
    onehot = np.eye(4)[act]
    dz = (-adv[:, None] * (onehot - p) + c_e * p * (lg + ent[:, None])) / R
    dv = 2.0 * c_v * (out[:, 4].astype(np.float64) - ret) / R
    dOut = rnd(np.concatenate([dz, dv[:, None]], axis=1), "dout")
    g = np.zeros(d.P)
    g[s["Wh"]] = (h2.astype(np.float64).T @ dOut).ravel()
    g[s["bh"]] = dOut.sum(0)
    dh2 = rnd((dOut @ Wh.T) * (h2 > 0), "dh2")
    g[s["W2"]] = (h1.astype(np.float64).T @ dh2).ravel()
    g[s["b2"]] = dh2.sum(0)
    dh1 = rnd((dh2 @ W2.T) * (h1 > 0), "dh1")
    g[s["W1"]] = (x.astype(np.float64).T @ dh1).ravel()
    g[s["b1"]] = dh1.sum(0)
    return g


def test_bf16_backward_rounds_the_three_gemm_inputs():
    """bf16 workload: the output gradients, dh2 and dh1 enter their products rounded to bf16 (and the bias gradients
    sum the same rounded values).  The oracle's gradient equals the restatement with all three roundings, and differs
    from each restatement that leaves one of them out, so none of the three can be dropped unnoticed."""
    N, H, B, T = 5, 32, 6, 4
    d = orc.Dims(N, H)
    walls, goal, tpos, tact, adv, ret = tiny_batch(4, N=N, H=H, B=B, T=T)
    adv, ret = adv.astype(np.float32), ret.astype(np.float32)
    theta = random_params(9, d.P, 0.25)
    x = np.stack([orc.observe(N, walls[b], int(tpos[t, b]), int(goal[b])) for t in range(T) for b in range(B)])
    out, h1, h2 = orc.forward(N, H, 1, theta, x, want_hidden=True)
    grads, _ = orc.learn(N, H, 1, theta, walls, goal, tpos, tact, adv, ret, 0.5, 0.01)
    args = (theta, N, H, x, h1, h2, out, tact.ravel().astype(int), adv.ravel().astype(np.float64), ret.ravel().astype(np.float64), 0.5, 0.01)
    want = numpy_backward_bf16(*args)
    rms = np.sqrt((want**2).mean())
    # double sums in another order, fp32 storage of the result; a bf16 tie decided the other way would show as 2^-9
    assert np.abs(grads - want).max() <= 2e-6 * (np.abs(want).max() + rms)
    sl = d.slices()
    for left_out, blocks in (("dout", ("Wh", "bh")), ("dh2", ("W2", "b2")), ("dh1", ("W1", "b1"))):
        kept = tuple(r for r in ("dout", "dh2", "dh1") if r != left_out)
        other = numpy_backward_bf16(*args, round_at=kept)
        for blk in blocks:  # the blocks fed directly by the unrounded tensor move by about a bf16 ulp (2^-9 relative)
            diff = np.abs(grads[sl[blk]] - other[sl[blk]]).max()
            assert diff > 1e-4 * np.abs(want[sl[blk]]).max(), (left_out, blk, diff)


def test_gradient_structure_and_linearity_fp32():
    N, H = 5, 64
    d = orc.Dims(N, H)
    ag = orc.Agent(64, N, H, 16)
    ag.reset(3)
    ag.theta = random_params(11, d.P, 0.2)
    tr = ag.rollout()
    adv, ret = orc.gae(0.99, 0.95, tr.reward, tr.value, tr.done)
    g, loss = orc.learn(N, H, 0, ag.theta, ag.walls, ag.goal, tr.pos, tr.action, adv, ret)
    s = d.slices()
    # softmax gradients sum to zero over actions in every row => policy-bias grads sum to ~0
    assert abs(g[s["bh"]][:4].sum()) < 1e-7 * np.abs(g[s["bh"]][:4]).max() + 1e-9
    # batch mean is linear: two half-batches (envs 0..31 and 32..63) average to the whole
    ga, _ = orc.learn(N, H, 0, ag.theta, ag.walls[:32], ag.goal[:32], tr.pos[:, :32].copy(), tr.action[:, :32].copy(),
                      adv[:, :32].copy(), ret[:, :32].copy())
    gb, _ = orc.learn(N, H, 0, ag.theta, ag.walls[32:], ag.goal[32:], tr.pos[:, 32:].copy(), tr.action[:, 32:].copy(),
                      adv[:, 32:].copy(), ret[:, 32:].copy())
    assert np.allclose(0.5 * (ga + gb), g, rtol=1e-5, atol=1e-8)
    # fp32 storage agrees with the fp64 instantiation to fp32 rounding
    g64, loss64 = orc.learn_f64(N, H, ag.theta, ag.walls, ag.goal, tr.pos, tr.action, adv, ret)
    assert np.allclose(loss, loss64, rtol=1e-5)
    assert np.abs(g - g64).max() <= 1e-5 * (np.abs(g64).max())


def test_learner_forward_reproduces_recorded_logp_and_value():
    """Params do not change between acting and learning, so the update may reuse the policy's forward
    pass (Section 3.1): the recomputed log pi(a_t|s_t) and V(s_t) equal the recorded ones."""
    N, H = 5, 64
    ag = orc.Agent(32, N, H, 12)
    ag.reset(5)
    tr = ag.rollout()
    T, B = tr.pos.shape
    x = np.stack([orc.observe(N, ag.walls[b], int(tr.pos[t, b]), int(ag.goal[b])) for t in range(T) for b in range(B)])
    out = orc.forward(N, H, 0, ag.theta, x)
    assert (out[:, 4].reshape(T, B) == tr.value[:-1]).all()
    assert (out[:, :4].reshape(T, B, 4) == tr.logits).all()
    lg = torch.log_softmax(torch.from_numpy(out[:, :4].astype(np.float64)), 1).numpy()
    assert np.allclose(lg[np.arange(T * B), tr.action.ravel()], tr.logp.ravel(), atol=1e-6)
    # the loss's policy term is -mean(A * logp_recorded)
    adv, ret = orc.gae(0.99, 0.95, tr.reward, tr.value, tr.done)
    _, loss = orc.learn(N, H, 0, ag.theta, ag.walls, ag.goal, tr.pos, tr.action, adv, ret, want_grads=False)
    assert abs(loss[1] + (adv.astype(np.float64) * tr.logp).mean()) < 1e-6


def test_rollout_records_consistent_trajectory():
    N, H, T, B = 8, 32, 40, 24
    ag = orc.Agent(B, N, H, T)
    ag.reset(8)
    pos0 = ag.pos.copy()
    tr = ag.rollout()
    assert (tr.pos[0] == pos0).all() and ag.gstep == T
    # replay the recorded actions through the single-env step
    pos, tep = pos0.copy(), np.zeros(B, np.uint8)
    for t in range(T):
        for b in range(B):
            assert tr.pos[t, b] == pos[b]
            p, e, r, dn = orc.env_step(N, ag.walls[b], int(ag.start[b]), int(ag.goal[b]), 50, int(pos[b]), int(tep[b]),
                                       int(tr.action[t, b]))
            assert (r, dn) == (tr.reward[t, b], tr.done[t, b])
            pos[b], tep[b] = p, e
    assert (pos == ag.pos).all() and (tep == ag.tep).all()
    # forcing the same actions reproduces the trajectory; sampling from recorded logits reproduces the actions
    ag2 = orc.Agent(B, N, H, T)
    ag2.reset(8)
    tr2 = ag2.rollout(forced=tr.action)
    for f in ("pos", "action", "done", "reward", "value", "logp", "logits"):
        assert (getattr(tr, f) == getattr(tr2, f)).all(), f
    act, logp, near = orc.sample_from_logits(8, 0, tr.logits)
    assert (act == tr.action).all() and (logp == tr.logp).all() and (near == tr.near).all()
    # bootstrap row: value of the state after the last step
    x = np.stack([orc.observe(N, ag.walls[b], int(ag.pos[b]), int(ag.goal[b])) for b in range(B)])
    assert (orc.forward(N, H, 0, ag.theta, x)[:, 4] == tr.value[T]).all()
    # a second rollout continues the global step counter (different uniforms)
    tr3 = ag.rollout()
    assert ag.gstep == 2 * T and (tr3.pos[0] == pos).all()


# ------------------------------------------------------------------------------------------------
# Adam
# ------------------------------------------------------------------------------------------------
def test_adam_closed_forms():
    rng = np.random.default_rng(0)
    P, lr, eps = 1000, 3e-4, 1e-8
    theta0 = rng.standard_normal(P).astype(np.float32)
    g = (rng.standard_normal(P) * 10.0 ** rng.integers(-6, 2, P)).astype(np.float32)
    g[:10] = 0.0
    theta, m, v = theta0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)
    orc.adam(theta, g, m, v, 1, lr=lr, eps=eps)
    g64 = g.astype(np.float64)
    # first step: -lr * g / (|g| + eps)
    want = theta0.astype(np.float64) - lr * g64 / (np.abs(g64) + eps)
    assert np.allclose(theta, want, rtol=0, atol=1e-7 * lr + 6e-8 * np.abs(theta0).max())
    assert (theta[:10] == theta0[:10]).all()  # zero gradient leaves the parameter alone
    assert np.allclose(m, 0.1 * g64, rtol=1e-6) and np.allclose(v, 0.001 * g64**2, rtol=1e-6)
    # constant gradient: the same step every time (bias correction cancels exactly)
    th = np.zeros(P, np.float32)
    m[:] = 0
    v[:] = 0
    prev = th.copy()
    for k in range(1, 6):
        orc.adam(th, g, m, v, k, lr=lr, eps=eps)
        step = th.astype(np.float64) - prev
        assert np.allclose(step[10:], -lr * g64[10:] / (np.abs(g64[10:]) + eps), rtol=1e-3, atol=2e-10)
        prev = th.copy()


def test_adam_against_plain_loop():
    rng = np.random.default_rng(1)
    P = 64
    theta = rng.standard_normal(P).astype(np.float32)
    ref = theta.astype(np.float64)
    m, v = np.zeros(P, np.float32), np.zeros(P, np.float32)
    m64, v64 = np.zeros(P), np.zeros(P)
    for k in range(1, 8):
        g = rng.standard_normal(P).astype(np.float32)
        orc.adam(theta, g, m, v, k)
        m64 = 0.9 * m64 + 0.1 * g
        v64 = 0.999 * v64 + 0.001 * g.astype(np.float64) ** 2
        ref -= 3e-4 * (m64 / (1 - 0.9**k)) / (np.sqrt(v64 / (1 - 0.999**k)) + 1e-8)
    assert np.allclose(theta, ref, atol=1e-6) and np.allclose(m, m64, rtol=1e-5) and np.allclose(v, v64, rtol=1e-5)


def test_agent_loop_is_deterministic_and_learns_from_its_own_rollout():
    a, b = orc.Agent(64, 5, 64, 16), orc.Agent(64, 5, 64, 16)
    a.reset(1)
    b.reset(1)
    a.run(2)
    b.run(2)
    assert (a.theta == b.theta).all() and (a.pos == b.pos).all() and a.k == 2 and a.gstep == 32
    c = orc.Agent(64, 5, 64, 16)
    c.reset(2)
    c.run(2)
    assert (a.theta != c.theta).any()


def test_recorded_relu_gates_override_only_the_backward_decision():
    """Passing the oracle its own gates changes nothing and reports no mismatch; flipping one gate of a unit
    whose pre-activation is far from zero is reported and changes exactly the gradients that unit feeds."""
    N, H = 5, 32
    d = orc.Dims(N, H)
    ag = orc.Agent(16, N, H, 6)
    ag.reset(4)
    ag.theta = random_params(3, d.P, 0.3)
    tr = ag.rollout()
    adv, ret = orc.gae(0.99, 0.95, tr.reward, tr.value, tr.done)
    g0, l0 = orc.learn(N, H, 0, ag.theta, ag.walls, ag.goal, tr.pos, tr.action, adv, ret)
    T, B = tr.pos.shape
    x = np.stack([orc.observe(N, ag.walls[b], int(tr.pos[t, b]), int(ag.goal[b])) for t in range(T) for b in range(B)])
    _, h1, h2 = orc.forward(N, H, 0, ag.theta, x, want_hidden=True)
    pack = lambda h: np.packbits(h > 0, axis=1, bitorder="little").view(np.uint32)
    g1, l1, rep = orc.learn(N, H, 0, ag.theta, ag.walls, ag.goal, tr.pos, tr.action, adv, ret, gates=(pack(h1), pack(h2)))
    assert (g1 == g0).all() and (l1 == l0).all()
    assert rep["layer1"]["mismatched"] == 0 and rep["layer2"]["mismatched"] == 0 and rep["layer2"]["rms_z"] > 0
    # flip the layer-2 gate of (row 7, unit 5)
    gates2 = pack(h2).copy()
    gates2[7, 0] ^= np.uint32(1 << 5)
    g2, l2, rep2 = orc.learn(N, H, 0, ag.theta, ag.walls, ag.goal, tr.pos, tr.action, adv, ret, gates=(pack(h1), gates2))
    assert rep2["layer2"]["mismatched"] == 1 and rep2["layer1"]["mismatched"] == 0 and rep2["layer2"]["max_abs_z"] > 0
    assert (l2 == l0).all()  # the forward pass and the loss do not depend on the gates
    s = d.slices()
    changed = g2 != g0
    W2c = changed[s["W2"]].reshape(H, H)
    assert W2c[:, 5].any() and not np.delete(W2c, 5, axis=1).any()  # only column 5 of dW2
    assert not changed[s["Wh"]].any() and not changed[s["bh"]].any()  # heads see h2, not its gate


# ------------------------------------------------------------------------------------------------
# clipped-surrogate objective (PPO, Schulman et al. 2017, Eq. 7) on the same trajectory buffers
# ------------------------------------------------------------------------------------------------
def ppo_batch(seed, spread):
    """tiny_batch plus recorded log-probabilities: the current policy's, shifted by N(0, spread) so that ratios spread
    around 1."""
    N, H = 5, 16
    d = orc.Dims(N, H)
    walls, goal, tpos, tact, adv, ret = tiny_batch(seed, B=6, T=5)
    theta = random_params(200 + seed, d.P, 0.3).astype(np.float64)
    T, B = tpos.shape
    x = np.stack([orc.observe(N, walls[b], int(tpos[t, b]), int(goal[b])) for t in range(T) for b in range(B)])
    out, z1, z2 = numpy_forward64(theta, N, H, x)
    lg = torch.log_softmax(torch.from_numpy(out[:, :4]), dim=1).numpy()
    logp_now = lg[np.arange(T * B), tact.ravel().astype(int)].reshape(T, B)
    rng = np.random.default_rng(seed + 1)
    return N, H, d, walls, goal, tpos, tact, adv, ret, theta, out, lg, logp_now, logp_now - spread * rng.standard_normal((T, B)), (z1, z2)


def test_ppo_loss_matches_numpy_restatement_and_reduces_to_a2c_at_ratio_one():
    N, H, d, walls, goal, tpos, tact, adv, ret, theta, out, lg, logp_now, logp_old, _ = ppo_batch(3, 0.3)
    eps = 0.2
    _, loss = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, 0.5, 0.01, want_grads=False, logp_old=logp_old, clip=eps)
    r = np.exp(logp_now - logp_old)
    pg = -np.minimum(r * adv, np.clip(r, 1 - eps, 1 + eps) * adv).mean()
    assert (np.abs(r - 1) > eps).any() and (np.abs(r - 1) < eps).any()  # both branches are exercised
    assert abs(loss[1] - pg) < 1e-12
    # recorded log-probabilities equal to the current ones: ratio 1 everywhere, the gradient is the A2C gradient
    g_ppo, l_ppo = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, 0.5, 0.01, logp_old=logp_now, clip=eps)
    g_a2c, l_a2c = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, 0.5, 0.01)
    assert np.allclose(g_ppo, g_a2c, rtol=1e-12, atol=1e-15)
    assert abs(l_ppo[1] - (-(adv).mean())) < 1e-12  # -mean(1 * A)
    assert np.allclose(l_ppo[2:], l_a2c[2:])


def test_ppo_rows_on_the_clipped_side_carry_no_policy_gradient():
    N, H, d, walls, goal, tpos, tact, adv, ret, theta, out, lg, logp_now, _, _ = ppo_batch(4, 0.0)
    eps = 0.2
    # every row far on the clipped side: ratio 2 with positive advantage, ratio 0.5 with negative advantage
    logp_old = np.where(adv > 0, logp_now - np.log(2.0), logp_now + np.log(2.0))
    g_ppo, _ = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, 0.5, 0.01, logp_old=logp_old, clip=eps)
    g_zero, _ = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, np.zeros_like(adv), ret, 0.5, 0.01)
    assert np.allclose(g_ppo, g_zero, rtol=1e-12, atol=1e-15)  # only the value and entropy terms are left
    # the other side (ratio 2 with negative advantage) is NOT clipped: gradient = A2C gradient scaled by the ratio
    logp_old2 = np.where(adv > 0, logp_now + np.log(2.0), logp_now - np.log(2.0))
    g2, _ = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, 0.5, 0.01, logp_old=logp_old2, clip=eps)
    r = np.exp(logp_now - logp_old2)
    g_scaled, _ = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv * r, ret, 0.5, 0.01)
    assert np.allclose(g2, g_scaled, rtol=1e-10, atol=1e-14)


def test_ppo_gradient_matches_central_finite_differences_fp64():
    eps, c_v, c_e = 0.2, 0.5, 0.01
    for seed in range(60):  # a draw with no ReLU kink and no ratio near a clip boundary
        N, H, d, walls, goal, tpos, tact, adv, ret, theta, out, lg, logp_now, logp_old, (z1, z2) = ppo_batch(seed, 0.3)
        r = np.exp(logp_now - logp_old)
        if min(np.abs(z1).min(), np.abs(z2).min()) > 1e-3 and np.abs(np.abs(r - 1) - eps).min() > 1e-3:
            break
    else:
        pytest.fail("no kink-free draw found")
    grads, _ = orc.learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, c_v, c_e, logp_old=logp_old, clip=eps)
    s = d.slices()
    rng = np.random.default_rng(1)
    idx = list(range(s["b2"].start, s["b2"].stop)) + list(range(s["Wh"].start, s["bh"].stop))
    idx += list(rng.choice(np.arange(s["W1"].start, s["W1"].stop), 100, replace=False))
    idx += list(rng.choice(np.arange(s["W2"].start, s["W2"].stop), 100, replace=False))
    h, scale = 1e-5, np.sqrt((grads**2).mean())
    for i in idx:
        tp, tm = theta.copy(), theta.copy()
        tp[i] += h
        tm[i] -= h
        lp = orc.learn_f64(N, H, tp, walls, goal, tpos, tact, adv, ret, c_v, c_e, want_grads=False, logp_old=logp_old, clip=eps)[1][0]
        lm = orc.learn_f64(N, H, tm, walls, goal, tpos, tact, adv, ret, c_v, c_e, want_grads=False, logp_old=logp_old, clip=eps)[1][0]
        fd = (lp - lm) / (2 * h)
        assert abs(fd - grads[i]) <= 1e-6 * (abs(fd) + scale), (i, fd, grads[i])


def test_agent_ppo_first_epoch_is_the_a2c_step():
    """The recorded log-probabilities are the policy's own at rollout time, so epoch 1 has ratio 1 everywhere."""
    a, b = orc.Agent(32, 5, 32, 8), orc.Agent(32, 5, 32, 8)
    for ag in (a, b):
        ag.reset(9)
        ag.rollout()
    a.learn()
    b.learn_ppo(1, 0.2)
    assert np.allclose(a.grads, b.grads, rtol=2e-5, atol=1e-9)  # exp(logp - logp) = 1 up to the fp32 record of logp
    c = orc.Agent(32, 5, 32, 8)
    c.reset(9)
    c.rollout()
    c.learn_ppo(3, 0.2)
    assert c.k == 3 and not np.allclose(c.theta, b.theta)
