"""Pins of the oracle's V-trace targets (CPU only).

V-trace (Espeholt et al. 2018, IMPALA, Eq. 1) is the off-policy correction the Podracer paper's other agent uses
(Section 3.2); here it is one more objective over the trajectory buffers of the Anakin loop.  The oracle's reverse scan
is pinned against the definition written out as a direct sum, against the cases where it reduces to other estimators,
and against the truncation limits.
"""
import numpy as np

from oracle import binding as orc


def inputs(seed, T, B, p_done=0.15, spread=0.7):
    rng = np.random.default_rng(seed)
    r = (rng.random((T, B)) < 0.2).astype(np.float32)
    v = rng.standard_normal((T + 1, B)).astype(np.float32)
    done = (rng.random((T, B)) < p_done).astype(np.uint8)
    lmu = -np.abs(rng.standard_normal((T, B))).astype(np.float32) - 0.1
    lpi = (lmu + spread * rng.standard_normal((T, B))).astype(np.float32)
    return r, v, done, lpi, lmu


def direct_vtrace(r, v, done, lpi, lmu, gamma, rho_bar, c_bar):
    """The definition, term by term in fp64:  v_s = V_s + sum_{t>=s} gamma^(t-s) (prod_{i=s}^{t-1} d_i c_i) rho_t
    (r_t + gamma d_t V_{t+1} - V_t);  adv_s = rho_s (r_s + gamma d_s v_{s+1} - V_s) with v_T = V_T."""
    T, B = r.shape
    r, v = r.astype(np.float64), v.astype(np.float64)
    d = 1.0 - done.astype(np.float64)
    w = np.exp(lpi.astype(np.float64) - lmu.astype(np.float64))
    rho, c = np.minimum(rho_bar, w), np.minimum(c_bar, w)
    vs = np.zeros((T + 1, B))
    vs[T] = v[T]
    for s in range(T):
        for b in range(B):
            acc, prod = 0.0, 1.0
            for t in range(s, T):
                acc += gamma ** (t - s) * prod * rho[t, b] * (r[t, b] + gamma * d[t, b] * v[t + 1, b] - v[t, b])
                prod *= d[t, b] * c[t, b]
            vs[s, b] = v[s, b] + acc
    adv = rho * (r + gamma * d * vs[1:] - v[:-1])
    return adv, vs[:-1]


def test_vtrace_matches_the_definition_as_a_direct_sum():
    for seed, (rb, cb) in enumerate([(1.0, 1.0), (2.0, 0.7), (0.5, 1.5)]):
        r, v, done, lpi, lmu = inputs(seed, 9, 6)
        adv, ret = orc.vtrace(0.97, rb, cb, r, v, done, lpi, lmu)
        A, V = direct_vtrace(r, v, done, lpi, lmu, 0.97, rb, cb)
        assert np.allclose(adv, A, rtol=1e-6, atol=1e-6)
        assert np.allclose(ret, V, rtol=1e-6, atol=1e-6)


def test_on_policy_vtrace_is_gae_with_lambda_one():
    """pi = mu and truncation levels >= 1: every weight is 1, the target is the bootstrapped n-step return (IMPALA,
    Section 4.1), i.e. GAE's return at lambda = 1, and the advantage is GAE's."""
    r, v, done, lpi, _ = inputs(3, 14, 5)
    adv, ret = orc.vtrace(0.99, 1.0, 1.0, r, v, done, lpi, lpi)
    a1, r1 = orc.gae(0.99, 1.0, r, v, done)
    assert np.allclose(adv, a1, rtol=1e-6, atol=1e-6) and np.allclose(ret, r1, rtol=1e-6, atol=1e-6)
    adv2, ret2 = orc.vtrace(0.99, 3.0, 2.0, r, v, done, lpi, lpi)  # larger truncation levels change nothing on-policy
    assert (adv2 == adv).all() and (ret2 == ret).all()


def test_zero_trace_gives_the_one_step_target():
    """c_bar = 0: no trace; v_s = V_s + rho_s (r_s + gamma d_s V_{s+1} - V_s)."""
    g = 0.9
    r, v, done, lpi, lmu = inputs(4, 10, 4)
    adv, ret = orc.vtrace(g, 1.0, 0.0, r, v, done, lpi, lmu)
    d = 1.0 - done.astype(np.float64)
    rho = np.minimum(1.0, np.exp(lpi.astype(np.float64) - lmu))
    td = r + g * d * v[1:].astype(np.float64) - v[:-1]
    assert np.allclose(ret, v[:-1] + rho * td, rtol=1e-6, atol=1e-6)
    vs = np.concatenate([v[:-1] + rho * td, v[-1:].astype(np.float64)], axis=0)
    assert np.allclose(adv, rho * (r + g * d * vs[1:] - v[:-1]), rtol=1e-6, atol=1e-6)


def test_zero_rho_leaves_the_value_and_kills_the_advantage():
    r, v, done, lpi, lmu = inputs(5, 8, 3)
    adv, ret = orc.vtrace(0.99, 0.0, 1.0, r, v, done, lpi, lmu)
    assert (adv == 0).all() and np.allclose(ret, v[:-1], atol=0)


def test_truncation_only_binds_above_the_level():
    """Ratios all below both levels: the weights are the plain importance ratios, and raising the levels changes
    nothing; ratios all above: the weights are the levels themselves, whatever the ratios."""
    T, B = 7, 4
    r, v, done, _, lmu = inputs(6, T, B)
    lo = (lmu - 0.5).astype(np.float32)  # ratio exp(-0.5) < 1
    a, b = orc.vtrace(0.95, 1.0, 1.0, r, v, done, lo, lmu), orc.vtrace(0.95, 9.0, 9.0, r, v, done, lo, lmu)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all()
    hi1, hi2 = (lmu + 1.0).astype(np.float32), (lmu + 2.5).astype(np.float32)  # ratios e and e^2.5 > 1
    a, b = orc.vtrace(0.95, 1.0, 1.0, r, v, done, hi1, lmu), orc.vtrace(0.95, 1.0, 1.0, r, v, done, hi2, lmu)
    assert np.allclose(a[0], b[0], atol=1e-7) and np.allclose(a[1], b[1], atol=1e-7)
    on = orc.vtrace(0.95, 1.0, 1.0, r, v, done, lmu, lmu)  # ... and equal to the on-policy targets
    assert np.allclose(a[0], on[0], atol=1e-7) and np.allclose(a[1], on[1], atol=1e-7)


def test_an_episode_end_blocks_the_future():
    T, B = 10, 3
    r, v, done, lpi, lmu = inputs(7, T, B, p_done=0.0)
    done[4] = 1
    a1, r1 = orc.vtrace(0.99, 1.0, 1.0, r, v, done, lpi, lmu)
    r2, v2 = r.copy(), v.copy()
    r2[5:] += 3.0
    v2[5:] -= 2.0
    a2, q2 = orc.vtrace(0.99, 1.0, 1.0, r2, v2, done, lpi, lmu)
    assert (a1[:5] == a2[:5]).all() and (r1[:5] == q2[:5]).all()
