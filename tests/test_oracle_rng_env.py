"""Pins for the oracle's random numbers, environment and observation (CPU only).

Each check ties the oracle to something other than itself: a library generator, an independent
big-integer restatement of the published algorithm, statistics, brute force, or a hand-traced example.
"""
import ctypes
import ctypes.util
import math
import os

import numpy as np
import pytest

from oracle import binding as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------------------------------------
# Philox4x32-10
# ------------------------------------------------------------------------------------------------
def philox_bigint(ctr, key):
    """Independent restatement with Python integers (Salmon et al., SC'11: the Philox-4x32 round is a
    pair of 32x32->64 multiplies whose halves are permuted and xored with neighbours and key)."""
    c = [int(v) for v in ctr]
    k = [int(v) for v in key]
    mask = (1 << 32) - 1
    for _ in range(10):
        prod_a = 0xD2511F53 * c[0]
        prod_b = 0xCD9E8D57 * c[2]
        c = [((prod_b >> 32) ^ c[1] ^ k[0]) & mask, prod_b & mask, ((prod_a >> 32) ^ c[3] ^ k[1]) & mask, prod_a & mask]
        k = [(k[0] + 0x9E3779B9) & mask, (k[1] + 0xBB67AE85) & mask]
    return c


def test_philox_matches_bigint_restatement():
    rng = np.random.default_rng(0)
    for _ in range(2000):
        ctr = rng.integers(0, 2**32, size=4, dtype=np.uint64).astype(np.uint32)
        key = rng.integers(0, 2**32, size=2, dtype=np.uint64).astype(np.uint32)
        assert list(orc.philox4x32_10(ctr, key)) == philox_bigint(ctr, key)
    # extreme words
    for ctr, key in (([0] * 4, [0] * 2), ([0xFFFFFFFF] * 4, [0xFFFFFFFF] * 2)):
        assert list(orc.philox4x32_10(ctr, key)) == philox_bigint(ctr, key)


def _curand():
    for name in ("libcurand.so", "libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so"):
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    return None


def test_philox_matches_curand_host_generator():
    """cuRAND's HOST Philox4_32_10 generator (it runs on the CPU) is an independent library
    implementation.  Observed layout of its output stream at offset 0 under seed s: the j-th group of
    four 32-bit outputs is the Philox block with key (s_lo, s_hi) and counter (j // 65536, 0, j % 65536, 0)."""
    lib = _curand()
    if lib is None:
        pytest.skip("libcurand not found")
    CURAND_RNG_PSEUDO_PHILOX4_32_10 = 161
    gen = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), CURAND_RNG_PSEUDO_PHILOX4_32_10) != 0:
        pytest.skip("cuRAND host generator unavailable")
    try:
        rng = np.random.default_rng(1)
        seeds = [0, 1, 0xFFFFFFFFFFFFFFFF] + [int(rng.integers(0, 2**63)) * 2 + int(rng.integers(0, 2)) for _ in range(5)]
        nblk = 2 * 65536 + 16
        for seed in seeds:
            assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
            assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(0)) == 0
            out = np.zeros(4 * nblk, dtype=np.uint32)
            assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(out.size)) == 0
            key = [seed & 0xFFFFFFFF, seed >> 32]
            blocks = list(range(0, 40)) + [65535, 65536, 65537, 2 * 65536 + 3] + [int(b) for b in rng.integers(0, nblk, 60)]
            for j in blocks:
                mine = orc.philox4x32_10([j // 65536, 0, j % 65536, 0], key)
                assert [int(x) for x in mine] == [int(x) for x in out[4 * j:4 * j + 4]], (seed, j)
    finally:
        lib.curandDestroyGenerator(gen)


def test_uniform_is_top_24_bits():
    assert orc.uniform24(0) == 0.0
    assert orc.uniform24(0xFFFFFFFF) == (2**24 - 1) / 2**24
    assert orc.uniform24(0x80000000) == 0.5
    assert orc.uniform24(0x000000FF) == 0.0  # low 8 bits are dropped


def test_action_uniform_statistics():
    """ACT-stream uniforms over 2^16 (env, step) pairs: mean, variance and a 16-bin chi-square."""
    n_b, n_g = 256, 256
    u = np.array([[orc.act_uniform(7, b, g) for g in range(n_g)] for b in range(n_b)]).ravel()
    n = u.size
    assert (u >= 0).all() and (u < 1).all()
    assert abs(u.mean() - 0.5) < 4 * math.sqrt(1 / 12 / n)
    assert abs(u.var() - 1 / 12) < 4 * math.sqrt(1 / 180 / n)
    counts = np.histogram(u, bins=16, range=(0, 1))[0]
    chi2 = ((counts - n / 16) ** 2 / (n / 16)).sum()
    assert chi2 < 45.0  # 15 dof: P(chi2 > 45) < 1e-4
    # the draw is word 0 of counter (b, g, 0, stream 3) under key (seed_lo, seed_hi)
    assert orc.act_uniform(7, 5, 9) == (philox_bigint([5, 9, 0, 3], [7, 0])[0] >> 8) / 2**24
    assert orc.act_uniform((3 << 32) | 7, 5, 9) == (philox_bigint([5, 9, 0, 3], [7, 3])[0] >> 8) / 2**24


# ------------------------------------------------------------------------------------------------
# Environment generation
# ------------------------------------------------------------------------------------------------
def unpack_walls(walls, C):
    B = walls.shape[0]
    bits = np.zeros((B, C), dtype=bool)
    for c in range(C):
        bits[:, c] = (walls[:, c // 32] >> np.uint32(c % 32)) & 1
    return bits


@pytest.mark.parametrize("N", [5, 8, 10, 16])
def test_env_init_invariants(N):
    B, C = 4096, N * N
    walls, start, goal = orc.env_init(11, B, N, 0.2)
    bits = unpack_walls(walls, C)
    assert (start < C).all() and (goal < C).all()
    assert (start != goal).all()
    idx = np.arange(B)
    assert not bits[idx, start].any() and not bits[idx, goal].any()
    # no stray bits above cell C-1
    if C % 32:
        assert ((walls[:, -1] >> np.uint32(C % 32)) == 0).all()
    # wall count ~ Binomial(B(C-2), 0.2)
    n = B * (C - 2)
    assert abs(bits.sum() - 0.2 * n) < 4 * math.sqrt(n * 0.2 * 0.8)
    # start and goal are uniform over cells: chi-square on start, and on goal
    for arr in (start, goal):
        counts = np.bincount(arr, minlength=C)
        chi2 = ((counts - B / C) ** 2 / (B / C)).sum()
        assert chi2 < (C - 1) + 6 * math.sqrt(2 * (C - 1))


def test_env_init_follows_the_stated_draws():
    """Rebuild env b from the written rule with the big-integer Philox and compare bit for bit."""
    seed, B, N = (5 << 32) | 99, 37, 10
    C = N * N
    walls, start, goal = orc.env_init(seed, B, N, 0.2)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    thr = math.floor(0.2 * 2**32)
    assert thr == 858993459
    bits = unpack_walls(walls, C)
    for b in range(B):
        x = philox_bigint([b, 0, 0, 1], key)
        s = (x[0] * C) >> 32
        g = (x[1] * (C - 1)) >> 32
        g += g >= s
        assert (s, g) == (start[b], goal[b])
        for c in range(C):
            y = philox_bigint([b, 1 + c // 4, 0, 1], key)
            want = (y[c % 4] < thr) and c != s and c != g
            assert bool(bits[b, c]) == want


def test_env_init_is_prefix_stable_and_seed_sensitive():
    w1, s1, g1 = orc.env_init(3, 64, 8, 0.2)
    w2, s2, g2 = orc.env_init(3, 128, 8, 0.2)
    assert (w1 == w2[:64]).all() and (s1 == s2[:64]).all() and (g1 == g2[:64]).all()
    w3, _, _ = orc.env_init(4, 64, 8, 0.2)
    assert (w1 != w3).any()


# ------------------------------------------------------------------------------------------------
# Environment step
# ------------------------------------------------------------------------------------------------
def load_trace(path):
    walls_cells, steps, meta = [], [], {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if not line:
            continue
        tok = line.split()
        if tok[0] == "walls":
            walls_cells = [int(t) for t in tok[1:]]
        elif tok[0] == "step":
            steps.append([int(t) for t in tok[1:]])
        else:
            meta[tok[0]] = int(tok[1])
    return walls_cells, steps, meta


def test_env_step_hand_traced_episode():
    cells, steps, meta = load_trace(os.path.join(GOLDEN, "gridworld_trace_5x5.txt"))
    w = np.zeros(1, np.uint32)
    for c in cells:
        w[0] |= np.uint32(1 << c)
    pos, tep = meta["start"], 0
    for a, p0, t0, p1, t1, r, dn in steps:
        assert (pos, tep) == (p0, t0)
        pos, tep, rew, done = orc.env_step(5, w, meta["start"], meta["goal"], meta["cap"], pos, tep, a)
        assert (pos, tep, rew, done) == (p1, t1, float(r), dn)


def bfs_reachable(bits_b, N, start):
    seen = {int(start)}
    todo = [int(start)]
    while todo:
        p = todo.pop()
        r, c = divmod(p, N)
        for nr, nc in ((r - 1, c), (r, c + 1), (r + 1, c), (r, c - 1)):
            if 0 <= nr < N and 0 <= nc < N:
                q = nr * N + nc
                if not bits_b[q] and q not in seen:
                    seen.add(q)
                    todo.append(q)
    return seen


@pytest.mark.parametrize("N", [5, 8])
def test_env_step_invariants_under_random_actions(N):
    B, steps, cap = 48, 400, 50
    C = N * N
    walls, start, goal = orc.env_init(21, B, N, 0.2)
    bits = unpack_walls(walls, C)
    rng = np.random.default_rng(5)
    for b in range(B):
        reach = bfs_reachable(bits[b], N, start[b])
        pos, tep = int(start[b]), 0
        since_reset = 0
        for _ in range(steps):
            a = int(rng.integers(0, 4))
            r0, c0 = divmod(pos, N)
            npos, ntep, rew, done = orc.env_step(N, walls[b], int(start[b]), int(goal[b]), cap, pos, tep, a)
            since_reset += 1
            # where the rule says the agent lands before any reset
            tr, tc = [(r0 - 1, c0), (r0, c0 + 1), (r0 + 1, c0), (r0, c0 - 1)][a]
            land = pos
            if 0 <= tr < N and 0 <= tc < N and not bits[b, tr * N + tc]:
                land = tr * N + tc
            assert rew in (0.0, 1.0)
            assert (rew == 1.0) == (land == goal[b])  # +1 only on reaching the goal
            if land == goal[b] or since_reset >= cap:
                assert done == 1 and npos == start[b] and ntep == 0
                since_reset = 0
            else:
                assert done == 0 and npos == land and ntep == since_reset
            assert not bits[b, npos]  # never on a wall
            assert npos in reach  # never leaves the component of the start cell
            assert ntep < cap
            pos, tep = npos, ntep


def test_env_timeout_after_exactly_cap_steps():
    # an agent boxed in by walls can never reach the goal: done fires at steps cap, 2cap, ...
    N, cap = 5, 50
    w = np.zeros(1, np.uint32)
    for c in (1, 5):  # start = cell 0 (corner), walls right and below
        w[0] |= np.uint32(1 << c)
    pos, tep = 0, 0
    dones = []
    for i in range(1, 121):
        pos, tep, rew, done = orc.env_step(N, w, 0, 24, cap, pos, tep, i % 4)
        assert rew == 0.0 and pos == 0
        if done:
            dones.append(i)
    assert dones == [50, 100]


# ------------------------------------------------------------------------------------------------
# Observation
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N", [5, 10, 16])
def test_observation_planes(N):
    C = N * N
    walls, start, goal = orc.env_init(2, 16, N, 0.2)
    bits = unpack_walls(walls, C)
    for b in range(16):
        x = orc.observe(N, walls[b], int(start[b]), int(goal[b]))
        assert x.shape == (3 * C,) and set(np.unique(x)) <= {0.0, 1.0}
        assert x.sum() == bits[b].sum() + 2
        assert (x[:C] == bits[b]).all()
        assert x[C:2 * C].argmax() == start[b] and x[C:2 * C].sum() == 1
        assert x[2 * C:].argmax() == goal[b] and x[2 * C:].sum() == 1


# ---- second env ("torus": a move off an edge re-enters at the opposite edge; walls still block) ----
def test_torus_step_hand_traced_episode():
    cells, steps, meta = load_trace(os.path.join(GOLDEN, "torus_trace_5x5.txt"))
    w = np.zeros(1, np.uint32)
    for c in cells:
        w[0] |= np.uint32(1 << c)
    pos, tep = meta["start"], 0
    for a, p0, t0, p1, t1, r, dn in steps:
        assert (pos, tep) == (p0, t0)
        pos, tep, rew, done = orc.env_step(5, w, meta["start"], meta["goal"], meta["cap"], pos, tep, a, orc.TORUS)
        assert (pos, tep, rew, done) == (p1, t1, float(r), dn)


def test_torus_without_walls_is_addition_modulo_n():
    """Closed form: on an empty board the position after any action sequence is start + sum of displacements, each
    coordinate modulo N (until the goal is entered)."""
    N, cap = 7, 255
    w = np.zeros(2, np.uint32)
    rng = np.random.default_rng(3)
    disp = [(-1, 0), (0, 1), (1, 0), (0, -1)]
    for trial in range(20):
        start, goal = (int(x) for x in rng.choice(N * N, 2, replace=False))
        pos, tep = start, 0
        r, c = divmod(start, N)
        for k in range(200):
            a = int(rng.integers(0, 4))
            r, c = (r + disp[a][0]) % N, (c + disp[a][1]) % N
            pos, tep, rew, done = orc.env_step(N, w, start, goal, cap, pos, tep, a, orc.TORUS)
            if r * N + c == goal:
                assert (rew, done, pos, tep) == (1.0, 1, start, 0)
                break
            assert (rew, done, pos, tep) == (0.0, 0, r * N + c, k + 1)


def test_torus_and_grid_agree_away_from_the_edges_and_differ_on_them():
    N, cap = 6, 50
    w = np.zeros(2, np.uint32)
    w[0] = np.uint32(1 << 14)  # one wall at (2, 2)
    for pos in range(N * N):
        if pos == 14:
            continue
        r, c = divmod(pos, N)
        for a, (dr, dc) in enumerate([(-1, 0), (0, 1), (1, 0), (0, -1)]):
            g = orc.env_step(N, w, 0, 35, cap, pos, 0, a, orc.GRID)
            t = orc.env_step(N, w, 0, 35, cap, pos, 0, a, orc.TORUS)
            inside = 0 <= r + dr < N and 0 <= c + dc < N
            if inside:
                assert g == t
            else:
                assert g[0] == pos or g[3] == 1  # the grid blocks at the edge
                want = ((r + dr) % N) * N + (c + dc) % N
                assert t[0] == (0 if want == 35 else want)  # entering the goal (cell 35) restarts at the start cell 0


@pytest.mark.parametrize("N", [5, 8])
def test_torus_invariants_under_random_actions(N):
    B, steps, cap = 32, 300, 50
    C = N * N
    walls, start, goal = orc.env_init(23, B, N, 0.2)
    bits = unpack_walls(walls, C)
    rng = np.random.default_rng(6)
    for b in range(B):
        # brute-force component of the start cell under wrap-around adjacency
        seen, todo = {int(start[b])}, [int(start[b])]
        while todo:
            p = todo.pop()
            r, c = divmod(p, N)
            for nr, nc in (((r - 1) % N, c), (r, (c + 1) % N), ((r + 1) % N, c), (r, (c - 1) % N)):
                q = nr * N + nc
                if not bits[b, q] and q not in seen:
                    seen.add(q)
                    todo.append(q)
        pos, tep, since = int(start[b]), 0, 0
        for _ in range(steps):
            a = int(rng.integers(0, 4))
            r0, c0 = divmod(pos, N)
            tr, tc = [((r0 - 1) % N, c0), (r0, (c0 + 1) % N), ((r0 + 1) % N, c0), (r0, (c0 - 1) % N)][a]
            land = pos if bits[b, tr * N + tc] else tr * N + tc
            npos, ntep, rew, done = orc.env_step(N, walls[b], int(start[b]), int(goal[b]), cap, pos, tep, a, orc.TORUS)
            since += 1
            assert (rew == 1.0) == (land == goal[b])
            if land == goal[b] or since >= cap:
                assert done == 1 and npos == start[b] and ntep == 0
                since = 0
            else:
                assert done == 0 and npos == land and ntep == since
            assert not bits[b, npos] and npos in seen and ntep < cap
            pos, tep = npos, ntep
