"""ctypes/numpy wrapper around the CPU oracle (oracle/anakin_oracle.cpp).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the benchmark's CPU-baseline
leg import this module.  It never imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "anakin_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, OpenMP) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_uniform24.restype = C.c_double
        _lib.orc_act_uniform.restype = C.c_double
        _lib.orc_param_count.restype = C.c_uint64
        _lib.orc_num_threads.restype = C.c_int
    return _lib


def _p(a: np.ndarray | None):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


@dataclass(frozen=True)
class Dims:
    """Sizes of one workload: grid side N, hidden width H; flat parameter offsets."""

    N: int
    H: int

    @property
    def C(self):
        return self.N * self.N

    @property
    def D(self):
        return 3 * self.C

    @property
    def W(self):
        return (self.C + 31) // 32

    @property
    def P(self):
        return self.D * self.H + self.H + self.H * self.H + self.H + 5 * self.H + 5

    def slices(self):
        D, H = self.D, self.H
        o = 0
        out = {}
        for name, n in (("W1", D * H), ("b1", H), ("W2", H * H), ("b2", H), ("Wh", 5 * H), ("bh", 5)):
            out[name] = slice(o, o + n)
            o += n
        return out


def num_threads() -> int:
    return int(lib().orc_num_threads())


def set_num_threads(n: int) -> None:
    lib().orc_set_num_threads(C.c_int(n))


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def uniform24(x: int) -> float:
    return float(lib().orc_uniform24(C.c_uint32(x)))


def act_uniform(seed: int, b: int, gstep: int) -> float:
    return float(lib().orc_act_uniform(C.c_uint64(seed), C.c_uint32(b), C.c_uint32(gstep)))


def param_count(N: int, H: int) -> int:
    return int(lib().orc_param_count(C.c_int(N), C.c_int(H)))


def env_init(seed: int, B: int, N: int, density: float = 0.2):
    d = Dims(N, 16)
    walls = np.zeros((B, d.W), dtype=np.uint32)
    start = np.zeros(B, dtype=np.uint8)
    goal = np.zeros(B, dtype=np.uint8)
    lib().orc_env_init(C.c_uint64(seed), C.c_int(B), C.c_int(N), C.c_double(density), _p(walls), _p(start), _p(goal))
    return walls, start, goal


def param_init(seed: int, N: int, H: int) -> np.ndarray:
    theta = np.zeros(Dims(N, H).P, dtype=np.float32)
    lib().orc_param_init(C.c_uint64(seed), C.c_int(N), C.c_int(H), _p(theta))
    return theta


GRID, TORUS = 0, 1  # env kinds: walls and borders block / walls block and borders wrap around


def env_step(N: int, walls_b: np.ndarray, start: int, goal: int, cap: int, pos: int, tep: int, action: int, kind: int = GRID):
    """One env, one step.  Returns (pos', tep', reward, done)."""
    w = np.ascontiguousarray(walls_b, dtype=np.uint32)
    p = C.c_uint8(pos)
    t = C.c_uint8(tep)
    r = C.c_float(0)
    dn = C.c_uint8(0)
    lib().orc_env_step_kind(C.c_int(kind), C.c_int(N), _p(w), C.c_uint8(start), C.c_uint8(goal), C.c_int(cap), C.byref(p),
                            C.byref(t), C.c_int(action), C.byref(r), C.byref(dn))
    return int(p.value), int(t.value), float(r.value), int(dn.value)


def observe(N: int, walls_b: np.ndarray, pos: int, goal: int) -> np.ndarray:
    w = np.ascontiguousarray(walls_b, dtype=np.uint32)
    x = np.zeros(3 * N * N, dtype=np.float32)
    lib().orc_observe(C.c_int(N), _p(w), C.c_uint8(pos), C.c_uint8(goal), _p(x))
    return x


def round_bf16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty_like(a)
    lib().orc_round_bf16(C.c_size_t(a.size), _p(a), _p(out))
    return out


def forward(N: int, H: int, prec: int, theta: np.ndarray, x: np.ndarray, want_hidden: bool = False):
    """Dense rows x[n][D] -> out[n][5] (4 logits, 1 value); optionally h1, h2."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    n = x.shape[0]
    out = np.zeros((n, 5), dtype=np.float32)
    h1 = np.zeros((n, H), dtype=np.float32) if want_hidden else None
    h2 = np.zeros((n, H), dtype=np.float32) if want_hidden else None
    lib().orc_forward(C.c_int(N), C.c_int(H), C.c_int(prec), _p(theta), C.c_size_t(n), _p(x), _p(h1), _p(h2), _p(out))
    return (out, h1, h2) if want_hidden else out


def forward_f64(N: int, H: int, theta: np.ndarray, x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    theta = np.ascontiguousarray(theta, dtype=np.float64)
    out = np.zeros((x.shape[0], 5), dtype=np.float64)
    lib().orc_forward_f64(C.c_int(N), C.c_int(H), _p(theta), C.c_size_t(x.shape[0]), _p(x), _p(out))
    return out


def sample_one(logits4, u: float):
    l = np.ascontiguousarray(logits4, dtype=np.float32)
    a = C.c_int(0)
    lp = C.c_float(0)
    nr = C.c_uint8(0)
    lib().orc_sample_one(_p(l), C.c_double(u), C.byref(a), C.byref(lp), C.byref(nr))
    return int(a.value), float(lp.value), int(nr.value)


def sample_from_logits(seed: int, gstep0: int, logits: np.ndarray):
    """logits[T][B][4] -> (actions int8 [T][B], logp f32, near u8) using the ACT stream uniforms."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    T, B = logits.shape[0], logits.shape[1]
    act = np.zeros((T, B), dtype=np.int8)
    logp = np.zeros((T, B), dtype=np.float32)
    near = np.zeros((T, B), dtype=np.uint8)
    lib().orc_sample_from_logits(C.c_uint64(seed), C.c_uint32(gstep0), C.c_int(T), C.c_int(B), _p(logits), _p(act),
                                 _p(logp), _p(near))
    return act, logp, near


@dataclass
class Trajectory:
    pos: np.ndarray  # u8 [T][B]  state the action was taken in
    action: np.ndarray  # i8 [T][B]
    done: np.ndarray  # u8 [T][B]
    reward: np.ndarray  # f32 [T][B]
    value: np.ndarray  # f32 [T+1][B]
    logp: np.ndarray  # f32 [T][B]
    logits: np.ndarray  # f32 [T][B][4]
    near: np.ndarray  # u8 [T][B]  uniform within 1e-5 of a CDF boundary


def rollout(N, H, prec, T, cap, theta, walls, start, goal, pos, tep, seed, gstep0, forced=None, kind: int = GRID,
            env0: int = 0) -> Trajectory:
    """Runs T steps for all envs; pos/tep (uint8 arrays) are updated in place.  env0 = global index of the batch's first
    env (the action uniforms are keyed by env0 + b)."""
    B = walls.shape[0]
    tr = Trajectory(
        pos=np.zeros((T, B), np.uint8), action=np.zeros((T, B), np.int8), done=np.zeros((T, B), np.uint8),
        reward=np.zeros((T, B), np.float32), value=np.zeros((T + 1, B), np.float32),
        logp=np.zeros((T, B), np.float32), logits=np.zeros((T, B, 4), np.float32), near=np.zeros((T, B), np.uint8))
    if forced is not None:
        forced = np.ascontiguousarray(forced, dtype=np.int8)
        assert forced.shape == (T, B)
    lib().orc_rollout_env0(C.c_int(kind), C.c_int(N), C.c_int(H), C.c_int(prec), C.c_int(B), C.c_int(T), C.c_int(cap), _p(theta),
                           _p(walls), _p(start), _p(goal), _p(pos), _p(tep), C.c_uint64(seed), C.c_uint32(gstep0), _p(forced),
                           _p(tr.pos), _p(tr.action), _p(tr.done), _p(tr.reward), _p(tr.value), _p(tr.logp), _p(tr.logits),
                           _p(tr.near), C.c_uint32(env0))
    return tr


# ---- many policies: K independent networks, policy p on envs [p*Bp, min(B, (p+1)*Bp)), Bp = ceil(B/K) ----
def policy_envs(B: int, K: int, p: int) -> tuple[int, int]:
    """(first env, number of envs) of policy p."""
    Bp = (B + K - 1) // K
    return p * Bp, min(Bp, B - p * Bp)


def param_init_policy(seed: int, N: int, H: int, policy: int) -> np.ndarray:
    theta = np.zeros(Dims(N, H).P, dtype=np.float32)
    lib().orc_param_init_policy(C.c_uint64(seed), C.c_int(N), C.c_int(H), C.c_uint32(policy), _p(theta))
    return theta


def block(a: np.ndarray, B: int, K: int, p: int, rows: int, width: int = 1) -> np.ndarray:
    """Block p of a per-step array stored as K consecutive blocks [rows][B_p][width] (flat input), as [rows][B_p](,width)."""
    e0, Bk = policy_envs(B, K, p)
    v = a.reshape(-1)[rows * e0 * width: rows * (e0 + Bk) * width]
    return v.reshape(rows, Bk, width) if width > 1 else v.reshape(rows, Bk)


@dataclass
class PolicyTrajectories:
    """Flat arrays of K consecutive per-policy blocks (block p = [T][B_p]; value [T+1][B_p]; logits [T][B_p][4])."""
    pos: np.ndarray
    action: np.ndarray
    done: np.ndarray
    reward: np.ndarray
    value: np.ndarray
    logp: np.ndarray
    logits: np.ndarray
    near: np.ndarray


def rollout_policies(K, N, H, prec, T, cap, theta, walls, start, goal, pos, tep, seed, gstep0, kind: int = GRID) -> PolicyTrajectories:
    """K independent single-policy rollouts; theta [K][P]; pos/tep updated in place."""
    B = walls.shape[0]
    theta = np.ascontiguousarray(theta, np.float32)
    assert theta.shape == (K, Dims(N, H).P) and (K - 1) * ((B + K - 1) // K) < B
    tr = PolicyTrajectories(pos=np.zeros(T * B, np.uint8), action=np.zeros(T * B, np.int8), done=np.zeros(T * B, np.uint8),
                            reward=np.zeros(T * B, np.float32), value=np.zeros((T + 1) * B, np.float32),
                            logp=np.zeros(T * B, np.float32), logits=np.zeros(T * B * 4, np.float32), near=np.zeros(T * B, np.uint8))
    lib().orc_rollout_policies(C.c_int(kind), C.c_int(N), C.c_int(H), C.c_int(prec), C.c_int(B), C.c_int(K), C.c_int(T), C.c_int(cap),
                               _p(theta), _p(walls), _p(start), _p(goal), _p(pos), _p(tep), C.c_uint64(seed), C.c_uint32(gstep0),
                               _p(tr.pos), _p(tr.action), _p(tr.done), _p(tr.reward), _p(tr.value), _p(tr.logp), _p(tr.logits), _p(tr.near))
    return tr


def gae_policies(K, B, T, gamma, lam, reward, value, done):
    adv = np.zeros(T * B, np.float32)
    ret = np.zeros(T * B, np.float32)
    lib().orc_gae_policies(C.c_int(T), C.c_int(B), C.c_int(K), C.c_double(gamma), C.c_double(lam), _p(np.ascontiguousarray(reward, np.float32)),
                           _p(np.ascontiguousarray(value, np.float32)), _p(np.ascontiguousarray(done, np.uint8)), _p(adv), _p(ret))
    return adv, ret


def learn_policies(K, N, H, prec, T, theta, walls, goal, tpos, tact, adv, ret, c_v=0.5, c_e=0.01, gates=None):
    """K independent single-policy loss/gradient evaluations: (grads [K][P] f32, loss [K][4] f64[, gate reports])."""
    B = walls.shape[0]
    theta = np.ascontiguousarray(theta, np.float32)
    grads = np.zeros((K, Dims(N, H).P), np.float32)
    loss = np.zeros((K, 4), np.float64)
    g1 = g2 = info = None
    if gates is not None:
        g1, g2 = np.ascontiguousarray(gates[0], np.uint32), np.ascontiguousarray(gates[1], np.uint32)
        assert g1.size == g2.size == T * B * ((H + 31) // 32)
        info = np.zeros((K, 6), np.float64)
    lib().orc_learn_policies(C.c_int(N), C.c_int(H), C.c_int(prec), C.c_int(B), C.c_int(K), C.c_int(T), _p(theta), _p(walls), _p(goal),
                             _p(np.ascontiguousarray(tpos, np.uint8)), _p(np.ascontiguousarray(tact, np.int8)),
                             _p(np.ascontiguousarray(adv, np.float32)), _p(np.ascontiguousarray(ret, np.float32)), C.c_double(c_v),
                             C.c_double(c_e), _p(grads), _p(loss), _p(g1), _p(g2), _p(info))
    if gates is not None:
        reports = [{"layer1": dict(mismatched=int(i[0]), max_abs_z=float(i[1]), rms_z=float(i[2])),
                    "layer2": dict(mismatched=int(i[3]), max_abs_z=float(i[4]), rms_z=float(i[5]))} for i in info]
        return grads, loss, reports
    return grads, loss


def gae(gamma: float, lam: float, reward: np.ndarray, value: np.ndarray, done: np.ndarray):
    reward = np.ascontiguousarray(reward, np.float32)
    value = np.ascontiguousarray(value, np.float32)
    done = np.ascontiguousarray(done, np.uint8)
    T, B = reward.shape
    assert value.shape == (T + 1, B)
    adv = np.zeros((T, B), np.float32)
    ret = np.zeros((T, B), np.float32)
    lib().orc_gae(C.c_int(T), C.c_int(B), C.c_double(gamma), C.c_double(lam), _p(reward), _p(value), _p(done), _p(adv),
                  _p(ret))
    return adv, ret


def vtrace(gamma: float, rho_bar: float, c_bar: float, reward, value, done, logp_pi, logp_mu):
    """V-trace value targets and policy-gradient advantages (IMPALA, Eq. 1): returns (adv, ret) f32 [T][B]."""
    reward = np.ascontiguousarray(reward, np.float32)
    value = np.ascontiguousarray(value, np.float32)
    done = np.ascontiguousarray(done, np.uint8)
    logp_pi = np.ascontiguousarray(logp_pi, np.float32)
    logp_mu = np.ascontiguousarray(logp_mu, np.float32)
    T, B = reward.shape
    assert value.shape == (T + 1, B) and done.shape == (T, B) and logp_pi.shape == (T, B) and logp_mu.shape == (T, B)
    adv = np.empty((T, B), np.float32)
    ret = np.empty((T, B), np.float32)
    lib().orc_vtrace(C.c_int(T), C.c_int(B), C.c_double(gamma), C.c_double(rho_bar), C.c_double(c_bar), _p(reward), _p(value),
                     _p(done), _p(logp_pi), _p(logp_mu), _p(adv), _p(ret))
    return adv, ret


def learn(N, H, prec, theta, walls, goal, tpos, tact, adv, ret, c_v=0.5, c_e=0.01, want_grads=True, gates=None,
          logp_old=None, clip=0.0):
    """fp32-storage loss and batch-mean gradient; with `logp_old` the policy term is the clipped surrogate (PPO).  Returns (grads f32 [P] or None, loss[4] f64), plus a
    gate report when `gates` = (gate1, gate2) uint32 bitmaps [R][ceil(H/32)] recorded by the implementation
    under test are given: the backward pass then takes the ReLU gate decisions from them."""
    T, B = tpos.shape
    grads = np.zeros(Dims(N, H).P, np.float32) if want_grads else None
    loss = np.zeros(4, np.float64)
    g1 = g2 = info = None
    if gates is not None:
        g1 = np.ascontiguousarray(gates[0], np.uint32)
        g2 = np.ascontiguousarray(gates[1], np.uint32)
        assert g1.size == g2.size == T * B * ((H + 31) // 32)
        info = np.zeros(6, np.float64)
    if logp_old is None:
        lib().orc_learn_f32(C.c_int(N), C.c_int(H), C.c_int(prec), C.c_int(B), C.c_int(T), _p(theta), _p(walls), _p(goal),
                            _p(np.ascontiguousarray(tpos, np.uint8)), _p(np.ascontiguousarray(tact, np.int8)),
                            _p(np.ascontiguousarray(adv, np.float32)), _p(np.ascontiguousarray(ret, np.float32)),
                            C.c_double(c_v), C.c_double(c_e), _p(grads), _p(loss), _p(g1), _p(g2), _p(info))
    else:
        lib().orc_learn_ppo_f32(C.c_int(N), C.c_int(H), C.c_int(prec), C.c_int(B), C.c_int(T), _p(theta), _p(walls), _p(goal),
                                _p(np.ascontiguousarray(tpos, np.uint8)), _p(np.ascontiguousarray(tact, np.int8)),
                                _p(np.ascontiguousarray(adv, np.float32)), _p(np.ascontiguousarray(ret, np.float32)),
                                _p(np.ascontiguousarray(logp_old, np.float32)), C.c_double(clip), C.c_double(c_v),
                                C.c_double(c_e), _p(grads), _p(loss), _p(g1), _p(g2), _p(info))
    if gates is not None:
        report = {"layer1": dict(mismatched=int(info[0]), max_abs_z=float(info[1]), rms_z=float(info[2])),
                  "layer2": dict(mismatched=int(info[3]), max_abs_z=float(info[4]), rms_z=float(info[5]))}
        return grads, loss, report
    return grads, loss


def learn_f64(N, H, theta, walls, goal, tpos, tact, adv, ret, c_v=0.5, c_e=0.01, want_grads=True, logp_old=None, clip=0.0):
    T, B = tpos.shape
    theta = np.ascontiguousarray(theta, np.float64)
    grads = np.zeros(Dims(N, H).P, np.float64) if want_grads else None
    loss = np.zeros(4, np.float64)
    if logp_old is not None:
        lib().orc_learn_ppo_f64(C.c_int(N), C.c_int(H), C.c_int(B), C.c_int(T), _p(theta), _p(walls), _p(goal),
                                _p(np.ascontiguousarray(tpos, np.uint8)), _p(np.ascontiguousarray(tact, np.int8)),
                                _p(np.ascontiguousarray(adv, np.float64)), _p(np.ascontiguousarray(ret, np.float64)),
                                _p(np.ascontiguousarray(logp_old, np.float64)), C.c_double(clip), C.c_double(c_v),
                                C.c_double(c_e), _p(grads), _p(loss))
        return grads, loss
    lib().orc_learn_f64(C.c_int(N), C.c_int(H), C.c_int(B), C.c_int(T), _p(theta), _p(walls), _p(goal),
                        _p(np.ascontiguousarray(tpos, np.uint8)), _p(np.ascontiguousarray(tact, np.int8)),
                        _p(np.ascontiguousarray(adv, np.float64)), _p(np.ascontiguousarray(ret, np.float64)),
                        C.c_double(c_v), C.c_double(c_e), _p(grads), _p(loss))
    return grads, loss


def adam(theta, g, m, v, k, lr=3e-4, b1=0.9, b2=0.999, eps=1e-8):
    """In-place Adam step number k (first step: k=1) on fp32 arrays."""
    for a in (theta, g, m, v):
        assert a.dtype == np.float32 and a.flags["C_CONTIGUOUS"]
    lib().orc_adam(C.c_size_t(theta.size), _p(theta), _p(g), _p(m), _p(v), C.c_int(k), C.c_double(lr), C.c_double(b1),
                   C.c_double(b2), C.c_double(eps))


class Agent:
    """The whole loop on the CPU: reset(seed), rollout(T), learn(), run(iters) with the same state the
    library keeps (params, Adam moments and step, env static/dynamic state, global step counter)."""

    def __init__(self, B, N, H, T, prec=0, cap=50, density=0.2, gamma=0.99, lam=0.95, c_e=0.01, c_v=0.5, lr=3e-4,
                 b1=0.9, b2=0.999, eps=1e-8, kind=GRID):
        self.kind = kind
        self.B, self.N, self.H, self.T, self.prec, self.cap, self.density = B, N, H, T, prec, cap, density
        self.gamma, self.lam, self.c_e, self.c_v = gamma, lam, c_e, c_v
        self.lr, self.b1, self.b2, self.eps = lr, b1, b2, eps
        self.dims = Dims(N, H)
        self.traj = None

    def reset(self, seed: int):
        self.seed = seed
        self.walls, self.start, self.goal = env_init(seed, self.B, self.N, self.density)
        self.pos = self.start.copy()
        self.tep = np.zeros(self.B, np.uint8)
        self.theta = param_init(seed, self.N, self.H)
        self.m = np.zeros_like(self.theta)
        self.v = np.zeros_like(self.theta)
        self.k = 0
        self.gstep = 0
        self.traj = None

    def rollout(self, T=None, forced=None) -> Trajectory:
        T = self.T if T is None else T
        self.traj = rollout(self.N, self.H, self.prec, T, self.cap, self.theta, self.walls, self.start, self.goal,
                            self.pos, self.tep, self.seed, self.gstep, forced, self.kind)
        self.gstep += T
        return self.traj

    def learn(self):
        tr = self.traj
        self.adv, self.ret = gae(self.gamma, self.lam, tr.reward, tr.value, tr.done)
        self.grads, self.loss = learn(self.N, self.H, self.prec, self.theta, self.walls, self.goal, tr.pos, tr.action,
                                      self.adv, self.ret, self.c_v, self.c_e)
        self.k += 1
        adam(self.theta, self.grads, self.m, self.v, self.k, self.lr, self.b1, self.b2, self.eps)
        self.traj = None

    def learn_ppo(self, epochs: int, clip: float):
        """`epochs` full-batch Adam steps on the clipped surrogate of the pending trajectory (advantages and recorded
        log-probabilities stay fixed; the forward pass is recomputed with the current parameters every epoch)."""
        tr = self.traj
        self.adv, self.ret = gae(self.gamma, self.lam, tr.reward, tr.value, tr.done)
        for _ in range(epochs):
            self.grads, self.loss = learn(self.N, self.H, self.prec, self.theta, self.walls, self.goal, tr.pos, tr.action,
                                          self.adv, self.ret, self.c_v, self.c_e, logp_old=tr.logp, clip=clip)
            self.k += 1
            adam(self.theta, self.grads, self.m, self.v, self.k, self.lr, self.b1, self.b2, self.eps)
        self.traj = None

    def run(self, iters: int):
        for _ in range(iters):
            self.rollout()
            self.learn()
