"""Thin Python binding over libanakin.so (the C ABI of include/anakin.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch is used for
device memory (the workspace is one torch uint8 tensor) and for the stream.  If the library has not been
built, importing this module raises: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libanakin.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2104_06272_b200.build` (nvcc, sm_100a). "
        "There is no CPU or PyTorch fallback."
    )
_lib = C.CDLL(LIB_PATH)


class AnakinCfg(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("B", C.c_int32), ("N", C.c_int32), ("H", C.c_int32), ("T_max", C.c_int32),
        ("episode_cap", C.c_int32), ("wall_density", C.c_double),
        ("gamma", C.c_float), ("gae_lambda", C.c_float), ("entropy_coef", C.c_float), ("value_coef", C.c_float),
        ("lr", C.c_float), ("adam_b1", C.c_float), ("adam_b2", C.c_float), ("adam_eps", C.c_float),
        ("precision", C.c_int32), ("device", C.c_int32), ("debug_logits", C.c_int32), ("env_offset", C.c_int32), ("env_kind", C.c_int32), ("n_policies", C.c_int32),
    ]


class AnakinStats(C.Structure):
    _fields_ = [("frames", C.c_uint64), ("episodes", C.c_uint64), ("goals", C.c_uint64), ("episode_steps", C.c_uint64),
                ("loss_total", C.c_float), ("loss_pg", C.c_float), ("loss_value", C.c_float), ("entropy", C.c_float)]


# error codes / blob selectors (mirrors of the header's enums)
OK, E_INVALID_ARG, E_BAD_STATE, E_WORKSPACE_TOO_SMALL, E_UNSUPPORTED_CFG, E_CUDA, E_DEVICE_STATUS = 0, -1, -2, -3, -4, -5, -6
(PARAMS, GRADS, ADAM_M, ADAM_V, ADAM_STEP, ENV_WALLS, ENV_START, ENV_GOAL, ENV_POS, ENV_TEP, GLOBAL_STEP, TRAJ_POS,
 TRAJ_ACTION, TRAJ_DONE, TRAJ_REWARD, TRAJ_VALUE, TRAJ_LOGP, ADV, RET, STATS, DEBUG_LOGITS, DEBUG_GATES) = range(22)

EXPORTS = [
    "anakin_workspace_bytes", "anakin_create", "anakin_destroy", "anakin_reset", "anakin_rollout",
    "anakin_rollout_forced", "anakin_learn", "anakin_gae", "anakin_update", "anakin_grads", "anakin_apply_grads", "anakin_apply_grads_mean", "anakin_learn_ppo", "anakin_learn_vtrace",
    "anakin_run", "anakin_get", "anakin_set",
    "anakin_blob_bytes", "anakin_status", "anakin_launch_count", "anakin_strerror", "anakin_last_cuda_error",
    "anakin_profile_enable", "anakin_profile_read", "anakin_kernel_count", "anakin_kernel_name",
    "anakin_rollout_noalloc", "anakin_noalloc_status", "anakin_selftest_wait_timeout",
]

_vp = C.c_void_p
_lib.anakin_workspace_bytes.argtypes = [C.POINTER(AnakinCfg), C.POINTER(C.c_size_t)]
_lib.anakin_create.argtypes = [C.POINTER(AnakinCfg), _vp, C.c_size_t, _vp, C.POINTER(_vp)]
_lib.anakin_destroy.argtypes = [_vp]
_lib.anakin_reset.argtypes = [_vp, C.c_uint64]
_lib.anakin_rollout.argtypes = [_vp, C.c_int]
_lib.anakin_rollout_forced.argtypes = [_vp, C.c_int, _vp]
_lib.anakin_learn.argtypes = [_vp]
_lib.anakin_gae.argtypes = [_vp]
_lib.anakin_update.argtypes = [_vp]
_lib.anakin_grads.argtypes = [_vp]
_lib.anakin_apply_grads.argtypes = [_vp]
_lib.anakin_apply_grads_mean.argtypes = [_vp, C.c_int]
_lib.anakin_learn_ppo.argtypes = [_vp, C.c_int, C.c_float]
_lib.anakin_learn_vtrace.argtypes = [_vp, C.c_int, C.c_float, C.c_float]
_lib.anakin_run.argtypes = [_vp, C.c_int]
_lib.anakin_get.argtypes = [_vp, C.c_int, _vp, C.c_size_t, C.c_int]
_lib.anakin_set.argtypes = [_vp, C.c_int, _vp, C.c_size_t, C.c_int]
_lib.anakin_blob_bytes.argtypes = [_vp, C.c_int]
_lib.anakin_blob_bytes.restype = C.c_size_t
_lib.anakin_status.argtypes = [_vp, C.POINTER(C.c_int)]
_lib.anakin_launch_count.argtypes = [_vp]
_lib.anakin_launch_count.restype = C.c_uint64
_lib.anakin_strerror.argtypes = [C.c_int]
_lib.anakin_strerror.restype = C.c_char_p
_lib.anakin_last_cuda_error.argtypes = [_vp]
_lib.anakin_last_cuda_error.restype = C.c_char_p
_lib.anakin_profile_enable.argtypes = [_vp, C.c_int]
_lib.anakin_profile_read.argtypes = [_vp, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]
_lib.anakin_kernel_count.argtypes = []
_lib.anakin_kernel_name.argtypes = [C.c_int]
_lib.anakin_kernel_name.restype = C.c_char_p
_lib.anakin_rollout_noalloc.argtypes = [C.POINTER(AnakinCfg), C.c_uint64, C.c_int64, C.c_int] + [_vp] * 13
_lib.anakin_selftest_wait_timeout.argtypes = [_vp, C.c_int64]
_lib.anakin_noalloc_status.argtypes = [_vp, C.POINTER(C.c_int)]
NOALLOC_MAX_BH = 1048576
ENV_GRID, ENV_TORUS = 0, 1  # anakin_cfg.env_kind

_BLOB_DTYPE = {
    PARAMS: np.float32, GRADS: np.float32, ADAM_M: np.float32, ADAM_V: np.float32, ENV_WALLS: np.uint32,
    ENV_START: np.uint8, ENV_GOAL: np.uint8, ENV_POS: np.uint8, ENV_TEP: np.uint8, TRAJ_POS: np.uint8,
    TRAJ_ACTION: np.int8, TRAJ_DONE: np.uint8, TRAJ_REWARD: np.float32, TRAJ_VALUE: np.float32, TRAJ_LOGP: np.float32,
    ADV: np.float32, RET: np.float32, DEBUG_LOGITS: np.float32, DEBUG_GATES: np.uint32,
}


class AnakinError(RuntimeError):
    def __init__(self, code: int, detail: str = ""):
        self.code = code
        msg = _lib.anakin_strerror(code).decode()
        super().__init__(f"anakin error {code}: {msg}" + (f" ({detail})" if detail else ""))


def lib() -> C.CDLL:
    return _lib


def make_cfg(B, N, H, T_max, precision=0, episode_cap=50, wall_density=0.2, gamma=0.99, gae_lambda=0.95,
             entropy_coef=0.01, value_coef=0.5, lr=3e-4, adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8, device=0,
             debug_logits=0, env_offset=0, env_kind=0, n_policies=0) -> AnakinCfg:
    c = AnakinCfg()
    c.struct_size = C.sizeof(AnakinCfg)
    c.B, c.N, c.H, c.T_max, c.episode_cap, c.wall_density = B, N, H, T_max, episode_cap, wall_density
    c.gamma, c.gae_lambda, c.entropy_coef, c.value_coef = gamma, gae_lambda, entropy_coef, value_coef
    c.lr, c.adam_b1, c.adam_b2, c.adam_eps = lr, adam_b1, adam_b2, adam_eps
    c.precision, c.device, c.debug_logits, c.env_offset = precision, device, debug_logits, env_offset
    c.env_kind, c.n_policies = env_kind, n_policies
    return c


def cfg_from_workload(w, device=0, debug_logits=0, T_max=None, env_offset=0) -> AnakinCfg:
    return make_cfg(w.B, w.N, w.H, w.T if T_max is None else T_max, w.precision, w.episode_cap, w.wall_density, w.gamma,
                    w.gae_lambda, w.entropy_coef, w.value_coef, w.lr, w.adam_b1, w.adam_b2, w.adam_eps, device,
                    debug_logits, env_offset, getattr(w, "env_kind", 0), getattr(w, "n_policies", 0))


def workspace_bytes(cfg: AnakinCfg) -> int:
    n = C.c_size_t(0)
    rc = _lib.anakin_workspace_bytes(C.byref(cfg), C.byref(n))
    if rc != OK:
        raise AnakinError(rc)
    return int(n.value)


def rollout_noalloc(cfg: AnakinCfg, seed: int, global_step: int, T: int, params, walls, start, goal, pos, tep,
                    traj_pos, traj_action, traj_done, traj_reward, traj_value, traj_logp, stream=None) -> int:
    """anakin_rollout_noalloc: a rollout without handle or workspace, for callers that cannot allocate device
    memory.  Every array argument is a CUDA tensor the caller owns (inputs, in/out env state, outputs); the call
    allocates nothing.  Returns the library's status code (0 = ok) instead of raising, so a caller can test limits."""
    ts = (params, walls, start, goal, pos, tep, traj_pos, traj_action, traj_done, traj_reward, traj_value, traj_logp)
    assert all(t.is_cuda and t.is_contiguous() for t in ts)
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(_lib.anakin_rollout_noalloc(C.byref(cfg), C.c_uint64(seed), C.c_int64(global_step), C.c_int(T),
                                           *[_vp(t.data_ptr()) for t in ts], _vp(s.cuda_stream)))


def noalloc_status(stream=None) -> tuple[int, int]:
    """anakin_noalloc_status: (return code, device status word) of the last rollout_noalloc call on the current
    device; synchronises the stream."""
    s = stream if stream is not None else torch.cuda.current_stream()
    st = C.c_int(0)
    rc = int(_lib.anakin_noalloc_status(_vp(s.cuda_stream), C.byref(st)))
    return rc, int(st.value)


class Anakin:
    """anakin_create / reset / rollout / learn / run over a torch-owned workspace and stream."""

    def __init__(self, cfg: AnakinCfg, stream: torch.cuda.Stream | None = None):
        if not torch.cuda.is_available():
            raise RuntimeError("the Anakin library needs a CUDA device; there is no CPU fallback")
        self.cfg = cfg
        self.device = torch.device("cuda", cfg.device)
        torch.cuda.set_device(self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self.nbytes = workspace_bytes(cfg)
        self.workspace = torch.empty(self.nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self._h = _vp()
        rc = _lib.anakin_create(C.byref(cfg), _vp(base), C.c_size_t(self.nbytes), _vp(self.stream.cuda_stream), C.byref(self._h))
        if rc != OK:
            raise AnakinError(rc)
        self.B, self.N, self.H, self.T_max = cfg.B, cfg.N, cfg.H, cfg.T_max
        self.K = cfg.n_policies if cfg.n_policies >= 2 else 1  # independent policies; blobs hold them one after the other
        self.P = 3 * cfg.N * cfg.N * cfg.H + cfg.H + cfg.H * cfg.H + cfg.H + 5 * cfg.H + 5

    def _ck(self, rc: int):
        if rc != OK:
            raise AnakinError(rc, _lib.anakin_last_cuda_error(self._h).decode())

    def close(self):
        if self._h:
            _lib.anakin_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self, seed: int):
        self._ck(_lib.anakin_reset(self._h, C.c_uint64(seed)))

    def rollout(self, T: int | None = None):
        self._ck(_lib.anakin_rollout(self._h, self.T_max if T is None else T))

    def rollout_forced(self, actions: torch.Tensor):
        """actions: int8 CUDA tensor [T][B]."""
        assert actions.is_cuda and actions.dtype == torch.int8 and actions.is_contiguous() and actions.shape[1] == self.B
        self._ck(_lib.anakin_rollout_forced(self._h, int(actions.shape[0]), _vp(actions.data_ptr())))

    def learn(self):
        self._ck(_lib.anakin_learn(self._h))

    def gae(self):
        self._ck(_lib.anakin_gae(self._h))

    def update(self):
        self._ck(_lib.anakin_update(self._h))

    def grads(self):
        self._ck(_lib.anakin_grads(self._h))

    def apply_grads(self, n_replicas: int = 1):
        """Adam from GRADS; n_replicas > 1: GRADS holds the sum over that many replicas (divided on the device)."""
        self._ck(_lib.anakin_apply_grads_mean(self._h, C.c_int(n_replicas)))

    def learn_ppo(self, epochs: int, clip_eps: float):
        self._ck(_lib.anakin_learn_ppo(self._h, epochs, C.c_float(clip_eps)))

    def learn_vtrace(self, epochs: int, rho_bar: float = 1.0, c_bar: float = 1.0):
        self._ck(_lib.anakin_learn_vtrace(self._h, epochs, C.c_float(rho_bar), C.c_float(c_bar)))

    def run(self, iters: int):
        self._ck(_lib.anakin_run(self._h, iters))

    def blob_bytes(self, which: int) -> int:
        return int(_lib.anakin_blob_bytes(self._h, which))

    def get(self, which: int) -> np.ndarray:
        """Copies a blob to a new host array (synchronises the stream)."""
        if which in (ADAM_STEP, GLOBAL_STEP):
            v = C.c_int64(0)
            self._ck(_lib.anakin_get(self._h, which, C.byref(v), 8, 0))
            return np.int64(v.value)
        if which == STATS:
            if self.K > 1:  # one record per policy
                arr = (AnakinStats * self.K)()
                self._ck(_lib.anakin_get(self._h, which, arr, C.sizeof(arr), 0))
                return list(arr)
            s = AnakinStats()
            self._ck(_lib.anakin_get(self._h, which, C.byref(s), C.sizeof(s), 0))
            return s
        n = self.blob_bytes(which)
        out = np.empty(n // np.dtype(_BLOB_DTYPE[which]).itemsize, dtype=_BLOB_DTYPE[which])
        self._ck(_lib.anakin_get(self._h, which, out.ctypes.data_as(_vp), n, 0))
        return out

    def get_into(self, which: int, out: torch.Tensor, wait: bool = True):
        """Copies a blob into a tensor of exactly the blob's size: a host tensor (synchronises; with wait=False and a pinned
        tensor the copy is only enqueued and the caller synchronises later, e.g. with status()) or a CUDA tensor on the
        handle's device (asynchronous, on the handle's stream)."""
        assert out.is_contiguous()
        if out.is_cuda:
            kind = 1
        elif not wait:
            assert out.is_pinned(), "an asynchronous read needs page-locked host memory"
            kind = 2
        else:
            kind = 0
        self._ck(_lib.anakin_get(self._h, which, _vp(out.data_ptr()), out.numel() * out.element_size(), kind))

    def set(self, which: int, value):
        if which in (ADAM_STEP, GLOBAL_STEP):
            v = C.c_int64(int(value))
            self._ck(_lib.anakin_set(self._h, which, C.byref(v), 8, 0))
            return
        if isinstance(value, torch.Tensor):
            assert value.is_contiguous()
            self._ck(_lib.anakin_set(self._h, which, _vp(value.data_ptr()), value.numel() * value.element_size(),
                                     1 if value.is_cuda else 0))
            return
        a = np.ascontiguousarray(value, dtype=_BLOB_DTYPE[which])
        self._ck(_lib.anakin_set(self._h, which, a.ctypes.data_as(_vp), a.nbytes, 0))

    def status(self) -> int:
        st = C.c_int(0)
        rc = _lib.anakin_status(self._h, C.byref(st))
        if rc not in (OK, E_DEVICE_STATUS):
            self._ck(rc)
        return int(st.value)

    def selftest_wait_timeout(self, limit_clocks: int = 1_000_000):
        """Enqueues the one-CTA kernel whose bounded wait must run out (status bit 4 afterwards)."""
        self._ck(_lib.anakin_selftest_wait_timeout(self._h, C.c_int64(limit_clocks)))

    def launch_count(self) -> int:
        return int(_lib.anakin_launch_count(self._h))

    def stats(self):
        """The statistics record (a list of K records with many policies)."""
        return self.get(STATS)

    def policy_envs(self, p: int) -> tuple[int, int]:
        """(first env, number of envs) of policy p: ceil(B/K) envs each, the last policy takes the rest."""
        bp = (self.B + self.K - 1) // self.K
        return p * bp, min(bp, self.B - p * bp)

    def policy_block(self, blob: np.ndarray, p: int, rows: int, width: int = 1) -> np.ndarray:
        """Policy p's block of a per-step blob read with get() (K consecutive blocks [rows][B_p][width])."""
        e0, n = self.policy_envs(p)
        v = blob.reshape(-1)[rows * e0 * width: rows * (e0 + n) * width]
        return v.reshape(rows, n, width) if width > 1 else v.reshape(rows, n)

    def profile_enable(self, on: bool):
        self._ck(_lib.anakin_profile_enable(self._h, 1 if on else 0))

    def profile_read(self) -> dict:
        """{kernel name: (total milliseconds, launches)} since the last read; synchronises the stream."""
        n = int(_lib.anakin_kernel_count())
        ms = (C.c_double * n)()
        cnt = (C.c_uint64 * n)()
        self._ck(_lib.anakin_profile_read(self._h, n, ms, cnt))
        return {_lib.anakin_kernel_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n) if cnt[i]}
