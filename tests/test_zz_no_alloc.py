"""anakin_rollout_noalloc against anakin_rollout (needs a B200).  Collected last on purpose.

The no-allocation entry point serves callers that cannot call cudaMalloc (fixed memory budgets, hosts that own
the allocator, loops that must not synchronise the device): they pass inputs and outputs only, and the rollout's
scratch is a fixed array inside the library.  It must give what the handle-based rollout gives, call after call,
although every call reuses the same array.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_noalloc_rollout_matches_handle_rollout_twice_in_a_row():
    from paper_2104_06272_b200 import binding as bnd
    from paper_2104_06272_b200.workloads import WORKLOADS, random_params

    w = WORKLOADS["throughput"].scaled(B=1000 + 13, T=12)  # B*H = 259,328 floats of scratch, ragged last CTA
    seed = 21
    cfg = bnd.cfg_from_workload(w)
    an = bnd.Anakin(cfg)
    an.reset(seed)
    an.set(bnd.PARAMS, random_params(3, w.P, 0.15))
    def dev(a):
        a = np.ascontiguousarray(a)
        return torch.from_numpy(a.view(np.int32) if a.dtype == np.uint32 else a).cuda()

    params, walls = dev(an.get(bnd.PARAMS)), dev(an.get(bnd.ENV_WALLS))
    start, goal = dev(an.get(bnd.ENV_START)), dev(an.get(bnd.ENV_GOAL))
    pos, tep = dev(an.get(bnd.ENV_POS)), dev(an.get(bnd.ENV_TEP))
    T, B = w.T, w.B
    out = dict(pos=torch.empty(T * B, dtype=torch.uint8, device="cuda"), action=torch.empty(T * B, dtype=torch.int8, device="cuda"),
               done=torch.empty(T * B, dtype=torch.uint8, device="cuda"), reward=torch.empty(T * B, dtype=torch.float32, device="cuda"),
               value=torch.empty((T + 1) * B, dtype=torch.float32, device="cuda"), logp=torch.empty(T * B, dtype=torch.float32, device="cuda"))
    blobs = dict(pos=bnd.TRAJ_POS, action=bnd.TRAJ_ACTION, done=bnd.TRAJ_DONE, reward=bnd.TRAJ_REWARD, value=bnd.TRAJ_VALUE,
                 logp=bnd.TRAJ_LOGP)
    n_allocs = lambda: torch.cuda.memory_stats().get("allocation.all.allocated", 0)  # cumulative allocation count
    for call in range(2):  # the second call continues from the first one's env state and step counter
        gstep = int(an.get(bnd.GLOBAL_STEP))
        assert gstep == call * T
        before = n_allocs()
        rc = bnd.rollout_noalloc(cfg, seed, gstep, T, params, walls, start, goal, pos, tep, out["pos"], out["action"],
                                 out["done"], out["reward"], out["value"], out["logp"])
        assert rc == bnd.OK
        assert n_allocs() == before  # torch's allocator saw nothing from the call
        assert bnd.noalloc_status() == (bnd.OK, 0)  # the word in the array's tail, which no handle owns
        an.rollout(T)
        torch.cuda.synchronize()
        for name, blob in blobs.items():
            want, got = an.get(blob), out[name].cpu().numpy()
            if want.dtype == np.float32:  # same kernels: well inside the fp32 tolerance of the parity tests (1e-4)
                assert np.allclose(got, want, rtol=1e-4, atol=1e-6), (call, name)
                assert (got.view(np.uint32) == want.view(np.uint32)).all(), (call, name)
            else:
                assert (got == want).all(), (call, name)
        assert (pos.cpu().numpy() == an.get(bnd.ENV_POS)).all() and (tep.cpu().numpy() == an.get(bnd.ENV_TEP)).all()


def test_noalloc_status_reports_a_start_position_on_a_wall():
    """A caller-supplied env state that is not a legal one (the agent on a wall cell) must not pass silently: the kernels
    flag it in the status word, and anakin_noalloc_status is the only way a handle-less caller can read that word."""
    from paper_2104_06272_b200 import binding as bnd
    from paper_2104_06272_b200.workloads import WORKLOADS, random_params

    w = WORKLOADS["tiny"]
    cfg = bnd.cfg_from_workload(w)
    an = bnd.Anakin(cfg)
    an.reset(5)
    walls_h = an.get(bnd.ENV_WALLS).reshape(w.B, -1)
    pos_h = an.get(bnd.ENV_POS).copy()
    env = next(b for b in range(w.B) if walls_h[b].any())
    cell = next(c for c in range(w.N * w.N) if (walls_h[env][c // 32] >> (c % 32)) & 1)
    pos_h[env] = cell  # the agent of one env now stands on a wall
    dev = lambda a: torch.from_numpy(a.view(np.int32) if a.dtype == np.uint32 else np.ascontiguousarray(a)).cuda()
    T, B = w.T, w.B
    u8 = lambda n: torch.empty(n, dtype=torch.uint8, device="cuda")
    f32 = lambda n: torch.empty(n, dtype=torch.float32, device="cuda")
    outs = (u8(T * B), torch.empty(T * B, dtype=torch.int8, device="cuda"), u8(T * B), f32(T * B), f32((T + 1) * B), f32(T * B))
    ins = (dev(random_params(3, w.P, 0.15)), dev(an.get(bnd.ENV_WALLS)), dev(an.get(bnd.ENV_START)), dev(an.get(bnd.ENV_GOAL)))
    for bad in (True, False):  # a clean call afterwards clears the word again
        pos = dev(pos_h if bad else an.get(bnd.ENV_POS))
        assert bnd.rollout_noalloc(cfg, 5, 0, T, *ins, pos, dev(an.get(bnd.ENV_TEP)), *outs) == bnd.OK
        rc, st = bnd.noalloc_status()
        assert (rc, st != 0) == ((bnd.E_DEVICE_STATUS, True) if bad else (bnd.OK, False)), (bad, rc, st)


def test_noalloc_rollout_refuses_what_does_not_fit():
    from paper_2104_06272_b200 import binding as bnd

    z8 = torch.zeros(8, dtype=torch.uint8, device="cuda")
    zf = torch.zeros(8, dtype=torch.float32, device="cuda")
    zi = torch.zeros(8, dtype=torch.int8, device="cuda")
    zw = torch.zeros(8, dtype=torch.int32, device="cuda")
    args = (zf, zw, z8, z8, z8, z8, z8, zi, z8, zf, zf, zf)
    too_big = bnd.make_cfg(B=bnd.NOALLOC_MAX_BH // 256 + 1, N=10, H=256, T_max=4)
    assert bnd.rollout_noalloc(too_big, 1, 0, 4, *args) == bnd.E_WORKSPACE_TOO_SMALL
    bf16 = bnd.make_cfg(B=64, N=5, H=64, T_max=4, precision=1)
    assert bnd.rollout_noalloc(bf16, 1, 0, 4, *args) == bnd.E_UNSUPPORTED_CFG
    ok_cfg = bnd.make_cfg(B=64, N=5, H=64, T_max=4)
    assert bnd.rollout_noalloc(ok_cfg, 1, 0, 5, *args) == bnd.E_INVALID_ARG  # T > T_max
    assert bnd.rollout_noalloc(ok_cfg, 1, -1, 4, *args) == bnd.E_INVALID_ARG
