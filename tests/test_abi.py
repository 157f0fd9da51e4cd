"""The C-ABI library loads and exports every call the header declares; host-side argument checks
(no GPU work is enqueued by anything here)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bnd():
    from paper_2104_06272_b200 import build

    build.build()
    from paper_2104_06272_b200 import binding

    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "anakin.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(anakin_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(bnd):
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(bnd.lib(), n), f"{n} declared in include/anakin.h but not exported"
    assert sorted(bnd.EXPORTS) == names


def test_cfg_struct_matches_header_size(bnd):
    # a wrong struct_size is refused, the right one accepted: the Python mirror has the C layout
    cfg = bnd.make_cfg(64, 5, 64, 16)
    assert bnd.workspace_bytes(cfg) > 0
    cfg.struct_size += 4
    with pytest.raises(bnd.AnakinError) as e:
        bnd.workspace_bytes(cfg)
    assert e.value.code == bnd.E_INVALID_ARG
    assert C.sizeof(bnd.AnakinCfg) == 88 and C.sizeof(bnd.AnakinStats) == 48


@pytest.mark.parametrize("kw,code", [
    (dict(B=0), -1), (dict(T_max=0), -1), (dict(episode_cap=0), -1), (dict(episode_cap=256), -1),
    (dict(wall_density=1.0), -1), (dict(precision=2), -1),
    (dict(N=17), -4), (dict(N=1), -4), (dict(H=100), -4), (dict(H=2048), -4), (dict(H=160), -4),
])
def test_bad_configs_are_refused(bnd, kw, code):
    args = dict(B=64, N=5, H=64, T_max=16)
    args.update(kw)
    cfg = bnd.make_cfg(**args)
    with pytest.raises(bnd.AnakinError) as e:
        bnd.workspace_bytes(cfg)
    assert e.value.code == code


def test_many_policies_take_one_sub_workspace_each_and_limits_are_refused(bnd):
    one = bnd.workspace_bytes(bnd.make_cfg(B=34, N=5, H=64, T_max=4))
    assert bnd.workspace_bytes(bnd.make_cfg(B=100, N=5, H=64, T_max=4, n_policies=3)) == 3 * one  # ceil(100/3) = 34 envs each
    assert bnd.workspace_bytes(bnd.make_cfg(B=34, N=5, H=64, T_max=4, n_policies=1)) == one
    for kw, code in ((dict(precision=1), bnd.E_UNSUPPORTED_CFG), (dict(H=96), bnd.E_UNSUPPORTED_CFG), (dict(B=2), bnd.E_INVALID_ARG),
                     (dict(B=9, n_policies=4), bnd.E_INVALID_ARG), (dict(n_policies=-1), bnd.E_INVALID_ARG)):
        args = dict(B=100, N=5, H=64, T_max=4, n_policies=3)
        args.update(kw)
        with pytest.raises(bnd.AnakinError) as e:
            bnd.workspace_bytes(bnd.make_cfg(**args))
        assert e.value.code == code, kw
    cfg = bnd.make_cfg(B=100, N=5, H=64, T_max=4, n_policies=3)
    z = [None] * 12
    assert bnd.lib().anakin_rollout_noalloc(C.byref(cfg), 1, 0, 4, *z, None) == bnd.E_UNSUPPORTED_CFG


def test_workspace_grows_with_the_workload(bnd):
    from paper_2104_06272_b200.workloads import WORKLOADS

    sizes = {k: bnd.workspace_bytes(bnd.cfg_from_workload(w)) for k, w in WORKLOADS.items()}
    assert sizes["tiny"] < sizes["throughput"] < sizes["large_batch"]
    assert all(v < 60e9 for v in sizes.values())  # every preset fits one B200 several times over
    # the workspace is a pure function of the configuration
    assert sizes["tiny"] == bnd.workspace_bytes(bnd.cfg_from_workload(WORKLOADS["tiny"]))
    assert bnd.workspace_bytes(bnd.cfg_from_workload(WORKLOADS["tiny"], debug_logits=1)) > sizes["tiny"]


def test_create_checks_its_arguments_before_touching_the_device(bnd):
    lib = bnd.lib()
    cfg = bnd.make_cfg(64, 5, 64, 16)
    h = C.c_void_p()
    assert lib.anakin_create(C.byref(cfg), None, 1 << 30, None, C.byref(h)) == bnd.E_INVALID_ARG
    assert lib.anakin_create(C.byref(cfg), C.c_void_p(0x1001), 1 << 30, None, C.byref(h)) == bnd.E_INVALID_ARG  # misaligned
    assert lib.anakin_create(C.byref(cfg), C.c_void_p(0x1000), 16, None, C.byref(h)) == bnd.E_WORKSPACE_TOO_SMALL
    assert lib.anakin_create(C.byref(cfg), C.c_void_p(0x1000), 1 << 30, None, None) == bnd.E_INVALID_ARG
    assert not h.value
    for fn in ("anakin_destroy", "anakin_learn", "anakin_gae", "anakin_update"):
        assert getattr(lib, fn)(None) == bnd.E_INVALID_ARG
    assert lib.anakin_reset(None, 1) == bnd.E_INVALID_ARG
    assert lib.anakin_rollout(None, 4) == bnd.E_INVALID_ARG
    assert lib.anakin_run(None, 1) == bnd.E_INVALID_ARG
    assert lib.anakin_strerror(bnd.E_UNSUPPORTED_CFG) == b"unsupported configuration"
    assert lib.anakin_strerror(12345) == b"unknown error code"


def test_binding_fails_loudly_without_the_library(tmp_path):
    """A missing libanakin.so is an ImportError, never a silent fallback."""
    import shutil
    import subprocess
    import sys

    pkg = tmp_path / "paper_2104_06272_b200"
    pkg.mkdir()
    for f in ("__init__.py", "binding.py"):
        shutil.copy(os.path.join(ROOT, "paper_2104_06272_b200", f), pkg / f)
    r = subprocess.run([sys.executable, "-c", "import paper_2104_06272_b200.binding"], cwd=tmp_path, capture_output=True, text=True)
    assert r.returncode != 0 and "libanakin.so is missing" in r.stderr and "no CPU or PyTorch fallback" in r.stderr
