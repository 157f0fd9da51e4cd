#!/usr/bin/env python
"""Benchmark of the Anakin hot path: env frames/s (acting + learning) on the "throughput" workload.

    python bench.py --gpus N --steps K --warmup W            # the CUDA library
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands

One step = one pass of the whole hot path: a T-step rollout of all B envs followed by one A2C/Adam update
(B*T frames).  Prints ONE JSON line.  With N > 1 (torchrun) every rank runs the workload's B envs as one shard of an
N*B-env job: same seed, env offsets rank*B, and one exchange per step, the mean of the gradients (NCCL all-reduce of P
floats) between the backward pass and Adam.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2104_06272_b200.workloads import MANY_POLICIES, ORDER, WORKLOADS  # noqa: E402

METRIC = "env_frames_per_sec_act_plus_learn"
UNIT = "frames/s"
# FP32 FMA peak of a B200: 148 SMs x 128 FMA lanes x 2 FLOP x max SM clock.
FP32_ALU_TFLOPS_PER_MHZ = 148 * 128 * 2 / 1e6


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    sm_max_mhz=float(p.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, sm_max_mhz=1965.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons while the timed region runs: a thread that polls NVML (read-only queries)
    every millisecond, so that even a timed region of a few milliseconds is covered; `nvidia-smi -lms` when NVML's Python
    module is missing."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines, self.samples = index, None, [], []
        self.nvml = self.handle = self.thread = None
        self.stop_flag = threading.Event()

    def _poll(self):
        n = self.nvml
        names = (("hw_slowdown", n.nvmlClocksEventReasonHwSlowdown), ("hw_thermal_slowdown", n.nvmlClocksEventReasonHwThermalSlowdown),
                 ("sw_thermal_slowdown", n.nvmlClocksEventReasonSwThermalSlowdown), ("sw_power_cap", n.nvmlClocksEventReasonSwPowerCap))
        while not self.stop_flag.is_set():
            try:
                sm = n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)
                mask = n.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                self.samples.append((float(sm), [nm for nm, bit in names if mask & bit]))
            except Exception:
                pass
            time.sleep(0.001)

    def start(self):
        try:
            import pynvml as n

            n.nvmlInit()
            # the visible device's index as NVML counts it (CUDA_VISIBLE_DEVICES may renumber)
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            ids = [v for v in vis.split(",") if v.strip()] if vis else []
            ent = ids[self.index] if self.index < len(ids) else str(self.index)
            self.handle = n.nvmlDeviceGetHandleByUUID(ent) if ent.startswith("GPU-") else n.nvmlDeviceGetHandleByIndex(int(ent))
            self.sm_max = float(n.nvmlDeviceGetMaxClockInfo(self.handle, n.NVML_CLOCK_SM))
            self.nvml = n
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.nvml is not None:
            self.stop_flag.set()
            self.thread.join(timeout=5)
            if not self.samples:
                return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["no samples"]}
            reasons = sorted({r for _, rs in self.samples for r in rs})
            return {"sm_mhz": float(np.median([s for s, _ in self.samples])), "sm_max_mhz": self.sm_max, "reasons": reasons,
                    "samples": len(self.samples), "how": "NVML polled every 1 ms during the timed region"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=5)
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons), "samples": len(sm),
                "how": "nvidia-smi -lms 20 during the timed region"}


# Which ncu summary under profiles/ covers a (workload, profiler kernel name) pair, and the source file of that kernel.
# The summary carries the counters (a table row "dram__bytes_read / write | X MB / Y MB") and the SHA-256 of the kernel's
# source file at capture time ("kernel source: <file> sha256 <hex>"); counters of a kernel that has changed since are
# not reported.
PROFILE_OF = {
    ("throughput", "rollout"): ("rollout_pair__throughput.md", "rollout_pair.cu"),
    ("throughput", "dh1"): ("dh1a_pair__throughput.md", "dh1a_tc.cu"),
    ("throughput", "heads_bwd"): ("heads_bwd__throughput.md", "learner_mma.cu"),
    ("throughput", "reduce_adam"): ("reduce_adam2__throughput.md", "learner_mma.cu"),
    ("throughput", "env_base"): ("env_base__throughput.md", "rollout.cu"),
    ("throughput", "dw1_walls"): ("gemm_tn_tc_env_planes__throughput.md", "gemm_tc.cu"),
}


def ncu_traffic_bytes(workload: str, kernel: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu summary, or None when there is no
    summary for this kernel and workload or the kernel's source has changed since the capture."""
    import hashlib
    import re

    ent = PROFILE_OF.get((workload, kernel))
    if ent is None:
        return None
    prof, src = os.path.join(ROOT, "profiles", ent[0]), os.path.join(ROOT, "paper_2104_06272_b200", "csrc", ent[1])
    if not (os.path.exists(prof) and os.path.exists(src)):
        return None
    text = open(prof).read()
    m = re.search(r"dram__bytes_read / write \| ([\d.]+) MB / ([\d.]+) MB", text)
    h = re.search(r"kernel source: \S+ sha256 ([0-9a-f]{64})", text)
    if not m or not h or h.group(1) != hashlib.sha256(open(src, "rb").read()).hexdigest():
        return None
    return (float(m.group(1)) + float(m.group(2))) * 1e6


def workload_label(w):
    pol = f"{w.n_policies} independent policies x {(w.B + w.n_policies - 1) // w.n_policies} envs, " if getattr(w, "n_policies", 0) >= 2 else ""
    return (f"{w.name}: {pol}B={w.B} envs, {w.N}x{w.N} gridworld (obs {w.D}), MLP {w.D}-{w.H}-{w.H}+5, "
            f"{'fp32' if w.precision == 0 else 'bf16'}, T={w.T}")


# ------------------------------------------------------------------------------------------------------
# Kernel work model (algorithmic FLOPs / bytes per launch) for the roofline entry
# ------------------------------------------------------------------------------------------------------
def kernel_work(w):
    """Per launch: which roofline bounds the kernel, the FLOPs it EXECUTES on that pipe (tensor kernels of the fp32
    workloads run three fp16 MMAs per product, two when one operand is an exact 0/1 plane) and its algorithmic HBM
    bytes.  Only work the kernels really do is counted (the one-hot first layer is a gather, not a GEMM)."""
    B, T, H, C, P = w.B, w.T, w.H, w.C, w.P
    R = B * T
    p3 = 1 if w.precision == 1 else 3
    p2 = 1 if w.precision == 1 else 2
    pl = 2 if w.precision == 1 else 4  # bytes per element of a 16-bit operand stored as (hi[, lo]) planes
    work = {
        # name: (bound, executed flops, bytes)
        "rollout": ("tensor", p3 * 2.0 * B * (T + 1) * H * H, R * (15.0 + pl * H + 4.0 * H) + B * 4),
        # fused kernel (H = 128, 256 with at most 128 cells, one policy): also the agent plane of dW1 over 128 padded cells;
        # reads the dh2 planes and one gate bit per element.  Otherwise: dh2 in, 16-bit h1 gates in, dh1 out.
        "dh1": (("tensor", p3 * 2.0 * R * H * H + p2 * 2.0 * R * 128 * H, R * H * (pl + 0.125))
                if H in (128, 256) and C <= 128 and getattr(w, "n_policies", 0) <= 1
                else ("tensor", p3 * 2.0 * R * H * H, R * H * (2.0 * pl + 2.0))),
        "dw2": ("tensor", p3 * 2.0 * R * H * H, R * H * 2.0 * pl),
        "dw1_agent": ("tensor", p2 * 2.0 * R * C * H, R * H * 1.0 * pl + R),
        "dw1_walls": ("tensor", 2 * 2.0 * B * (C + 1) * H, B * H * 4.0),
        "dw1_goal": ("tensor", 2 * 2.0 * B * C * H, B * H * 4.0),
        # hidden width 128 / 256 (one policy): the kernel also takes dW2 = h1^T dh2 on the tensor pipe and reads the h1 planes
        "heads_bwd": (("hbm", R * H * 22.0 + p3 * 2.0 * R * H * H, R * H * (4.0 + 2.0 * pl) + R * 10.0)
                      if H in (128, 256) and getattr(w, "n_policies", 0) <= 1
                      else ("hbm", R * H * 22.0, R * H * (4.0 + pl) + R * 10.0)),
        "gae": ("hbm", R * 6.0, R * 17.0),
        "env_base": ("hbm", B * H * (0.2 * C + 2), B * H * 4.0),
        "pack_w2": ("hbm", 0.0, H * H * 16.0),
        "reduce_adam": ("hbm", P * 12.0, P * 28.0),
        "replay": ("tensor", p3 * 2.0 * R * H * H, R * H * (pl + 4.0)),
    }
    if w.precision == 1 and H in (512, 1024):
        # wide bf16 path: two launches per env step (layer-2 GEMM; heads + env step + next step's h1), bf16 activations in HBM
        work.update({
            "h1": ("hbm", B * H * 2.0, B * H * (4.0 + 2.0) + B),                  # first step only: base fp32 in, h1 bf16 out
            "fwd2": ("tensor", 2.0 * B * H * H, B * H * 4.0 + H * H * 2.0),       # per step: h1 in, h2 out, W2
            "rollout": ("hbm", B * H * 12.0, B * H * 8.0 + B * 47.0),             # per step: h2 in, records out; base in, next h1 out
            "heads_bwd": ("hbm", R * H * 22.0, R * H * 4.0 + R * 42.0),           # h2 in, dh2 out (bf16 each)
            "dh1": ("tensor", 2.0 * R * H * H, R * H * 6.0),                      # dh2 in, h1 gates in, dh1 out
            "sum_over_t": ("hbm", R * H * 1.0, R * H * 2.0 + B * H * 4.0),
            "dw2": ("tensor", 2.0 * R * H * H, R * H * 4.0),
            "dw1_agent": ("tensor", 2.0 * R * C * H, R * H * 2.0 + R),
            "env_base": ("tensor", 2.0 * B * C * H, B * H * 4.0 + B * C * 2.0),   # two launches: operand expansion + GEMM
        })
    return work


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """The slowest rank's value (the time every multi-GPU number is reported on).  Works on any backend: the tensor
    lives on `device` ("cuda" under NCCL, "cpu" under gloo)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist

    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_frames_per_sec(frames_per_rank: float, world: int, max_seconds: float) -> float:
    """Every rank processes frames_per_rank frames of its own shard; the job's rate is the sum over ranks divided by
    the slowest rank's time."""
    return frames_per_rank * world / max_seconds


def time_steps(an, run_steps, w, K, W, stream, flush, barrier, rank, local_rank, world):
    """W untimed steps, then K steps each bracketed by CUDA events on the library's stream with the L2 flushed between
    them (outside the brackets), clocks sampled meanwhile; then the same K steps once more with events around every
    kernel launch.  Returns (frames/s over all ranks, total ms (max over ranks), launches, clocks, per-kernel times,
    wall seconds of the timed region)."""
    import torch

    run_steps(W)
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    n0 = an.launch_count()
    barrier()
    t_wall0 = time.perf_counter()
    with torch.cuda.stream(stream):
        for a, b in ev:
            flush.fill_(0)
            a.record(stream)
            run_steps(1)
            b.record(stream)
    barrier()
    t_wall = time.perf_counter() - t_wall0
    launches = an.launch_count() - n0
    clocks = sampler.stop() if rank == 0 else None
    step_ms = [a.elapsed_time(b) for a, b in ev]
    total_ms = max_over_ranks(float(sum(step_ms)), world, "cuda")
    value = whole_job_frames_per_sec(float(w.B) * w.T * K, world, total_ms * 1e-3)
    an.profile_enable(True)
    with torch.cuda.stream(stream):
        for _ in range(K):
            flush.fill_(0)
            run_steps(1)
    prof = an.profile_read()
    an.profile_enable(False)
    return value, total_ms, launches, clocks, prof, t_wall


def roofline_of(w, prof, K, peaks, clocks):
    """Roofline entry of the dominant kernel (largest total time in the per-kernel pass) plus one line per kernel.
    Tensor kernels: executed FLOPs / duration against the measured cuBLAS bf16 figure -- the burst figure when the SM
    clock stayed near its maximum during the timed region (short kernels, no power cap), the sustained one otherwise;
    both fractions are printed."""
    work = kernel_work(w)
    tot = sum(ms for ms, _ in prof.values())

    def kernel_line(k, ms, n):
        line = {"us_per_launch": ms / n * 1e3, "launches_per_step": n / K, "share": ms / tot}
        if k in work:
            bnd_, fl, by = work[k]
            sec = ms / n * 1e-3
            line["bound"] = bnd_
            line["tflops"] = fl / sec / 1e12
            line["gbs"] = by / sec / 1e9
        return line

    top = max(prof, key=lambda k: prof[k][0])
    top_ms, top_n = prof[top]
    bound, flops, nbytes = work.get(top, ("hbm", 0.0, 0.0))
    per_launch_s = top_ms / top_n * 1e-3
    sm_max = (clocks or {}).get("sm_max_mhz") or peaks["sm_max_mhz"]
    sm_now = (clocks or {}).get("sm_mhz") or sm_max
    extra = {}
    if bound == "alu":
        achieved, peak, unit = flops / per_launch_s / 1e12, FP32_ALU_TFLOPS_PER_MHZ * sm_max, "TFLOP/s"
        peak_note = f"fp32 FMA peak = 148 SMs x 128 lanes x 2 x {sm_max:.0f} MHz (derived)"
    elif bound == "tensor":
        achieved, unit = flops / per_launch_s / 1e12, "TFLOP/s"
        at_full_clock = sm_now >= 0.9 * sm_max
        peak = peaks["bf16_tflops"] if at_full_clock else peaks["bf16_tflops_sustained"]
        extra = {"frac_of_burst": achieved / peaks["bf16_tflops"], "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"]}
        peak_note = (f"dense 16-bit tensor throughput (cuBLAS bf16, {'burst: SM clock at ' if at_full_clock else 'sustained: SM clock at '}"
                     f"{sm_now:.0f} of {sm_max:.0f} MHz during the timed region), {peaks['source']}; achieved counts executed FLOPs "
                     "(3 fp16 MMAs per fp32 product)")
    else:
        achieved, peak, unit = nbytes / per_launch_s / 1e9, peaks["hbm_gbs"], "GB/s"
        peak_note = f"HBM copy bandwidth, {peaks['source']}"
    base_name = w.name.split("[")[0]
    out = {"kernel": top, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
           "traffic": ncu_traffic_bytes(base_name, top) if base_name == w.name else None, "peak_source": peak_note,
           "us_per_launch": per_launch_s * 1e6, "share_of_step": top_ms / tot,
           "kernels": {k: kernel_line(k, ms, n) for k, (ms, n) in sorted(prof.items(), key=lambda kv: -kv[1][0])}}
    out.update(extra)
    return out


def time_other_workload(bnd, w, stream, flush, local_rank, peaks, seed, K=4, W=3):
    """A short device-timed run of another workload (same event / flush method as the headline), for the per-workload
    table: frames/s, ms per step, clocks of that segment, the dominant kernel and its roofline fraction."""
    import torch

    with torch.cuda.stream(stream):
        an = bnd.Anakin(bnd.cfg_from_workload(w, device=local_rank), stream=stream)
    an.reset(seed)
    value, total_ms, launches, clocks, prof, _ = time_steps(an, an.run, w, K, W, stream, flush, torch.cuda.synchronize, 0, local_rank, 1)
    st = an.stats()
    ok = an.status() == 0 and bool(np.isfinite([s.loss_total for s in (st if isinstance(st, list) else [st])]).all())
    rl = roofline_of(w, prof, K, peaks, clocks)
    del an
    torch.cuda.empty_cache()
    return {"workload": workload_label(w), "value": value, "unit": UNIT, "ms_per_step": total_ms / K, "steps": K, "warmup": W,
            "dtype": "bf16" if w.precision == 1 else "f32", "gpu_launches": int(launches), "clocks": clocks, "status_ok": ok,
            "roofline": rl}


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2104_06272_b200 import binding as bnd

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("launch with torchrun --nproc-per-node N for --gpus N")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    w = MANY_POLICIES if args.workload == MANY_POLICIES.name else WORKLOADS[args.workload]
    if args.envs:  # reduced batch for profiler captures; such a run is not a bench line of the named workload
        w = w.scaled(name=f"{w.name}[B={args.envs}]", B=args.envs)
    peaks = load_peaks()
    stream = torch.cuda.Stream()
    seed = 1
    if world > 1:
        from paper_2104_06272_b200 import replicas

        with torch.cuda.stream(stream):
            rep = replicas.ReplicatedAnakin(w.scaled(B=w.B * world), rank, world, device=local_rank, stream=stream)
        an = rep.an
        rep.reset(seed)

        def run_steps(n):
            rep.run(n)
    else:
        with torch.cuda.stream(stream):
            an = bnd.Anakin(bnd.cfg_from_workload(w, device=local_rank), stream=stream)
        an.reset(seed)

        def run_steps(n):
            an.run(n)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")  # > 126 MB L2

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    K, W = args.steps, args.warmup
    value, total_ms, launches, clocks, prof, t_wall = time_steps(an, run_steps, w, K, W, stream, flush, barrier, rank, local_rank, world)

    # ---- end to end through the C ABI with host buffers: per step, parameters and env state go host->device
    # from pinned memory, one act+learn pass runs, statistics and parameters come back
    P = an.blob_bytes(bnd.PARAMS) // 4  # (all policies' parameters when there are many)
    h_theta = torch.from_numpy(an.get(bnd.PARAMS)).pin_memory()
    h_pos = torch.from_numpy(an.get(bnd.ENV_POS)).pin_memory()
    h_tep = torch.from_numpy(an.get(bnd.ENV_TEP)).pin_memory()
    h_out = torch.empty(P, dtype=torch.float32).pin_memory()
    Ke = max(3, min(K, 20))
    sb = an.blob_bytes(bnd.STATS)
    h_stats = torch.zeros((Ke, sb), dtype=torch.uint8).pin_memory()

    def e2e_pass(i, sync_each_step):
        nonlocal h_theta, h_out
        an.set(bnd.PARAMS, h_theta)
        an.set(bnd.ENV_POS, h_pos)
        an.set(bnd.ENV_TEP, h_tep)
        run_steps(1)
        an.get_into(bnd.PARAMS, h_out, wait=False)   # device -> pinned host, enqueued behind the pass
        an.get_into(bnd.ENV_POS, h_pos, wait=False)
        an.get_into(bnd.ENV_TEP, h_tep, wait=False)
        an.get_into(bnd.STATS, h_stats[i], wait=False)  # this step's losses and counters, in their own slot
        if sync_each_step:
            stream.synchronize()
        h_theta, h_out = h_out, h_theta              # the parameters that came back are the next step's input

    def e2e_loop(sync_each_step):
        barrier()
        t0 = time.perf_counter()
        for i in range(Ke):
            e2e_pass(i, sync_each_step)
        barrier()  # (synchronises the device: every copy of every step has landed)
        dt = max_over_ranks(time.perf_counter() - t0, world, "cuda")
        return whole_job_frames_per_sec(float(w.B) * w.T * Ke, world, dt)

    # (a) the host waits for every step's results before it submits the next step; (b) the host only enqueues: a step's
    # host->device copies are ordered behind the previous step's device->host copies by the stream, so the loop is the same
    # computation without the host's turnaround between steps.  (b) is the reported value, (a) is printed beside it.
    e2e_sync = e2e_loop(True)
    e2e_value = e2e_loop(False)
    rec = C.sizeof(bnd.AnakinStats)  # one record per policy: four counters, then the four loss terms as floats
    losses = h_stats.numpy().reshape(Ke, -1, rec)[:, :, rec - 16:].copy().view(np.float32)
    assert np.isfinite(losses).all() and h_stats.any(dim=1).all() and an.status() == 0

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    roofline = roofline_of(w, prof, K, peaks, clocks)

    # ---- the other workloads, device-timed the same way (short runs): one entry each
    others = None
    if world == 1 and not args.envs and not args.no_workloads and args.workload == "throughput":
        others = {}
        for name in ORDER:
            if name == args.workload:
                continue
            others[name] = time_other_workload(bnd, WORKLOADS[name], stream, flush, local_rank, peaks, seed)
        others[MANY_POLICIES.name] = time_other_workload(bnd, MANY_POLICIES, stream, flush, local_rank, peaks, seed)

    # ---- the oracle on the host cores, bounded sample of the same workload (about 10-30 s of CPU work)
    if args.no_cpu_baseline or rank != 0:
        cpu = None
    elif args.workload == "throughput" and not args.envs:
        cpu = cpu_baseline(w, iters=6)
    else:
        mac_per_frame = 3.0 * (w.D * w.H + w.H * w.H + 5 * w.H) + w.H * w.H
        frames = 5.0e11 / mac_per_frame
        cpu = cpu_baseline(w, iters=1, B=int(max(16, min(w.B, frames / w.T))))

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.precision == 1 else "f32", "data": "synthetic",
        "config": {"workload": workload_label(w), "frames_per_step": w.B * w.T, "seed": seed,
                   "l2": "flushed between timed steps (256 MiB write outside the event brackets)",
                   "multi_gpu": (f"{world} replicas of B envs each (one job of {world * w.B} envs), gradients averaged with one NCCL "
                                 "all-reduce per step" if world > 1 else "single GPU")},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": P * 4 + 2 * w.B, "d2h_bytes_per_step": P * 4 + 2 * w.B + an.blob_bytes(bnd.STATS),
                "steps": Ke, "value_sync_each_step": e2e_sync,
                "what": ("per step: set(PARAMS, ENV_POS, ENV_TEP) from pinned host, run(1), get(STATS, PARAMS, ENV_POS, ENV_TEP) into pinned "
                         "host buffers, all enqueued on the handle's stream, one synchronisation after the last step (each step's "
                         "inputs are the previous step's outputs, ordered by the stream); value_sync_each_step: the same with the "
                         "host waiting for every step's results before it submits the next")},
        "gpu_launches": int(launches),
        "wall_s_timed_region": t_wall,
        "roofline": roofline,
        "cpu_baseline": cpu,
    }
    if others is not None:
        out["workloads"] = others
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def cpu_baseline(w, iters: int, B: int | None = None):
    """Times the oracle, as it stands, on `iters` act+learn passes of the workload (optionally on a reduced batch)."""
    from oracle import binding as orc

    Bs = w.B if B is None else B
    ag = orc.Agent(Bs, w.N, w.H, w.T, w.precision, w.episode_cap, w.wall_density, w.gamma, w.gae_lambda, w.entropy_coef,
                   w.value_coef, w.lr, w.adam_b1, w.adam_b2, w.adam_eps)
    ag.reset(1)
    t0 = time.perf_counter()
    ag.run(iters)
    dt = time.perf_counter() - t0
    return {"value": Bs * w.T * iters / dt, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"{iters} full act+learn passes of B={Bs}, T={w.T} ({Bs * w.T * iters} frames, {dt:.1f} s)"}


def run_reference(args):
    """The reference arm is the CPU oracle: each step is one act+learn pass on a quarter of the batch."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import binding as orc

    w = WORKLOADS["throughput"]
    Bs = w.B // 4
    ag = orc.Agent(Bs, w.N, w.H, w.T, w.precision, w.episode_cap, w.wall_density, w.gamma, w.gae_lambda, w.entropy_coef,
                   w.value_coef, w.lr, w.adam_b1, w.adam_b2, w.adam_eps)
    ag.reset(1)
    K, W = args.steps, args.warmup
    ag.run(W)
    t0 = time.perf_counter()
    ag.run(K)
    dt = time.perf_counter() - t0
    value = Bs * w.T * K / dt
    sample = f"each step = one act+learn pass on B={Bs} of the workload's {w.B} envs, T={w.T}"
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K, "warmup": W,
        "ms_per_step": dt / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": {"workload": workload_label(w), "frames_per_step": Bs * w.T, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiler captures only)")
    ap.add_argument("--no-workloads", action="store_true", help="skip the short runs of the other four workloads")
    ap.add_argument("--envs", type=int, default=0, help="override the workload's number of envs (small profiler captures only)")
    ap.add_argument("--workload", default="throughput", choices=list(WORKLOADS) + [MANY_POLICIES.name],
                    help="the metric is quoted on 'throughput'; the others are for the per-workload table")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
