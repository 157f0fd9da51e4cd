"""The five synthetic workloads and seeded input generators shared by the tests, the benchmark and the
CPU checker.  This module holds sizes, hyper-parameters and plain random draws only: none of the
method's arithmetic lives here.

The Podracer paper describes Anakin's workload only as small networks on grid-world environments
(Section 4.1); it names no dataset.  These presets are the stand-in: every input (walls, start and
goal cells, initial weights, action noise) is generated from one integer seed.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int  # environments
    N: int  # grid side
    H: int  # hidden width
    T: int  # rollout length
    iters: int
    precision: int = 0  # 0 = fp32, 1 = bf16 inputs / fp32 accumulate / fp32 master params
    episode_cap: int = 50
    wall_density: float = 0.2
    gamma: float = 0.99
    gae_lambda: float = 0.95
    entropy_coef: float = 0.01
    value_coef: float = 0.5
    lr: float = 3e-4
    adam_b1: float = 0.9
    adam_b2: float = 0.999
    adam_eps: float = 1e-8
    env_kind: int = 0  # 0 = gridworld (borders block), 1 = torus (borders wrap around)
    n_policies: int = 0  # 0 or 1 = one policy; K >= 2 = K independent networks, policy p on envs [p*ceil(B/K), ...)

    @property
    def C(self):
        return self.N * self.N

    @property
    def D(self):
        return 3 * self.C

    @property
    def P(self):
        return self.D * self.H + self.H + self.H * self.H + self.H + 5 * self.H + 5

    @property
    def frames_per_iter(self):
        return self.B * self.T

    def scaled(self, **kw) -> "Workload":
        d = asdict(self)
        d.update(kw)
        return Workload(**d)


WORKLOADS = {
    "tiny": Workload("tiny", B=64, N=5, H=64, T=16, iters=2),
    "throughput": Workload("throughput", B=4096, N=10, H=256, T=32, iters=100),
    "memory_bound": Workload("memory_bound", B=131072, N=8, H=128, T=64, iters=20),
    "large_batch": Workload("large_batch", B=65536, N=10, H=256, T=32, iters=50),
    "tensor_core": Workload("tensor_core", B=16384, N=16, H=1024, T=32, iters=20, precision=1),
}
ORDER = ["tiny", "throughput", "memory_bound", "large_batch", "tensor_core"]
# The many-policies shape (Section 4.1 of the paper describes a meta-learning run with 1K policies on 60K environments):
# 1024 independent small networks with 64 envs each.  Not one of the five headline workloads; benchmarked as an extra.
MANY_POLICIES = Workload("many_policies", B=65536, N=5, H=64, T=16, iters=20, n_policies=1024)


def forced_actions(seed: int, T: int, B: int) -> np.ndarray:
    """Uniform random actions in {0,1,2,3}, int8 [T][B], for driving both sides with one sequence."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, 4, size=(T, B), dtype=np.int8)


def random_params(seed: int, P: int, scale: float = 0.3) -> np.ndarray:
    """Dense random fp32 parameter vector (biases included), for tests that need non-zero biases."""
    rng = np.random.default_rng(seed)
    return (rng.standard_normal(P) * scale).astype(np.float32)
