"""Replicated Anakin (Podracer paper, Section 3.1; Figure 2, bottom): every device runs the same minimal unit on its
own slice of the environments, and the one exchange per iteration is the mean of the gradients before the optimizer
step.  One process per GPU; `torch.distributed` carries the all-reduce (NCCL on GPUs).

Rank r of G owns envs [r*B/G, (r+1)*B/G): its handle is created with env_offset = r*B/G, so the G shards hold exactly
the envs of one B-env handle and, with equal shard sizes, the mean of the shard gradients is the full-batch gradient
(up to summation order).  Parameters start identical (they are a function of the seed alone) and stay identical
because every rank applies the same averaged gradient.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding as bnd


def shard_of(B: int, rank: int, world: int) -> tuple[int, int]:
    """(env_offset, local B) of a rank; the batch must divide evenly so that the mean of means is the mean."""
    if B % world != 0:
        raise ValueError(f"B={B} envs do not divide over {world} replicas")
    return rank * (B // world), B // world


def sum_over_replicas_(flat: torch.Tensor, group=None, always: bool = False) -> int:
    """In-place SUM of a tensor over the ranks of `group` (one all-reduce); returns the group size, by which the
    consumer divides (the library does that inside its Adam kernel: `apply_grads(n_replicas)`).  `always` runs the
    collective even in a group of one (to exercise the backend)."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world > 1 or (always and dist.is_initialized()):
        dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    return world


class ReplicatedAnakin:
    """A rank's shard of a B-env Anakin job.  run(iters) = iters x (rollout, local gradient, mean over replicas, Adam)."""

    def __init__(self, workload, rank: int, world: int, device: int = 0, stream: torch.cuda.Stream | None = None, group=None,
                 debug_logits: int = 0, always_exchange: bool = False):
        self.rank, self.world, self.group, self.always_exchange = rank, world, group, always_exchange
        off, b_local = shard_of(workload.B, rank, world)
        self.shard = workload.scaled(B=b_local)
        self.an = bnd.Anakin(bnd.cfg_from_workload(self.shard, device=device, debug_logits=debug_logits, env_offset=off), stream=stream)
        self.gbuf = torch.empty(self.an.P, dtype=torch.float32, device=self.an.device)

    def reset(self, seed: int):
        self.an.reset(seed)  # the same seed on every rank: identical parameters, disjoint env counters

    def iteration(self):
        an = self.an
        an.rollout()
        an.grads()
        n = 1
        if self.world > 1 or self.always_exchange:
            with torch.cuda.stream(an.stream):  # the copies, the collective and Adam are ordered on the handle's stream
                an.get_into(bnd.GRADS, self.gbuf)
                n = sum_over_replicas_(self.gbuf, self.group, self.always_exchange)
                an.set(bnd.GRADS, self.gbuf)
        an.apply_grads(n)  # the division by the number of replicas happens in the Adam kernel

    def run(self, iters: int):
        for _ in range(iters):
            self.iteration()
