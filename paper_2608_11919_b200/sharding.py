"""Multi-GPU form of the step: tensors are owned by ranks (whole tensors, so quantization blocks never
straddle ranks) and the only exchange is a sum all-reduce of the 8-byte squared gradient norm between
the norm kernel and the step kernel. Host-side plumbing only (no arithmetic of the method)."""
from __future__ import annotations

from typing import List, Sequence

import torch


def partition_tensors(sizes: Sequence[int], world: int) -> List[List[int]]:
    """Deterministic balanced partition of tensor indices over `world` ranks (largest first onto the
    least loaded rank; ties to the lower rank). Every index appears exactly once; ranks keep list order."""
    assert world >= 1
    load = [0] * world
    out: List[List[int]] = [[] for _ in range(world)]
    for i in sorted(range(len(sizes)), key=lambda k: (-int(sizes[k]), k)):
        r = min(range(world), key=lambda k: (load[k], k))
        out[r].append(i)
        load[r] += int(sizes[i])
    return [sorted(x) for x in out]


def allreduce_sqnorm(sqnorm: torch.Tensor, group=None) -> None:
    """Sum the per-rank squared norms in place (one fp64 element). On CUDA tensors this is enqueued on
    the current stream by NCCL, so it sits between the norm and the step without a host sync."""
    assert sqnorm.dtype == torch.float64 and sqnorm.numel() == 1
    if torch.distributed.is_available() and torch.distributed.is_initialized() and \
            torch.distributed.get_world_size(group) > 1:
        torch.distributed.all_reduce(sqnorm, op=torch.distributed.ReduceOp.SUM, group=group)


class ShardedHybrid8:
    """One rank's optimizer over the tensors it owns: norm (local) -> all-reduce -> step (local)."""

    def __init__(self, optimizer, group=None):
        self.opt, self.group = optimizer, group

    def step(self) -> None:
        from . import binding as B
        o = self.opt
        o.t += 1
        o.hp.step = o.t
        o.sqnorm.zero_()
        for ch in o.chunks:
            B.lt_grad_sqnorm_multi(ch, o.sqnorm, o.workspace)
        allreduce_sqnorm(o.sqnorm, self.group)
        for ch in o.chunks:
            B.lt_hybrid8_step(ch, o.block, o.hp, o.sqnorm, o.status)
