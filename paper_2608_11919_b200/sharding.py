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


def partition_contiguous(sizes: Sequence[int], world: int) -> List[range]:
    """Splits the tensor list into `world` consecutive runs of near-equal element counts (run r ends at
    the tensor boundary closest to r+1 world-ths of the total; runs may be empty when there are fewer
    tensors than ranks). With tensors packed back to back, each rank then owns ONE contiguous slice of
    the flat parameter buffer, which is what `allgather_params` exchanges."""
    assert world >= 1
    total = sum(int(x) for x in sizes)
    cum, acc = [0], 0
    for x in sizes:
        acc += int(x)
        cum.append(acc)
    cuts = [0]
    for r in range(1, world):
        target = total * r / world
        j = min(range(cuts[-1], len(sizes) + 1), key=lambda k: (abs(cum[k] - target), k))
        cuts.append(j)
    cuts.append(len(sizes))
    return [range(cuts[r], cuts[r + 1]) for r in range(world)]


def partition_blocks(sizes: Sequence[int], block: int, world: int) -> List[List[tuple]]:
    """Balanced partition by QUANTIZATION BLOCKS rather than whole tensors: the list is read as one sequence
    of blocks (tensor after tensor) and cut into `world` consecutive runs whose block counts differ by at most
    one. Returns, per rank, pieces (tensor index, first block, number of blocks) in list order; a tensor that
    straddles a cut is split at a block boundary, which changes nothing in the result because blocks are
    independent once the global norm is known. This removes the imbalance a large embedding causes when whole
    tensors are the unit (a tied 3B embedding is 10 % of the model)."""
    assert world >= 1 and block >= 1
    nbs = [(int(x) + block - 1) // block for x in sizes]
    total = sum(nbs)
    out: List[List[tuple]] = [[] for _ in range(world)]
    t, used = 0, 0                       # next tensor, blocks of it already handed out
    for r in range(world):
        want = total * (r + 1) // world - total * r // world
        while want > 0 and t < len(nbs):
            take = min(want, nbs[t] - used)
            if take > 0:
                out[r].append((t, used, take))
                used += take
                want -= take
            if used == nbs[t]:
                t, used = t + 1, 0
    return out


def allgather_params(param_flat: torch.Tensor, bounds: Sequence[Sequence[int]], group=None) -> None:
    """For replicated parameters: after the step every rank has updated only the slice it owns;
    `bounds[r] = (begin, end)` is rank r's element range of `param_flat`. Each slice is broadcast from
    its owner into the same place on every other rank (each GPU receives into its own memory; plain
    NCCL, no peer loads in any kernel of this library). Slices may be empty or of different lengths."""
    if not (torch.distributed.is_available() and torch.distributed.is_initialized()):
        return
    world = torch.distributed.get_world_size(group)
    if world == 1:
        return
    assert len(bounds) == world
    work = []
    for r, (a, b) in enumerate(bounds):
        if b > a:
            src = torch.distributed.get_global_rank(group, r) if group is not None else r
            work.append(torch.distributed.broadcast(param_flat[a:b], src=src, group=group, async_op=True))
    for w in work:
        w.wait()


def allreduce_sqnorm(sqnorm: torch.Tensor, group=None) -> None:
    """Sum the per-rank squared norms in place (one fp64 element). On CUDA tensors this is enqueued on
    the current stream by NCCL, so it sits between the norm and the step without a host sync."""
    assert sqnorm.dtype == torch.float64 and sqnorm.numel() == 1
    if torch.distributed.is_available() and torch.distributed.is_initialized() and \
            torch.distributed.get_world_size(group) > 1:
        torch.distributed.all_reduce(sqnorm, op=torch.distributed.ReduceOp.SUM, group=group)


class ShardedHybrid8:
    """One rank's optimizer over the tensors it owns: norm (local) -> all-reduce -> step (local).

    `optimizer` is a Hybrid8Optimizer over this rank's tensors only. The step is split in its two phases
    so that a caller without a process group (several shards driven by one process, as in the one-GPU
    tests) can put its own reduction between them: norm_phase() of every shard, then reduce, then
    update_phase() of every shard."""

    def __init__(self, optimizer, group=None):
        self.opt, self.group = optimizer, group

    def norm_phase(self) -> None:
        """S1 over the owned tensors: opt.sqnorm = this rank's partial sum of squares."""
        from . import binding as B
        o = self.opt
        o.t += 1
        o.hp.step = o.t
        o.sqnorm.zero_()
        for ch in o.chunks:
            B.lt_grad_sqnorm_multi(ch, o.sqnorm, o.workspace)

    def update_phase(self) -> None:
        """S2..S5 over the owned tensors; opt.sqnorm must hold the global sum by now."""
        from . import binding as B
        o = self.opt
        B.lt_skip_count_update(o.sqnorm, o.skip_count)
        for ch in o.chunks:
            B.lt_hybrid8_step(ch, o.block, o.hp, o.sqnorm, o.status)

    def step(self) -> None:
        self.norm_phase()
        allreduce_sqnorm(self.opt.sqnorm, self.group)
        self.update_phase()
