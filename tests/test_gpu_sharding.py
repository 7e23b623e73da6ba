"""The sharded step on the CUDA path (one GPU standing in for K ranks).

Every shard owns a subset of the list (whole tensors, or block-aligned pieces of tensors), runs the norm
kernel over what it owns into its own scalar, the K scalars are summed (the stand-in for the 8-byte
all-reduce), and every shard runs the step kernel over what it owns with the summed scalar. The result must be
bit-identical to one unsharded step fed the same scalar, and within tolerance of the oracle. One more test
drives ShardedHybrid8.step through a real (single-rank) NCCL process group."""
import os

import numpy as np
import pytest
import torch

import oracle as O
import paper_2608_11919_b200 as L
from paper_2608_11919_b200 import workloads as W
from paper_2608_11919_b200.sharding import ShardedHybrid8, partition_blocks, partition_tensors
from parity_util import NORM_RTOL, compare, oracle_tensors, parallel_oracle_step, refresh_grads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KEYS = ("param", "m_code", "v_code", "m_absmax", "v_absmax")


def _bits(t):
    return t.view(torch.int16 if t.element_size() == 2 else torch.int32) if t.dtype.is_floating_point else t


def _run(world, by_blocks, param_dtype, block=2048, steps=3):
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=160, max_numel=1 << 17, seed=5)
    spec.param_dtype = param_dtype
    whole, shard = W.Buffers(spec, block, DEV), W.Buffers(spec, block, DEV)
    W.fill_params(whole)
    shard.param.copy_(whole.param)
    hp = dict(max_norm=spec.max_norm)
    if by_blocks:
        parts = partition_blocks(spec.sizes, block, world)
        lists = [L.TensorList.from_buffer_pieces(shard, p) for p in parts]
        owned = [sum(min(spec.sizes[t], (b0 + nb) * block) - b0 * block for t, b0, nb in p) for p in parts]
        nblk = [sum(nb for _, _, nb in p) for p in parts]
        assert max(nblk) - min(nblk) <= 1                                   # balanced to one block
    else:
        parts = partition_tensors(spec.sizes, world)
        lists = [L.TensorList.from_buffers(shard, p) for p in parts]
        owned = [sum(spec.sizes[t] for t in p) for p in parts]
    assert sum(owned) == spec.numel
    ranks = [ShardedHybrid8(L.Hybrid8Optimizer(tl, block, L.HParams(**hp), device=torch.device(DEV))) for tl in lists]
    tl_whole = L.TensorList.from_buffers(whole)
    L.lt_hybrid8_state_init(tl_whole, block)
    for r in ranks:
        if r.opt.tensors.n:
            r.opt.init_state()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    W.fill_grads(whole, 1)
    ots, slices = oracle_tensors(whole)
    for k in range(1, steps + 1):
        W.fill_grads(whole, k)
        shard.grad.copy_(whole.grad)
        if k > 1:
            refresh_grads(ots, whole, slices)
        for r in ranks:
            r.norm_phase()
        total = torch.zeros(1, dtype=torch.float64, device=DEV)
        for r in ranks:                                   # the all-reduce: a sum of K scalars
            total += r.opt.sqnorm
        for r in ranks:
            r.opt.sqnorm.copy_(total)
            r.update_phase()
        L.lt_hybrid8_step(tl_whole, block, L.HParams(step=k, **hp), total, status)
        torch.cuda.synchronize()
        for key in KEYS:
            assert torch.equal(_bits(getattr(whole, key)), _bits(getattr(shard, key))), (k, key)
        S = O.sqnorm(ots)
        assert abs(float(total.item()) - S) <= NORM_RTOL * S
        assert parallel_oracle_step(ots, block, O.HParams(step=k, **hp), S) == 0
        compare(shard, ots, slices).check()
    assert int(status.item()) == 0 and all(int(r.opt.status.item()) == 0 for r in ranks)


@pytest.mark.parametrize("world", [2, 3, 8])
def test_shards_of_whole_tensors_equal_the_unsharded_step(world):
    _run(world, False, torch.float32)


@pytest.mark.parametrize("world", [2, 8])
@pytest.mark.parametrize("param_dtype", [torch.float32, torch.bfloat16])
def test_shards_of_block_ranges_equal_the_unsharded_step(world, param_dtype):
    _run(world, True, param_dtype)


def test_sharded_step_through_a_single_rank_nccl_group():
    """ShardedHybrid8.step with its real all-reduce (NCCL, one rank, on the compute stream)."""
    import torch.distributed as dist
    torch.cuda.set_device(0)
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29611")
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(DEV))
    try:
        spec = W.ragged_spec(n_tensors=60, max_numel=1 << 15, seed=6)
        a, b = W.Buffers(spec, 2048, DEV), W.Buffers(spec, 2048, DEV)
        W.fill_params(a)
        b.param.copy_(a.param)
        plain = L.Hybrid8Optimizer(L.TensorList.from_buffers(a), 2048, L.HParams(max_norm=0.5))
        sharded = ShardedHybrid8(L.Hybrid8Optimizer(L.TensorList.from_buffers(b), 2048, L.HParams(max_norm=0.5)))
        plain.init_state()
        sharded.opt.init_state()
        for k in (1, 2):
            W.fill_grads(a, k)
            b.grad.copy_(a.grad)
            plain.step()
            sharded.step()
            torch.cuda.synchronize()
            assert float(plain.sqnorm.item()) == float(sharded.opt.sqnorm.item())
            for key in KEYS:
                assert torch.equal(_bits(getattr(a, key)), _bits(getattr(b, key))), (k, key)
    finally:
        if created:
            dist.destroy_process_group()
