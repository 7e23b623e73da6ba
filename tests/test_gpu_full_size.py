"""Parity at the benchmark's full sizes (3B, 7B, 27B-shaped lists) in the launch configuration
`bench.py` times: five GPU steps populate the state, then one more GPU step is compared against the
oracle on sampled whole quantization blocks (every small tensor entirely; first, last and random
blocks of every large tensor). The oracle's norm is its own fp64 sum over ALL gradients, streamed
through the host. The full Ragged configuration (1000 tensors up to 4M elements, 10 free-running steps)
is compared on every element after every step."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2608_11919_b200 as L
from paper_2608_11919_b200 import workloads as W
from parity_util import (NORM_RTOL, compare, oracle_sqnorm_of_buffers, oracle_tensors, parallel_oracle_step,
                         refresh_grads)

import bench

pytestmark = pytest.mark.gpu
WARM_STEPS = 5


def sample_slices(spec, block, rng, per_tensor_blocks=24, small=1 << 16):
    out = []
    for t, size in enumerate(spec.sizes):
        nb = (size + block - 1) // block
        if size <= small:
            out.append((t, 0, None))
            continue
        picks = {0, nb - 1} | set(int(x) for x in rng.integers(0, nb, per_tensor_blocks))
        runs = sorted(picks)
        out.append((t, runs[0], 2))                     # first two blocks
        out.append((t, max(nb - 2, 0), 2))              # last two (the tail may be ragged)
        for b in runs[1:-1]:
            out.append((t, b, 1))
    return out


def run_full_size(name, block):
    torch.cuda.set_device(0)
    need = {"3b": 30e9, "7b": 70e9, "27b": 170e9}[name]
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip(f"{name}: needs {need / 1e9:.0f} GB of device memory, {free / 1e9:.0f} GB free")
    spec, buf, opt = bench.build_workload(name, block, torch.device("cuda:0"))
    for k in range(1, WARM_STEPS + 1):
        W.fill_grads(buf, k)
        opt.step()
    torch.cuda.synchronize()
    assert int(opt.status.item()) == 0
    rng = np.random.default_rng(1234)
    slices = sample_slices(spec, block, rng)
    W.fill_grads(buf, WARM_STEPS + 1)
    ots, slices = oracle_tensors(buf, slices=slices)     # state after the warm-up + this step's gradients
    opt.step()
    torch.cuda.synchronize()
    S_gpu = float(opt.sqnorm.item())
    S = oracle_sqnorm_of_buffers(buf)
    assert abs(S_gpu - S) <= NORM_RTOL * S, (S_gpu, S)
    ohp = O.HParams(max_norm=spec.max_norm, step=WARM_STEPS + 1)
    assert parallel_oracle_step(ots, block, ohp, S) == 0
    st = compare(buf, ots, slices)
    st.norm_rel = abs(S_gpu - S) / S
    print(name, block, "norm rel", st.norm_rel, st)
    st.check()
    assert st.n >= 2 * 10_000_000
    del opt, buf
    torch.cuda.empty_cache()


@pytest.mark.parametrize("block", [2048, 4096])
def test_3b_sampled_parity(block):
    run_full_size("3b", block)


def test_7b_sampled_parity():
    run_full_size("7b", 2048)


def test_27b_sampled_parity_chunked_bf16():
    run_full_size("27b", 2048)


def test_ragged_full_ten_steps_every_element():
    """The full Ragged configuration: 1000 tensors packed back to back (element-aligned bases), about 2.7e8
    elements, ten free-running steps; every element of every tensor is compared after every step (the oracle
    is fanned out over host threads, one tensor per call)."""
    torch.cuda.set_device(0)
    block = 2048
    spec = W.ragged_spec()                               # 1000 tensors, sizes up to 4M, seed 1
    buf = W.Buffers(spec, block, "cuda:0")
    W.fill_params(buf)
    tl = L.TensorList.from_buffers(buf)
    opt = L.Hybrid8Optimizer(tl, block, L.HParams(max_norm=spec.max_norm))
    opt.init_state()
    W.fill_grads(buf, 1)
    ots, slices = oracle_tensors(buf)
    assert sum(t.numel for t in ots) == spec.numel
    ohp = O.HParams(max_norm=spec.max_norm)
    for k in range(1, spec.steps + 1):
        if k > 1:
            W.fill_grads(buf, k)
            refresh_grads(ots, buf, slices)
        opt.step()
        torch.cuda.synchronize()
        S_gpu, S = float(opt.sqnorm.item()), O.sqnorm(ots)
        assert abs(S_gpu - S) <= NORM_RTOL * S
        ohp.step = k
        assert parallel_oracle_step(ots, block, ohp, S) == 0
        st = compare(buf, ots, slices)
        st.check()
    print("ragged full:", spec.numel, "elements in", len(ots), "tensors, all compared on", spec.steps, "steps", st)
    assert st.n == 2 * spec.numel
    assert int(opt.status.item()) == 0


def test_single_tensor_beyond_two_to_the_31_elements():
    """Index arithmetic at the top of the range: one tensor of 2^31 + 6161 elements (8.6 GB of fp32
    parameters, a ragged last block), compared on blocks at the start, around the 2^30 / 2^31 element marks
    (the 2^32-byte marks of the fp32 and bf16 arrays and the 2^31-byte mark of the code arrays) and at the end."""
    torch.cuda.set_device(0)
    free, _ = torch.cuda.mem_get_info()
    if free < 24e9:
        pytest.skip("needs 24 GB of device memory")
    block = 2048
    n = (1 << 31) + 3 * block + 17
    spec = W.Spec("huge", ["w"], [n], [-1], torch.float32, seed=31, grad_std=1e-4, grad_kind="normal",
                  max_norm=1.0, steps=1, align_elems=16)
    buf = W.Buffers(spec, block, "cuda:0")
    W.fill_params(buf)
    tl = L.TensorList.from_buffers(buf)
    opt = L.Hybrid8Optimizer(tl, block, L.HParams(max_norm=1.0))
    opt.init_state()
    for k in (1, 2):
        W.fill_grads(buf, k)
        opt.step()
    nb = (n + block - 1) // block
    marks = [0, (1 << 30) // block - 1, (1 << 31) // block - 2, nb - 3]
    slices = [(0, b, 3) for b in marks]
    W.fill_grads(buf, 3)
    ots, slices = oracle_tensors(buf, slices=slices)
    opt.step()
    torch.cuda.synchronize()
    S_gpu, S = float(opt.sqnorm.item()), oracle_sqnorm_of_buffers(buf)
    assert abs(S_gpu - S) <= NORM_RTOL * S
    assert parallel_oracle_step(ots, block, O.HParams(max_norm=1.0, step=3), S) == 0
    st = compare(buf, ots, slices)
    print("huge tensor:", st)
    st.check()
    assert ots[-1].numel == 2 * block + 17                      # the ragged tail was among the compared blocks
