"""Seeded random configurations (block size, tensor sizes and alignment, parameter / gradient / state types,
hyper-parameters, gradient scale, number of steps, chunking of the list) against the oracle. Every step is compared from identical
inputs: after each comparison the oracle takes over the GPU's parameters (the state has to be identical
anyway), so a one-ulp difference that the tolerance allows at one step cannot be magnified by a later step
that shrinks the parameter."""
import numpy as np
import pytest
import torch

from paper_2608_11919_b200 import workloads as W
from test_gpu_parity import run_free

pytestmark = pytest.mark.gpu


def make_case(case: int, bf16_params=None, lr_max_exp: float = -3.0, extreme: bool = False):
    rng = np.random.default_rng(1000 + case)
    block = int(rng.choice([256, 512, 1024, 2048, 2048, 4096, 4096, 8192, 16384]))
    nt = int(rng.integers(1, 120))
    mult = int(rng.choice([block, 4, 8, 16, 2048]))
    spec = W.ragged_spec(n_tensors=nt, max_numel=int(rng.choice([1 << 12, 1 << 15, 1 << 17, 1 << 19])), seed=case,
                         multiple=mult)
    bf16 = rng.uniform() < 0.5
    spec.param_dtype = torch.bfloat16 if (bf16 if bf16_params is None else bf16_params) else torch.float32
    spec.grad_dtype = torch.float32 if rng.uniform() < 0.25 else torch.bfloat16
    spec.align_elems = int(rng.choice([1, 1, 2, 4, 8, 16]))
    if rng.uniform() < 0.4:
        spec.state_f32 = [bool(rng.uniform() < 0.5) for _ in spec.sizes]
    spec.grad_std = float(10.0 ** (rng.uniform(-12, 4) if extreme else rng.uniform(-6, 0)))
    spec.max_norm = float(rng.choice([0.5, 1.0, 1e-3, 100.0]))
    if extreme:
        hp = dict(lr=float(10.0 ** rng.uniform(-6, lr_max_exp)), beta1=float(rng.choice([0.0, 0.5, 0.9, 0.95, 0.999])),
                  beta2=float(rng.choice([0.0, 0.5, 0.95, 0.999, 0.99999])),
                  eps=float(rng.choice([0.0, 1e-12, 1e-8, 1e-6, 1e-3, 1.0])),
                  weight_decay=float(rng.choice([0.0, 0.01, 0.1, 1.0, 10.0])))
        if hp["eps"] == 0.0:
            spec.zero_grad_frac = 0.0        # whole tensors of 0/0 are nobody's parity case (single elements stay)
    else:
        hp = dict(lr=float(10.0 ** rng.uniform(-6, lr_max_exp)), beta1=float(rng.choice([0.0, 0.5, 0.9, 0.95])),
                  beta2=float(rng.choice([0.5, 0.95, 0.999, 0.9999])), eps=float(rng.choice([1e-8, 1e-6, 1e-10])),
                  weight_decay=float(rng.choice([0.0, 0.01, 0.1])))
    steps = int(rng.integers(1, 5))
    chunks = None
    if rng.uniform() < 0.3 and nt >= 4:          # the list updated in two to four calls under one norm
        cuts = sorted(set(int(c) for c in rng.integers(1, nt, size=int(rng.integers(1, 4)))))
        bounds = [0] + cuts + [nt]
        chunks = [list(range(a, b)) for a, b in zip(bounds[:-1], bounds[1:])]
    return spec, block, hp, steps, chunks


@pytest.mark.parametrize("first", [0, 25, 50, 75])
def test_random_configurations(first):
    for case in range(first, first + 25):
        spec, block, hp, steps, chunks = make_case(case)
        run_free(spec, block, steps, hp_kw=hp, chunks=chunks, resync=True)


@pytest.mark.parametrize("case", [2449, 2567])
def test_parameter_cancelling_against_its_update(case):
    # bf16 parameters, found by a longer run of the generator above: an element whose decayed parameter and
    # update cancel to a few thousandths of either. Without the kernel's cancellation guard the approximate
    # update's error (1e-7 of the update) is 2 to 3 bf16 ulps of that tiny result.
    spec, block, hp, steps, chunks = make_case(case, bf16_params=True)
    run_free(spec, block, steps, hp_kw=hp, chunks=chunks, resync=True)


def test_bf16_parameters_at_large_learning_rates():
    # learning rates up to 0.3: update and parameter are of one size, so they cancel often; every launch stays on
    # the approximate path with its guard (there is no switch to the exact path by step size)
    for case in range(20000, 20040):
        spec, block, hp, steps, chunks = make_case(case, bf16_params=True, lr_max_exp=-0.5)
        run_free(spec, block, steps, hp_kw=hp, chunks=chunks, resync=True)


def test_fp32_parameters_at_large_learning_rates():
    # updates of the parameters' own size: the two cancel often. The approximate update stays within 1e-5 of
    # max(|p'|, |update|) there (its error is 6.6e-7 of the update); measured against |p'| alone, 6 % of
    # these cases show 1.1e-5 to 3.4e-5 on an element that cancelled, as any arithmetic would
    for case in range(32361, 32480, 3):
        spec, block, hp, steps, chunks = make_case(case, bf16_params=False, lr_max_exp=-0.5)
        run_free(spec, block, steps, hp_kw=hp, chunks=chunks, resync=True)


def test_extreme_hyper_parameters_and_gradient_scales():
    # gradient scales from 1e-12 to 1e4, eps from 0 to 1, weight decay up to 10, beta2 = 0: overflow to Inf and
    # 0/0 do occur, and must occur on both sides alike (the comparison requires equal NaN-ness and equal infinities)
    for case in range(40000, 40060):
        spec, block, hp, steps, chunks = make_case(case, extreme=True)
        run_free(spec, block, steps, hp_kw=hp, chunks=chunks, resync=True)
