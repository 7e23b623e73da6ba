"""GPU-vs-oracle parity of the CUDA path, through the C ABI (ctypes binding), on seeded inputs.

Small configurations are compared element by element on every step, free-running (both sides start
from the same initial state and never re-synchronise). See tests/test_gpu_full_size.py for the
full-size configurations, compared on sampled blocks."""
import math

import numpy as np
import pytest
import torch

import oracle as O
import paper_2608_11919_b200 as L
from paper_2608_11919_b200 import workloads as W
from parity_util import (NORM_RTOL, Stats, adopt_gpu_params, compare, host_np, oracle_sqnorm_of_buffers, oracle_step, oracle_tensors,
                         parallel_oracle_step, refresh_grads)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def to_bf16_params(spec):
    spec.param_dtype = torch.bfloat16
    return spec


def run_free(spec, block, steps, hp_kw=None, chunks=None, check_every_step=True, resync=False):
    """GPU and oracle run `steps` steps independently from the same start; returns per-step stats.
    resync: after every comparison the oracle takes over the GPU's parameters, so that each step is
    compared from identical inputs (the state is compared for identity anyway)."""
    torch.cuda.set_device(0)
    buf = W.Buffers(spec, block, DEV, guard_bytes=256)
    W.fill_params(buf)
    tl = L.TensorList.from_buffers(buf)
    hp = L.HParams(max_norm=spec.max_norm, **(hp_kw or {}))
    chunk_lists = None
    if chunks:
        chunk_lists = [L.TensorList.from_buffers(buf, c) for c in chunks]
    opt = L.Hybrid8Optimizer(tl, block, hp, chunk_lists)
    opt.init_state()
    W.fill_grads(buf, 1)
    ots, slices = oracle_tensors(buf)
    # S0 parity: the kernel's initial state equals the oracle's
    init = [O.OracleTensor(t.param.copy(), t.grad.copy(), block, fp32_state=t.fp32_state) for t in ots]
    O.state_init(init, block)
    for a, b in zip(ots, init):
        for k in ("m_code", "v_code", "m_absmax", "v_absmax"):
            assert np.array_equal(getattr(a, k), getattr(b, k)), k
    ohp = O.HParams(lr=hp.lr, beta1=hp.beta1, beta2=hp.beta2, eps=hp.eps, weight_decay=hp.weight_decay,
                    max_norm=hp.max_norm)
    out = []
    for k in range(1, steps + 1):
        if k > 1:
            W.fill_grads(buf, k)
            refresh_grads(ots, buf, slices)
        opt.step()
        torch.cuda.synchronize()
        S_gpu = float(opt.sqnorm.item())
        S = O.sqnorm(ots)
        assert abs(S_gpu - S) <= NORM_RTOL * S, (k, S_gpu, S)
        ohp.step = k
        assert parallel_oracle_step(ots, block, ohp, S) == 0
        assert int(opt.status.item()) == 0
        buf.check_guards()                       # nothing was written past the end of any flat buffer
        if check_every_step or k == steps:
            st = compare(buf, ots, slices)
            st.norm_rel = abs(S_gpu - S) / S if S else 0.0
            st.check()
            out.append(st)
        if resync:
            adopt_gpu_params(ots, buf, slices)
    return out


@pytest.mark.parametrize("block", [2048, 4096])
@pytest.mark.parametrize("param_dtype", [torch.float32, torch.bfloat16])
def test_tiny_three_steps(block, param_dtype):
    spec = W.tiny_spec()
    spec.param_dtype = param_dtype
    stats = run_free(spec, block, 3)
    # the clip fires on every step of this configuration (||g|| ~ 2 > max_norm); heavily on step 2
    assert stats[-1].n == 2 * spec.numel


def test_forty_free_running_steps_do_not_drift():
    # both sides run 40 steps without ever re-synchronising; the state stays bit-identical and the
    # parameters do not walk away (a parameter update with a different rounding sequence than the
    # definition's passes the per-step tolerance but drifts linearly: 6e-8 per step was measured)
    for pd in (torch.float32, torch.bfloat16):
        spec = W.tiny_spec()
        spec.param_dtype = pd
        spec.step_scale = {2: 1e3, 7: 1e-2, 13: 50.0}
        stats = run_free(spec, 2048, 40, check_every_step=False)
        assert stats[-1].code_mismatch == 0 and stats[-1].scale_max_rel == 0.0
        assert stats[-1].param_max_rel <= 1e-6 and stats[-1].param_max_ulp <= 1, stats[-1]   # the one-FMA form: 2.7e-6


def test_tiny_unclipped_variant():
    spec = W.tiny_spec()
    spec.max_norm = 10.0
    spec.step_scale = {}
    run_free(spec, 2048, 3)


def test_tiny_clipping_disabled_null_norm():
    torch.cuda.set_device(0)
    spec = W.tiny_spec()
    buf = W.Buffers(spec, 2048, DEV)
    W.fill_params(buf); W.fill_grads(buf, 1)
    tl = L.TensorList.from_buffers(buf)
    L.lt_hybrid8_state_init(tl, 2048)
    ots, slices = oracle_tensors(buf)
    hp = L.HParams(max_norm=0.0)
    L.lt_hybrid8_step(tl, 2048, hp, None, None)
    torch.cuda.synchronize()
    oracle_step(ots, 2048, O.HParams(max_norm=0.0), 1.0)
    compare(buf, ots, slices).check()


@pytest.mark.parametrize("block", [2048, 4096])
def test_ragged_small_ten_steps(block):
    spec = W.ragged_spec(n_tensors=1000, max_numel=1 << 16, seed=1)
    stats = run_free(spec, block, 10)
    assert stats[-1].code_max_dist <= 1


def test_ragged_small_bf16_params_other_blocks():
    for block in (256, 1024, 8192, 16384):
        spec = to_bf16_params(W.ragged_spec(n_tensors=120, max_numel=1 << 16, seed=5))
        run_free(spec, block, 2)
    spec = W.ragged_spec(n_tensors=60, max_numel=1 << 15, seed=6)
    run_free(spec, 512, 2)


def test_every_small_size_and_alignment():
    # numel 1 .. a little over two blocks, packed back to back so that every base alignment occurs
    block = 256
    sizes = list(range(1, 2 * block + 4)) + [3 * block - 1, 3 * block, 3 * block + 1, 4 * block + 3]
    spec = W.ragged_spec(n_tensors=len(sizes), seed=9)
    spec.sizes = sizes
    for pd in (torch.float32, torch.bfloat16):
        spec.param_dtype = pd
        run_free(spec, block, 2)


def test_bf16_parameters_at_every_multiple_of_four_offset():
    # tensor sizes that are multiples of 4 but not of 8 or 16: packed back to back, the bases run through
    # every 4-element offset, so full blocks meet the 8-element vector path (16-byte aligned arrays), the
    # 4-element one (8-byte aligned) and, with the single odd size, the shifted one
    for block in (2048, 4096, 8192):
        sizes = [2 * block + 4, block + 12, 3 * block + 8, block + 4, 2 * block + 16, block + 20, 2 * block + 1,
                 block + 28, 2 * block + 4, block]
        spec = to_bf16_params(W.ragged_spec(n_tensors=len(sizes), seed=31))
        spec.sizes = sizes
        run_free(spec, block, 3)


def test_fp32_gradients():
    spec = W.ragged_spec(n_tensors=50, max_numel=1 << 15, seed=11)
    spec.grad_dtype = torch.float32
    run_free(spec, 2048, 2)


def test_norm_parity_and_reproducibility():
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=1000, max_numel=1 << 18, seed=3)
    buf = W.Buffers(spec, 2048, DEV)
    W.fill_grads(buf, 1)
    tl = L.TensorList.from_buffers(buf)
    ws = torch.empty(L.lt_workspace_bytes(), dtype=torch.uint8, device=DEV)
    S = oracle_sqnorm_of_buffers(buf)
    vals = []
    for _ in range(3):
        acc = torch.zeros(1, dtype=torch.float64, device=DEV)
        L.lt_grad_sqnorm_multi(tl, acc, ws)
        vals.append(float(acc.item()))
    assert abs(vals[0] - S) <= 1e-9 * S, (vals, S)       # far inside the 1e-5 tolerance
    assert vals[0] == vals[1] == vals[2]                # bit-reproducible
    # accumulates: chunked calls into one scalar, and a non-zero start value
    acc = torch.full((1,), 5.0, dtype=torch.float64, device=DEV)
    for a in range(0, tl.n, 300):
        L.lt_grad_sqnorm_multi(tl.slice(a, a + 300), acc, ws)
    assert abs(float(acc.item()) - 5.0 - S) <= 1e-9 * S
    # all-ones gradient: ||g||^2 = N exactly
    buf.grad.fill_(1.0)
    acc.zero_()
    L.lt_grad_sqnorm_multi(tl, acc, ws)
    assert float(acc.item()) == float(spec.numel)


def test_chunk_invariance_bit_identical():
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=200, max_numel=1 << 16, seed=4)
    bufs = []
    for chunked in (False, True):
        buf = W.Buffers(spec, 2048, DEV)
        W.fill_params(buf); W.fill_grads(buf, 1)
        tl = L.TensorList.from_buffers(buf)
        chunks = [tl.slice(a, a + 37) for a in range(0, tl.n, 37)] if chunked else None
        opt = L.Hybrid8Optimizer(tl, 2048, L.HParams(max_norm=0.5), chunks)
        opt.init_state()
        for k in (1, 2):
            W.fill_grads(buf, k)
            opt.step()
        torch.cuda.synchronize()
        bufs.append(buf)
    for key in ("param", "m_code", "v_code", "m_absmax", "v_absmax"):
        a, b = getattr(bufs[0], key), getattr(bufs[1], key)
        if key == "param":
            a, b = a.view(torch.int32), b.view(torch.int32)
        assert torch.equal(a, b), key


@pytest.mark.parametrize("bad", [float("nan"), float("inf"), float("-inf")])
def test_nonfinite_gradient_skips_step(bad):
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=40, max_numel=1 << 15, seed=8)
    buf = W.Buffers(spec, 2048, DEV)
    W.fill_params(buf); W.fill_grads(buf, 1)
    tl = L.TensorList.from_buffers(buf)
    opt = L.Hybrid8Optimizer(tl, 2048, L.HParams(max_norm=0.5))
    opt.init_state()
    opt.step()                                  # one good step so the state is not trivial
    torch.cuda.synchronize()
    assert int(opt.status.item()) == 0
    W.fill_grads(buf, 2)
    buf.view("grad", 17)[3] = bad               # injected from the host side of the API
    before = {k: getattr(buf, k).clone() for k in ("param", "m_code", "v_code", "m_absmax", "v_absmax")}
    opt.step()
    torch.cuda.synchronize()
    assert int(opt.status.item()) & 1
    assert not math.isfinite(float(opt.sqnorm.item()))
    for k, v in before.items():
        a, b = getattr(buf, k), v
        if a.dtype == torch.float32:
            a, b = a.view(torch.int32), b.view(torch.int32)
        assert torch.equal(a, b), k
    # the next finite step runs again
    opt.status.zero_()
    W.fill_grads(buf, 3)
    opt.step()
    torch.cuda.synchronize()
    assert int(opt.status.item()) == 0
    assert not torch.equal(buf.param, before["param"])


@pytest.mark.parametrize("graphed", [False, True])
def test_a_skipped_step_does_not_count_towards_the_bias_corrections(graphed):
    """Steps 1, 2(non-finite: skipped), 3 must leave exactly what steps 1, 2 of a run without the bad step leave:
    the step count that forms lr / (1 - beta1^t) and 1 / sqrt(1 - beta2^t) does not advance on a skipped step
    (device-side in the graphed driver; settle_skipped_step() in the eager one)."""
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=30, max_numel=1 << 14, seed=12)
    cls = L.GraphedHybrid8Optimizer if graphed else L.Hybrid8Optimizer
    bufs = []
    for with_bad_step in (False, True):
        buf = W.Buffers(spec, 2048, DEV)
        W.fill_params(buf)
        opt = cls(L.TensorList.from_buffers(buf), 2048, L.HParams(max_norm=0.5, lr=1e-3))
        opt.init_state()
        W.fill_grads(buf, 1)
        opt.step()
        if with_bad_step:
            W.fill_grads(buf, 7)
            buf.view("grad", 5)[0] = float("nan")
            opt.step()
            torch.cuda.synchronize()
            assert int(opt.status.item()) & 1
            if graphed:
                assert int(opt.state.cpu()[0]) == 1 and int(opt.skip_count.item()) == 1
                opt.status.zero_()
            else:
                assert opt.settle_skipped_step() and opt.t == 1 and not opt.settle_skipped_step()
        W.fill_grads(buf, 2)
        opt.step()
        torch.cuda.synchronize()
        assert int(opt.status.item()) == 0
        bufs.append(buf)
    for key in ("param", "m_code", "v_code", "m_absmax", "v_absmax"):
        a, b = getattr(bufs[0], key), getattr(bufs[1], key)
        if a.dtype == torch.float32:
            a, b = a.view(torch.int32), b.view(torch.int32)
        assert torch.equal(a, b), key


def test_byte_zero_state_equals_value_zero_state():
    torch.cuda.set_device(0)
    spec = W.tiny_spec()
    res = []
    for byte_zero in (False, True):
        buf = W.Buffers(spec, 2048, DEV)
        W.fill_params(buf); W.fill_grads(buf, 1)
        tl = L.TensorList.from_buffers(buf)
        opt = L.Hybrid8Optimizer(tl, 2048, L.HParams())
        opt.init_state()
        if byte_zero:
            buf.m_code.zero_()
        opt.step()
        torch.cuda.synchronize()
        res.append(buf)
    for key in ("m_code", "v_code", "m_absmax", "v_absmax", "param"):
        assert torch.equal(getattr(res[0], key), getattr(res[1], key)), key


def test_two_host_threads_on_two_streams():
    # two optimizers with their own buffers, scratch and streams, driven from two host threads at once
    # (ctypes drops the GIL inside the library): each must end exactly where it ends when run alone
    import threading
    torch.cuda.set_device(0)
    specs = [W.ragged_spec(n_tensors=200, max_numel=1 << 16, seed=51),
             to_bf16_params(W.ragged_spec(n_tensors=150, max_numel=1 << 16, seed=52))]

    def run(spec, block, stream, out, barrier=None):
        torch.cuda.set_device(0)
        with torch.cuda.stream(stream):
            buf = W.Buffers(spec, block, DEV)
            W.fill_params(buf)
            opt = L.Hybrid8Optimizer(L.TensorList.from_buffers(buf), block, L.HParams(max_norm=0.5))
            opt.init_state()
            if barrier is not None:
                barrier.wait()
            for k in range(1, 9):
                W.fill_grads(buf, k)
                opt.step()
            stream.synchronize()
            out.append({k: getattr(buf, k).clone() for k in ("param", "m_code", "v_code", "m_absmax", "v_absmax")})

    alone = []
    for spec, block in zip(specs, (2048, 4096)):
        res = []
        run(spec, block, torch.cuda.Stream(), res)
        alone.append(res[0])
    together = [[], []]
    barrier = threading.Barrier(2)
    threads = [threading.Thread(target=run, args=(spec, block, torch.cuda.Stream(), together[i], barrier))
               for i, (spec, block) in enumerate(zip(specs, (2048, 4096)))]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
        assert not t.is_alive()
    for a, b in zip(alone, together):
        assert len(b) == 1
        for k, v in a.items():
            assert torch.equal(v, b[0][k]), k


def test_resume_from_saved_state_is_bit_identical():
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=64, max_numel=1 << 15, seed=12)

    def fresh():
        buf = W.Buffers(spec, 2048, DEV)
        W.fill_params(buf)
        tl = L.TensorList.from_buffers(buf)
        opt = L.Hybrid8Optimizer(tl, 2048, L.HParams(max_norm=0.5))
        opt.init_state()
        return buf, opt

    a, oa = fresh()
    for k in (1, 2):
        W.fill_grads(a, k); oa.step()
    saved = {k: getattr(a, k).cpu() for k in ("param", "m_code", "v_code", "m_absmax", "v_absmax")}
    W.fill_grads(a, 3); oa.step()
    b, ob = fresh()
    for k, v in saved.items():
        getattr(b, k).copy_(v)
    ob.t = 2
    W.fill_grads(b, 3); ob.step()
    torch.cuda.synchronize()
    for key in ("m_code", "v_code", "m_absmax", "v_absmax", "param"):
        assert torch.equal(getattr(a, key), getattr(b, key)), key


def test_hybrid_fp32_and_8bit_state_in_one_list():
    # the paper's hybrid split: most tensors keep plain fp32 moments, a slice is 8-bit; one call updates both
    for pd in (torch.float32, torch.bfloat16):
        spec = W.ragged_spec(n_tensors=120, max_numel=1 << 16, seed=13)
        spec.param_dtype = pd
        spec.state_f32 = [i % 3 != 0 for i in range(len(spec.sizes))]
        stats = run_free(spec, 4096, 4)
        assert stats[-1].state32_max_rel == 0.0          # fp32 moments are bit-identical


def test_hybrid_decoder_split_matches_target_fraction():
    spec = W.hybrid_split(W.small_spec())
    n8 = sum(s for s, f in zip(spec.sizes, spec.state_f32) if not f)
    assert 0.015 <= n8 / spec.numel <= 0.03
    run_free(spec, 4096, 2, check_every_step=False)


def test_per_tensor_norms_and_skip_counter():
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=700, max_numel=1 << 17, seed=19)      # more tensors than one launch holds
    buf = W.Buffers(spec, 2048, DEV)
    W.fill_params(buf); W.fill_grads(buf, 1)
    tl = L.TensorList.from_buffers(buf)
    out = torch.zeros(tl.n, dtype=torch.float64, device=DEV)
    L.lt_grad_sqnorm_per_tensor(tl, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    ots, _ = oracle_tensors(buf)
    ref = np.array([O.sqnorm([t]) for t in ots])
    assert np.all(np.abs(got - ref) <= 1e-12 * np.maximum(ref, 1e-300))
    assert np.all(got[ref == 0] == 0)                                      # the all-zero-gradient tensors
    assert abs(got.sum() - O.sqnorm(ots)) <= 1e-11 * ref.sum()
    # consecutive non-finite steps are counted on the device and reset by a finite one
    opt = L.Hybrid8Optimizer(tl, 2048, L.HParams(max_norm=0.5))
    opt.init_state()
    seen = []
    for k, bad in enumerate([False, True, True, False, True, True, True], start=1):
        W.fill_grads(buf, k)
        if bad:
            buf.view("grad", 5)[0] = float("inf")
        opt.step()
        seen.append(int(opt.skip_count.item()))
    assert seen == [0, 1, 2, 0, 1, 2, 3]
    assert int(opt.status.item()) & 1


@pytest.mark.parametrize("hp_kw", [
    dict(eps=0.0),                                   # tiny eps: the kernel takes IEEE sqrt and divide for the parameter
    dict(eps=1e-20, lr=1e-3),
    dict(beta1=0.0, beta2=0.5, weight_decay=0.0, lr=1e-2),
    dict(beta1=0.99, beta2=0.9999, eps=1e-6, lr=3e-4, weight_decay=0.1),
    dict(lr=0.0),                                    # zero step size: only the decay factor (1) touches the parameter
    dict(lr=1e-37, weight_decay=0.0),                # eps / step_size leaves the fp32 range
    dict(lr=1e-6, eps=1e3),                          # the denominator is all eps
])
def test_other_hyper_parameters(hp_kw):
    for pd in (torch.float32, torch.bfloat16):
        spec = W.ragged_spec(n_tensors=80, max_numel=1 << 15, seed=23)
        spec.param_dtype = pd
        spec.zero_grad_frac = 0.0 if hp_kw.get("eps", 1.0) == 0.0 else spec.zero_grad_frac   # 0/0 is nobody's parity case
        run_free(spec, 2048, 3, hp_kw=hp_kw)


def test_late_step_count_and_infinite_max_norm():
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=60, max_numel=1 << 15, seed=24)
    buf = W.Buffers(spec, 4096, DEV)
    W.fill_params(buf); W.fill_grads(buf, 1)
    tl = L.TensorList.from_buffers(buf)
    L.lt_hybrid8_state_init(tl, 4096)
    ots, slices = oracle_tensors(buf)
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    ws = torch.empty(L.lt_workspace_bytes(), dtype=torch.uint8, device=DEV)
    for t in (1000, 100000):                         # bias corrections ~1
        W.fill_grads(buf, t)
        refresh_grads(ots, buf, slices)
        sq.zero_()
        L.lt_grad_sqnorm_multi(tl, sq, ws)
        L.lt_hybrid8_step(tl, 4096, L.HParams(max_norm=float("inf"), step=t), sq, None)
        torch.cuda.synchronize()
        oracle_step(ots, 4096, O.HParams(max_norm=float("inf"), step=t), O.sqnorm(ots))
        compare(buf, ots, slices).check()


def test_empty_lists_and_empty_tensors():
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=12, max_numel=1 << 13, seed=25)
    buf = W.Buffers(spec, 2048, DEV)
    W.fill_params(buf); W.fill_grads(buf, 1)
    views = {k: [buf.view(k, t) for t in range(12)] for k in ("param", "grad", "m_code", "v_code", "m_absmax", "v_absmax")}
    for k in views:                                   # tensors 2 and 7 become empty
        for t in (2, 7):
            views[k][t] = views[k][t][:0]
    tl = L.TensorList(*[views[k] for k in ("param", "grad", "m_code", "v_code", "m_absmax", "v_absmax")])
    full = L.TensorList.from_buffers(buf, [t for t in range(12) if t not in (2, 7)])
    ws = torch.empty(L.lt_workspace_bytes(), dtype=torch.uint8, device=DEV)
    a = torch.zeros(1, dtype=torch.float64, device=DEV); b = torch.zeros(1, dtype=torch.float64, device=DEV)
    L.lt_hybrid8_state_init(tl, 2048)
    L.lt_grad_sqnorm_multi(tl, a, ws); L.lt_grad_sqnorm_multi(full, b, ws)
    L.lt_grad_sqnorm_multi(tl.slice(0, 0), a, ws)     # an empty list is a no-op
    L.lt_hybrid8_step(tl.slice(0, 0), 2048, L.HParams(), a, None)
    before = buf.param.clone()
    L.lt_hybrid8_step(tl, 2048, L.HParams(), a, None)
    torch.cuda.synchronize()
    assert float(a.item()) == float(b.item()) > 0
    for t in range(12):
        changed = not torch.equal(buf.view("param", t), before[buf.off[t]: buf.off[t] + spec.sizes[t]])
        assert changed == (t not in (2, 7)), t         # the emptied tensors' storage was not touched


def test_overflowing_moments_do_not_fault():
    # clipping disabled and absurd gradients: v' overflows to +inf, the block maximum is inf, the normalised
    # values are NaN. Nothing sensible can come out, but every table index stays in range, nothing faults,
    # and the next ordinary step runs.
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=20, max_numel=1 << 14, seed=26)
    for pd in (torch.float32, torch.bfloat16):
        spec.param_dtype = pd
        buf = W.Buffers(spec, 2048, DEV)
        W.fill_params(buf)
        tl = L.TensorList.from_buffers(buf)
        opt = L.Hybrid8Optimizer(tl, 2048, L.HParams(max_norm=0.0))
        opt.init_state()
        buf.grad.fill_(1e30)
        opt.step()
        torch.cuda.synchronize()
        assert int(opt.status.item()) == 0
        opt.init_state()
        W.fill_grads(buf, 1)
        opt.step()
        torch.cuda.synchronize()
        assert bool(torch.isfinite(buf.m_absmax).all()) and bool(torch.isfinite(buf.param.float()).all())


def test_gpu_norm_against_exact_sum():
    # the kernel adds exact fp64 squares; against the exactly rounded sum (math.fsum) it is far more accurate
    # than the 1e-5 tolerance asks for, and more accurate than one long sequential fp64 sum
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=300, max_numel=1 << 16, seed=27)
    buf = W.Buffers(spec, 2048, DEV)
    W.fill_grads(buf, 1)
    tl = L.TensorList.from_buffers(buf)
    acc = torch.zeros(1, dtype=torch.float64, device=DEV)
    ws = torch.empty(L.lt_workspace_bytes(), dtype=torch.uint8, device=DEV)
    L.lt_grad_sqnorm_multi(tl, acc, ws)
    g = buf.grad[:buf.total].float().double().cpu().numpy()
    exact = math.fsum((g * g).tolist())
    assert abs(float(acc.item()) - exact) <= 1e-13 * exact


@pytest.mark.parametrize("block", [256, 512, 1024, 8192, 16384])
def test_aligned_tensors_at_every_other_block_size(block):
    # 16-byte aligned tensors take the vector path with bulk L2 prefetch at every supported block size
    for pd in (torch.float32, torch.bfloat16):
        spec = W.tiny_spec()
        spec.param_dtype = pd
        run_free(spec, block, 2)
