"""Helpers of the parity tests: move device state to the CPU oracle and compare element by element.

Tolerances (the ones the task fixes): squared-norm relative error <= 1e-5; fp32 parameters relative
error <= 1e-5; bf16 parameters <= 1 ulp; block scales relative error <= 1e-6; codes identical on
>= 99.99 % of elements and never more than one index apart.

fp32 parameters: the error is taken relative to max(|p_new|, U), U = the sum of |p_new - p_old| over the
oracle's steps since both sides last held identical parameters: the larger of the result and of the updates
that formed it (where a parameter and its update cancel, no arithmetic, the oracle's included, can hold
the difference to 1e-5 of the small result; in a free run the allowances of the steps add up), with an
absolute floor of 1e-12. The error relative to |p_new| alone is recorded beside it (param_max_rel_raw) and
not asserted.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle as O
from paper_2608_11919_b200 import workloads as W

NORM_RTOL = 1e-5
PARAM_RTOL = 1e-5
PARAM_FLOOR = 1e-12
SCALE_RTOL = 1e-6
CODE_MATCH_MIN = 0.9999


def host_np(t: torch.Tensor) -> np.ndarray:
    """Device (or host) tensor -> fresh host numpy array; bf16 as uint16 bits."""
    t = t.detach().to("cpu").contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


def oracle_tensors(buf: W.Buffers, indices=None, slices=None):
    """OracleTensors holding copies of the device state of tensors `indices` (or of the
    block-aligned element ranges `slices` = [(tensor, first_block, n_blocks), ...])."""
    out = []
    if slices is None:
        idx = range(len(buf.spec.sizes)) if indices is None else indices
        slices = [(t, 0, None) for t in idx]
    for t, b0, nb in slices:
        size = buf.spec.sizes[t]
        tb = (size + buf.block - 1) // buf.block
        b1 = tb if nb is None else min(tb, b0 + nb)
        e0, e1 = b0 * buf.block, min(size, b1 * buf.block)
        out.append(O.OracleTensor(
            host_np(buf.view("param", t)[e0:e1]), host_np(buf.view("grad", t)[e0:e1]), buf.block,
            host_np(buf.view("m_code", t)[e0:e1]), host_np(buf.view("v_code", t)[e0:e1]),
            None if buf.f32[t] else host_np(buf.view("m_absmax", t)[b0:b1]),
            None if buf.f32[t] else host_np(buf.view("v_absmax", t)[b0:b1])))
    return out, slices


def refresh_grads(ots, buf: W.Buffers, slices) -> None:
    for ot, (t, b0, nb) in zip(ots, slices):
        e0 = b0 * buf.block
        ot.set_grad(host_np(buf.view("grad", t)[e0:e0 + ot.numel]))


def oracle_sqnorm_of_buffers(buf: W.Buffers, chunk: int = 1 << 27) -> float:
    """fp64 sequential squared norm of ALL gradients of the workload, streamed through the host in
    tensor order (flat buffers keep tensors in list order; alignment padding is zero-filled)."""
    S = 0.0
    lib = O.lib()
    dt = O.BF16 if buf.spec.grad_dtype == torch.bfloat16 else O.F32
    for t in range(len(buf.spec.sizes)):
        v = buf.view("grad", t)
        for a in range(0, v.numel(), chunk):
            h = host_np(v[a:a + chunk])
            S = float(lib.lto_sqnorm_accumulate(h.ctypes.data, dt, h.size, S))
    return S


class Stats:
    def __init__(self):
        self.n = 0
        self.param_max_rel = 0.0
        self.param_max_rel_raw = 0.0    # relative to |p_new| alone, no floor (reported, not asserted)
        self.param_max_ulp = 0
        self.scale_max_rel = 0.0
        self.code_mismatch = 0
        self.code_max_dist = 0
        self.state32_max_rel = 0.0      # fp32 moments of tensors with plain fp32 state

    def __repr__(self):
        return (f"Stats(n={self.n}, param_max_rel={self.param_max_rel:.3g}, raw={self.param_max_rel_raw:.3g}, "
                f"param_max_ulp={self.param_max_ulp}, "
                f"scale_max_rel={self.scale_max_rel:.3g}, code_mismatch={self.code_mismatch}, "
                f"code_max_dist={self.code_max_dist})")

    def check(self):
        assert self.param_max_rel <= PARAM_RTOL, self
        assert self.param_max_ulp <= 1, self
        assert self.scale_max_rel <= SCALE_RTOL, self
        assert self.state32_max_rel <= SCALE_RTOL, self
        assert self.code_max_dist <= 1, self
        assert self.code_mismatch <= (1.0 - CODE_MATCH_MIN) * max(self.n, 1), self


def _bf16_ordinal(bits: np.ndarray) -> np.ndarray:
    b = bits.astype(np.int64)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def compare(buf: W.Buffers, ots, slices, stats: Stats | None = None) -> Stats:
    st = stats or Stats()
    for ot, (t, b0, nb) in zip(ots, slices):
        e0 = b0 * buf.block
        n = ot.numel
        nbk = ot.m_absmax.size
        gp = host_np(buf.view("param", t)[e0:e0 + n])
        # a NaN parameter (0/0 with eps = 0 on an element whose moments are zero) must be NaN on both sides;
        # its bit pattern is nobody's business
        if ot.param.dtype == np.float32:
            ref = ot.param.astype(np.float64)
            got = gp.astype(np.float64)
            same = (np.isnan(ref) & np.isnan(got)) | (got == ref)          # equal values include equal infinities
            upd = getattr(ot, "upd_accum", None)            # sum of |update| since the parameters were last identical
            with np.errstate(invalid="ignore", divide="ignore"):
                scale = np.maximum(np.abs(ref), PARAM_FLOOR / PARAM_RTOL)
                if upd is not None:
                    scale = np.maximum(scale, upd)
                err = np.abs(got - ref) / scale
                raw = np.abs(got - ref) / np.abs(ref)
            err = np.where(same, 0.0, np.where(np.isnan(err), np.inf, err))
            raw = np.where(same | ~np.isfinite(raw), 0.0, raw)
            if n:
                st.param_max_rel = max(st.param_max_rel, float(err.max()))
                st.param_max_rel_raw = max(st.param_max_rel_raw, float(raw.max()))
        else:
            if n:
                is_nan = lambda b: (b & 0x7FFF) > 0x7F80      # noqa: E731
                d = np.abs(_bf16_ordinal(gp) - _bf16_ordinal(ot.param))
                d = np.where(is_nan(gp) & is_nan(ot.param), 0, d)
                st.param_max_ulp = max(st.param_max_ulp, int(d.max()))
        if ot.fp32_state:                 # plain fp32 moments: compared as values
            for key in ("m_code", "v_code"):
                g = host_np(buf.view(key, t)[e0:e0 + n]).astype(np.float64)
                r = getattr(ot, key).astype(np.float64)
                if n:
                    rel = np.abs(g - r) / np.maximum(np.abs(r), 1e-30)
                    st.state32_max_rel = max(st.state32_max_rel, float(np.where(g == r, 0.0, rel).max()))
            st.n += 2 * n
            continue
        for key in ("m_absmax", "v_absmax"):
            g = host_np(buf.view(key, t)[b0:b0 + nbk]).astype(np.float64)
            r = getattr(ot, key).astype(np.float64)
            if nbk:
                rel = np.abs(g - r) / np.where(r != 0, np.abs(r), 1.0)
                st.scale_max_rel = max(st.scale_max_rel, float(rel.max()))
        for key in ("m_code", "v_code"):
            g = host_np(buf.view(key, t)[e0:e0 + n]).astype(np.int32)
            d = np.abs(g - getattr(ot, key).astype(np.int32))
            if n:
                st.code_mismatch += int(np.count_nonzero(d))
                st.code_max_dist = max(st.code_max_dist, int(d.max()))
        st.n += 2 * n
    return st


def _remember_params(ots) -> None:
    for t in ots:
        if t.param.dtype == np.float32:
            t.prev_param = t.param.copy()


def _accumulate_updates(ots) -> None:
    """After an oracle step: adds |p_new - p_old| to each fp32 tensor's running sum (see compare)."""
    for t in ots:
        if t.param.dtype == np.float32:
            with np.errstate(invalid="ignore", over="ignore"):
                d = np.nan_to_num(np.abs(t.param - t.prev_param), nan=0.0, posinf=0.0)
            t.upd_accum = d if getattr(t, "upd_accum", None) is None else t.upd_accum + d
            t.prev_param = None


def adopt_gpu_params(ots, buf: W.Buffers, slices) -> None:
    """Resynchronisation: the oracle takes over the GPU's parameters; the update sums start again."""
    for ot, (t, b0, nb) in zip(ots, slices):
        e0 = b0 * buf.block
        ot.param[:] = host_np(buf.view("param", t)[e0:e0 + ot.numel])
        ot.upd_accum = None


def oracle_step(ots, block, hp, S) -> int:
    _remember_params(ots)
    r = O.hybrid8_step(ots, block, hp, S)
    _accumulate_updates(ots)
    return r


def parallel_oracle_step(ots, block, hp, S) -> int:
    """Runs the (single-threaded) oracle step on several tensors at once from Python threads; each
    tensor is an independent oracle call, so results are those of the sequential loop."""
    from concurrent.futures import ThreadPoolExecutor
    import os
    if len(ots) <= 1:
        return oracle_step(ots, block, hp, S)
    _remember_params(ots)
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
        res = list(ex.map(lambda t: O.hybrid8_step([t], block, hp, S), ots))
    _accumulate_updates(ots)
    r = 0
    for x in res:
        r |= x
    return r
