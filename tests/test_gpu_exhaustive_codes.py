"""Every fp32 value a normalised first moment can take between 2^-33 and 1, of either sign, goes through
the real step kernel and must get the oracle's code.

With beta1 = beta2 = 0, clipping disabled and fp32 gradients, the new moments are m' = g and
v' = fl(g * g) exactly on both sides. Each quantization block starts with g = peak, so the block maxima are
peak and fl(peak^2). With peak = 1 the normalised values handed to the quantizer are g itself (signed map) and
fl(g * g) (unsigned map, which this way also sees values down to 2^-66, far below its smallest threshold);
with a peak that is no power of two they are the quotients, which puts the kernel's division (reciprocal,
exact remainder, one correction) against the oracle's IEEE division on every input. The remaining 2047
elements of every block enumerate consecutive bit patterns from 2^-33 up to the peak. Run with fp32 and with
bf16 parameters, because the kernel stages differently laid out lookup tables for the two.

Below 2^-33 (where every code is the zero code, but the full-range tables are still indexed by every
exponent field and the signed lookup takes the integer absolute value of the raw bits) a second test plants
+0 and -0, the values around every exponent boundary down to the smallest subnormal, and a strided sweep of
[2^-149, 2^-33) of both signs; their squares put [0, 2^-66) through the unsigned table.
"""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2608_11919_b200 as L
from paper_2608_11919_b200 import workloads as W
from parity_util import compare, oracle_tensors, parallel_oracle_step

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
BLOCK = 2048
LO_BITS = 0x2F000000                            # 2^-33
N_TENSORS_PER_SIGN = 16


def _build(param_dtype, peak, bits=None):
    """bits: magnitudes to plant (int64 tensor of fp32 bit patterns); default: every pattern of [2^-33, peak)."""
    HI_BITS = int(np.float32(peak).view(np.uint32))   # enumerate [2^-33, peak)
    count = HI_BITS - LO_BITS if bits is None else int(bits.numel())
    per_block = BLOCK - 1
    n_blocks = (count + per_block - 1) // per_block
    blocks_per_tensor = (n_blocks + N_TENSORS_PER_SIGN - 1) // N_TENSORS_PER_SIGN
    sizes, b = [], 0
    while b < n_blocks:
        nb = min(blocks_per_tensor, n_blocks - b)
        sizes.append(nb * BLOCK)
        b += nb
    n_half = len(sizes)
    spec = W.Spec("exhaustive", [f"x{i}" for i in range(2 * n_half)], sizes + sizes, [-1] * (2 * n_half),
                  param_dtype, grad_dtype=torch.float32, seed=41, align_elems=16)
    buf = W.Buffers(spec, BLOCK, DEV)
    W.fill_params(buf)
    if bits is None:
        bits = torch.arange(LO_BITS, LO_BITS + n_blocks * per_block, dtype=torch.int64, device=DEV)
        bits = torch.where(bits < HI_BITS, bits, torch.zeros_like(bits)).to(torch.int32)  # tail of the last block: zeros
    else:
        pad = torch.zeros(n_blocks * per_block - count, dtype=torch.int64, device=DEV)
        bits = torch.cat([bits.to(DEV), pad]).to(torch.int32)
    mag = bits.view(torch.float32).view(n_blocks, per_block)
    ones = torch.full((n_blocks, 1), float(np.float32(peak)), dtype=torch.float32, device=DEV)
    pos = torch.cat([ones, mag], dim=1).reshape(-1)
    neg = torch.cat([ones, -mag], dim=1).reshape(-1)
    assert buf.total == 2 * pos.numel()                 # sizes are multiples of 16: no padding between tensors
    buf.grad[:pos.numel()].copy_(pos)
    buf.grad[pos.numel():].copy_(neg)
    return spec, buf


@pytest.mark.parametrize("peak", [1.0, 1.7182817])
@pytest.mark.parametrize("param_dtype", [torch.float32, torch.bfloat16])
def test_every_normalised_value_gets_the_oracle_code(param_dtype, peak):
    torch.cuda.set_device(0)
    spec, buf = _build(param_dtype, peak)
    tl = L.TensorList.from_buffers(buf)
    L.lt_hybrid8_state_init(tl, BLOCK)
    ots, slices = oracle_tensors(buf)
    kw = dict(beta1=0.0, beta2=0.0, max_norm=float("inf"), step=1)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    L.lt_hybrid8_step(tl, BLOCK, L.HParams(**kw), None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert parallel_oracle_step(ots, BLOCK, O.HParams(**kw), 0.0) == 0
    st = compare(buf, ots, slices)
    assert st.code_mismatch == 0 and st.scale_max_rel == 0.0, st
    st.check()
    # the inputs did reach every code of both maps, and every block maximum is the planted peak
    m_seen = np.zeros(256, bool)
    v_seen = np.zeros(256, bool)
    for ot in ots:
        m_seen[np.unique(ot.m_code)] = True
        v_seen[np.unique(ot.v_code)] = True
        assert np.all(ot.m_absmax == np.float32(peak)) and np.all(ot.v_absmax == np.float32(peak) * np.float32(peak))
    assert m_seen.all() and v_seen.all()


def _tiny_bits():
    edges = []
    for e in range(0, 0x2F0 // 8 + 1):                  # exponent fields 0 .. 94: [2^-149 .. 2^-33)
        b = e << 23
        edges += [b - 1, b, b + 1, b + 0x400000, b + 0x7FFFFF]
    edges = [x for x in edges if 0 <= x < LO_BITS]
    edges += [0, 1, 2, 3, 0x007FFFFF, 0x00800000, LO_BITS - 1]       # zero, smallest / largest subnormal, smallest normal
    sweep = torch.arange(1, LO_BITS, 197, dtype=torch.int64)          # 4.0e6 values, every exponent field many times
    return torch.cat([torch.tensor(edges, dtype=torch.int64), sweep])


@pytest.mark.parametrize("peak", [1.0, 1.7182817])
@pytest.mark.parametrize("param_dtype", [torch.float32, torch.bfloat16])
def test_zero_subnormal_and_tiny_values_get_the_oracle_code(param_dtype, peak):
    torch.cuda.set_device(0)
    spec, buf = _build(param_dtype, peak, _tiny_bits())
    tl = L.TensorList.from_buffers(buf)
    L.lt_hybrid8_state_init(tl, BLOCK)
    ots, slices = oracle_tensors(buf)
    # the planted values are what the test says: -0.0 is among the negated half, subnormals survive the copy
    g = buf.grad.view(torch.int32)
    assert int((g == -0x80000000).sum()) > 0 and int(((g & 0x7F800000) == 0).sum()) > 8000
    kw = dict(beta1=0.0, beta2=0.0, max_norm=float("inf"), step=1)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    L.lt_hybrid8_step(tl, BLOCK, L.HParams(**kw), None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert parallel_oracle_step(ots, BLOCK, O.HParams(**kw), 0.0) == 0
    st = compare(buf, ots, slices)
    assert st.code_mismatch == 0 and st.scale_max_rel == 0.0, st
    st.check()
    for ot in ots:                                       # below the smallest threshold everything is the zero code
        m = ot.m_code.reshape(-1, BLOCK)[:, 1:]
        v = ot.v_code.reshape(-1, BLOCK)[:, 1:]
        assert np.all(m == 127) and np.all(v == 0)
