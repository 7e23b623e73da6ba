"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared symbol,
reports sizes and tables, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle as O
import paper_2608_11919_b200 as L
from paper_2608_11919_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names += re.findall(r"\b(lt_[a-z0-9_]+)\s*\(", src)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    lib = C.CDLL(L.library_path())
    names = declared_functions()
    assert {"lt_hybrid8_state_init", "lt_grad_sqnorm_multi", "lt_hybrid8_step"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_tables_bit_equal_to_oracle():
    for signed in (True, False):
        assert np.array_equal(L.lt_hybrid8_code_table(signed).numpy().view(np.uint32),
                              O.code_table(signed).view(np.uint32))


def test_state_bytes_and_workspace():
    assert L.lt_hybrid8_state_bytes(0, 2048) == (0, 0)
    assert L.lt_hybrid8_state_bytes(2049, 2048) == (2049, 8)
    assert L.lt_hybrid8_state_bytes(1 << 30, 4096) == (1 << 30, 4 * (1 << 18))
    for n in (1, 5000, 123457):
        for b in (2048, 4096):
            assert L.lt_hybrid8_state_bytes(n, b) == O.state_bytes(n, b)
    with pytest.raises(L.LtError) as e:
        L.lt_hybrid8_state_bytes(10, 3000)
    assert e.value.code == -3
    assert 0 < L.lt_workspace_bytes() <= 1 << 20


def _tensor(**kw):
    d = dict(param=0x1000, grad=0x2000, m_code=0x3000, v_code=0x4000, m_absmax=0x5000, v_absmax=0x6000,
             numel=100, param_dtype=0, grad_dtype=1)
    d.update(kw)
    return B._LtTensor(**d)


def _step(t, block=2048, hp=None, sq=0x7000, n=1):
    hp = hp or L.HParams()
    h = hp.c()
    arr = (B._LtTensor * 1)(t)
    return B._lib.lt_hybrid8_step(C.cast(arr, C.c_void_p), n, block, C.byref(h), sq, None, None)


def test_bad_arguments_are_rejected_on_the_host():
    # none of these may reach the device: the pointers are fake
    assert _step(_tensor(), block=3000) == -3
    assert _step(_tensor(), block=128) == -3
    assert _step(_tensor(), block=32768) == -3
    assert _step(_tensor(numel=-1)) == -1
    assert _step(_tensor(grad=0)) == -1
    assert _step(_tensor(m_code=0)) == -1
    assert _step(_tensor(v_absmax=0)) == -1
    assert _step(_tensor(param_dtype=7)) == -1
    assert _step(_tensor(grad_dtype=-1)) == -1
    assert _step(_tensor(param=0x1002)) == -2          # fp32 parameter at a 2-byte offset
    assert _step(_tensor(grad=0x2001)) == -2           # bf16 gradient at an odd address
    assert _step(_tensor(m_absmax=0x5002)) == -2
    assert _step(_tensor(), hp=L.HParams(step=0)) == -1
    assert _step(_tensor(), hp=L.HParams(beta1=1.0)) == -1
    assert _step(_tensor(), hp=L.HParams(beta2=-0.1)) == -1
    assert _step(_tensor(), hp=L.HParams(eps=-1.0)) == -1
    assert _step(_tensor(), sq=None) == -1              # clipping on but no norm
    assert _step(_tensor(), sq=0x7004) == -2
    assert _step(_tensor(), n=-1) == -1
    arr = (B._LtTensor * 1)(_tensor())
    ws = 0x10000
    f = B._lib.lt_grad_sqnorm_multi
    assert f(C.cast(arr, C.c_void_p), 1, None, ws, 1 << 20, None) == -1
    assert f(C.cast(arr, C.c_void_p), 1, 0x7000, None, 1 << 20, None) == -5
    assert f(C.cast(arr, C.c_void_p), 1, 0x7000, ws, 16, None) == -5
    assert f(C.cast(arr, C.c_void_p), 1, 0x7000, ws + 8, 1 << 20, None) == -5
    assert f(None, 1, 0x7000, ws, 1 << 20, None) == -1
    assert B._lib.lt_hybrid8_state_init(C.cast(arr, C.c_void_p), 1, 1000, None) == -3
    assert L.lt_status_str(0) == "LT_OK" and L.lt_status_str(-2) == "LT_ERR_ALIGNMENT"
    assert B._lib.lt_hybrid8_code_table(1, None) == -1
