"""lt_grad_sqnorm_multi_noalloc: the squared-norm entry point for callers that cannot allocate device
scratch (they run under an allocator they may not call, or where cudaMalloc would stall the device).
It must give what lt_grad_sqnorm_multi gives, call after call, although every call reuses the same
library-owned device array. Collected last on purpose: a failure here cannot hide another test."""
import ctypes as C

import pytest
import torch

import paper_2608_11919_b200 as L
from paper_2608_11919_b200 import binding as B
from paper_2608_11919_b200 import workloads as W

DEV = "cuda:0"


@pytest.mark.gpu
def test_noalloc_norm_matches_workspace_norm_twice_in_a_row():
    torch.cuda.set_device(0)
    spec = W.ragged_spec(n_tensors=400, max_numel=1 << 18, seed=17)     # unaligned bases, ragged sizes
    buf = W.Buffers(spec, 2048, DEV)
    ws = torch.empty(L.lt_workspace_bytes(), dtype=torch.uint8, device=DEV)
    tl = L.TensorList.from_buffers(buf)
    for call in (1, 2):                        # second call meets the array as the first one left it
        W.fill_grads(buf, call)
        ref = torch.zeros(1, dtype=torch.float64, device=DEV)
        got = torch.full((1,), 3.0, dtype=torch.float64, device=DEV)    # accumulates onto what is there
        L.lt_grad_sqnorm_multi(tl, ref, ws)
        L.lt_grad_sqnorm_multi_noalloc(tl, got)
        torch.cuda.synchronize()
        r, g = float(ref.item()), float(got.item()) - 3.0
        assert r > 0 and abs(g - r) <= 1e-9 * r, (call, g, r)
    # a chunked list through the same array, and an empty list
    got = torch.zeros(1, dtype=torch.float64, device=DEV)
    for a in range(0, tl.n, 150):
        L.lt_grad_sqnorm_multi_noalloc(tl.slice(a, a + 150), got)
    L.lt_grad_sqnorm_multi_noalloc(tl.slice(0, 0), got)
    torch.cuda.synchronize()
    assert abs(float(got.item()) - r) <= 1e-9 * r


@pytest.mark.gpu
def test_noalloc_rejects_lists_beyond_its_maximum():
    torch.cuda.set_device(0)
    n = 481
    spec = W.ragged_spec(n_tensors=n, max_numel=64, seed=18)
    buf = W.Buffers(spec, 2048, DEV)
    buf.grad.zero_()
    tl = L.TensorList.from_buffers(buf)
    acc = torch.zeros(1, dtype=torch.float64, device=DEV)
    with pytest.raises(L.LtError) as e:
        L.lt_grad_sqnorm_multi_noalloc(tl, acc)
    assert e.value.code == -5
    L.lt_grad_sqnorm_multi_noalloc(tl.slice(0, 480), acc)              # exactly the maximum is fine
    torch.cuda.synchronize()
    assert float(acc.item()) == 0.0


def test_noalloc_argument_checks_on_the_host():
    t = B._LtTensor(param=0, grad=0x2000, m_code=0, v_code=0, m_absmax=0, v_absmax=0, numel=8,
                    param_dtype=0, grad_dtype=1)
    arr = (B._LtTensor * 1)(t)
    f = B._lib.lt_grad_sqnorm_multi_noalloc
    assert f(C.cast(arr, C.c_void_p), 1, None, None) == -1
    assert f(None, 1, 0x7000, None) == -1
    assert f(C.cast(arr, C.c_void_p), 1, 0x7004, None) == -2
    arr[0].grad = 0x2001
    assert f(C.cast(arr, C.c_void_p), 1, 0x7000, None) == -2
    arr[0].grad = 0
    assert f(C.cast(arr, C.c_void_p), 1, 0x7000, None) == -1
