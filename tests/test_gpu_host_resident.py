"""Host-resident variant: state in pinned host memory streamed through the kernels in chunks must give
exactly what the device-resident optimizer gives with the same chunking, and match the oracle."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2608_11919_b200 as L
from paper_2608_11919_b200 import workloads as W
from paper_2608_11919_b200.host_resident import HostResidentOptimizer
from parity_util import compare, oracle_tensors, parallel_oracle_step, refresh_grads

pytestmark = pytest.mark.gpu
BLOCK = 2048


@pytest.mark.parametrize("keep_grads", [True, False])
def test_host_resident_equals_device_resident_and_oracle(keep_grads):
    torch.cuda.set_device(0)
    spec = W.hybrid_split(W.scaled_decoder_spec("mini", 256, 5, 4, 2, 768, 4096, False), 0.3)
    chunks = W.layer_groups(spec, 2)
    host = W.Buffers(spec, BLOCK, "cpu", pin=True)
    dev = W.Buffers(spec, BLOCK, "cuda:0")
    W.fill_params(dev)
    host.param.copy_(dev.param)
    hopt = HostResidentOptimizer(host, BLOCK, L.HParams(max_norm=0.5), chunks, keep_grads=keep_grads)
    hopt.init_state()
    tl = L.TensorList.from_buffers(dev)
    dopt = L.Hybrid8Optimizer(tl, BLOCK, L.HParams(max_norm=0.5), [L.TensorList.from_buffers(dev, c) for c in chunks])
    dopt.init_state()
    W.fill_grads(dev, 1)
    ots, slices = oracle_tensors(dev)
    ohp = O.HParams(max_norm=0.5)
    for k in (1, 2, 3):
        W.fill_grads(dev, k)
        host.grad.copy_(dev.grad)
        if k > 1:
            refresh_grads(ots, dev, slices)
        dopt.step()
        hopt.step()
        torch.cuda.synchronize()
        assert float(hopt.result[0]) == float(dopt.sqnorm.item())
        for key in ("param", "m_code", "v_code", "m_absmax", "v_absmax", "m_f32", "v_f32"):
            a, b = getattr(host, key), getattr(dev, key).cpu()
            if a.dtype.is_floating_point:
                a, b = a.view(torch.int16 if a.element_size() == 2 else torch.int32), b.view(torch.int16 if b.element_size() == 2 else torch.int32)
            assert torch.equal(a, b), (k, key)
        ohp.step = k
        parallel_oracle_step(ots, BLOCK, ohp, O.sqnorm(ots))
        compare(dev, ots, slices).check()
    assert hopt.h2d_bytes > 0 and hopt.d2h_bytes > 0 and float(hopt.result[1]) == 0.0


def test_host_resident_over_caller_owned_pinned_tensors():
    """The same with the host side given as separately allocated pinned tensors (a trainer's own master
    weights, gradients and state), no workload container involved."""
    from paper_2608_11919_b200.host_resident import HostTensors
    torch.cuda.set_device(0)
    spec = W.hybrid_split(W.scaled_decoder_spec("mini", 256, 4, 4, 2, 768, 4096, True, param_dtype=torch.bfloat16), 0.4)
    chunks = W.layer_groups(spec, 2)
    dev = W.Buffers(spec, BLOCK, "cuda:0")
    W.fill_params(dev)
    n = len(spec.sizes)

    def pinned(x):
        return torch.empty(x.shape, dtype=x.dtype).pin_memory().copy_(x)

    cols = {k: [pinned(dev.view(k, t).cpu()) for t in range(n)]
            for k in ("param", "grad", "m_code", "v_code", "m_absmax", "v_absmax")}
    host = HostTensors(cols["param"], cols["grad"], cols["m_code"], cols["v_code"], cols["m_absmax"], cols["v_absmax"])
    hopt = HostResidentOptimizer(host, BLOCK, L.HParams(max_norm=0.5), chunks)
    hopt.init_state()
    dopt = L.Hybrid8Optimizer(L.TensorList.from_buffers(dev), BLOCK, L.HParams(max_norm=0.5),
                              [L.TensorList.from_buffers(dev, c) for c in chunks])
    dopt.init_state()
    for k in (1, 2, 3):
        W.fill_grads(dev, k)
        for t in range(n):
            cols["grad"][t].copy_(dev.view("grad", t))
        dopt.step()
        hopt.step()
        torch.cuda.synchronize()
        assert float(hopt.result[0]) == float(dopt.sqnorm.item()) and float(hopt.result[1]) == 0.0
        for key in ("param", "m_code", "v_code", "m_absmax", "v_absmax"):
            for t in range(n):
                a, b = host.view(key, t), dev.view(key, t).cpu()
                if a.dtype.is_floating_point:
                    iv = torch.int16 if a.element_size() == 2 else torch.int32
                    a, b = a.view(iv), b.view(iv)
                assert torch.equal(a, b), (k, key, t)
