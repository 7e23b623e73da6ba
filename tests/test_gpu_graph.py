"""The optimizer step recorded once in a CUDA graph (device-resident step count and step scalars) and
replayed must give what the eager path gives, and match the oracle."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2608_11919_b200 as L
from paper_2608_11919_b200 import workloads as W
from parity_util import compare, oracle_tensors, parallel_oracle_step, refresh_grads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("pd", [torch.float32, torch.bfloat16])
def test_graph_replay_equals_eager_steps_and_oracle(pd):
    torch.cuda.set_device(0)
    spec = W.hybrid_split(W.scaled_decoder_spec("mini", 256, 4, 4, 2, 768, 2048, False, param_dtype=pd), 0.4)
    chunks = W.layer_groups(spec, 2)
    bufs, opts = [], []
    for graphed in (False, True):
        buf = W.Buffers(spec, 2048, DEV)
        W.fill_params(buf)
        tl = L.TensorList.from_buffers(buf)
        ch = [L.TensorList.from_buffers(buf, c) for c in chunks]
        cls = L.GraphedHybrid8Optimizer if graphed else L.Hybrid8Optimizer
        opt = cls(tl, 2048, L.HParams(max_norm=0.5, lr=1e-4), ch)
        opt.init_state()
        bufs.append(buf); opts.append(opt)
    W.fill_grads(bufs[0], 1)
    ots, slices = oracle_tensors(bufs[0])
    ohp = O.HParams(max_norm=0.5, lr=1e-4)
    for k in range(1, 6):
        W.fill_grads(bufs[0], k)
        bufs[1].grad.copy_(bufs[0].grad)               # the graph reads the same buffers every replay
        if k > 1:
            refresh_grads(ots, bufs[0], slices)
        for o in opts:
            o.step()
        torch.cuda.synchronize()
        assert float(opts[0].sqnorm.item()) == float(opts[1].sqnorm.item())
        for key in ("m_code", "v_code", "m_absmax", "v_absmax", "m_f32", "v_f32"):
            a, b = getattr(bufs[0], key), getattr(bufs[1], key)
            if a.dtype == torch.float32:
                a, b = a.view(torch.int32), b.view(torch.int32)
            assert torch.equal(a, b), (k, key)          # the state path does not depend on the step scalars
        pa, pb = bufs[0].param.float(), bufs[1].param.float()
        assert float(((pa - pb).abs() / pa.abs().clamp_min(1e-3)).max()) <= 4e-3 * (pd == torch.bfloat16) + 1e-6
        ohp.step = k
        parallel_oracle_step(ots, 2048, ohp, O.sqnorm(ots))
        compare(bufs[1], ots, slices).check()           # the replayed graph against the oracle
    st = opts[1].state.cpu()
    assert int(st[0]) == 5 and int(opts[1].skip_count.item()) == 0
    scal = st[1:2].view(torch.float32)
    s = O.step_scalars(O.HParams(lr=1e-4, step=5))
    assert abs(float(scal[0]) - s["step_size"]) <= 2e-7 * s["step_size"]
    assert abs(float(scal[1]) - s["inv_sqrt_bc2"]) <= 2e-7 * s["inv_sqrt_bc2"]
