"""Host-resident variant: parameters, gradients and optimizer state live in pinned HOST memory (the
paper's layout, Sec. 3.5: master parameters and optimizer states stay in CPU memory) and are streamed through
the same kernels chunk by chunk, with copies and compute overlapped on three streams.

Per optimizer step:
  pass 1  every chunk's gradients  H2D -> lt_grad_sqnorm_multi  (one device scalar; the gradients stay on
          the device if `keep_grads` so that pass 2 does not send them again)
  pass 2  every chunk: parameters + state H2D -> lt_hybrid8_step -> parameters + state D2H
          (two staging slots: chunk k+1 is copied in while chunk k is updated and chunk k-1 is copied out)
The bound is the host link, not HBM: per parameter 8 bytes go in (gradient, fp32 parameter, two codes) and 6
come back, and while both directions are busy each gets less than it gets alone, so the floor of a step is
(bytes out) / (per-direction rate with both busy) + (bytes in - bytes out) / (one-direction rate). This module
is plumbing only: every arithmetic step is in the library's kernels.

The host side is a `HostTensors`: per-tensor pinned tensors the caller owns (a trainer's own master weights,
gradients and state), or the flat buffers of a synthetic workload through `HostTensors.from_buffers`.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as B

_KEYS = ("param", "m_code", "v_code", "m_absmax", "v_absmax")


class HostTensors:
    """The host side of the optimizer: one pinned CPU tensor per model tensor and kind.

    params[t], grads[t]: [numel_t]; m_state[t], v_state[t]: uint8 [numel_t] codes, or float32 [numel_t] moments for
    a tensor with plain fp32 state; m_absmax[t], v_absmax[t]: float32 [ceil(numel_t / block)] (ignored, may be
    None, for fp32-state tensors). All parameters share one dtype, all gradients share one dtype. Tensors that
    lie back to back in host memory are copied with one transfer."""

    def __init__(self, params, grads, m_state, v_state, m_absmax, v_absmax):
        n = len(params)
        assert all(len(x) == n for x in (grads, m_state, v_state, m_absmax, v_absmax))
        self._t = {"param": list(params), "grad": list(grads), "m_code": list(m_state), "v_code": list(v_state),
                   "m_absmax": list(m_absmax), "v_absmax": list(v_absmax)}
        self.sizes = [int(p.numel()) for p in params]
        self.f32 = [m.dtype == torch.float32 for m in m_state]
        self.param_dtype = params[0].dtype if n else torch.float32
        self.grad_dtype = grads[0].dtype if n else torch.bfloat16
        for t in range(n):
            assert params[t].dtype == self.param_dtype and grads[t].dtype == self.grad_dtype
            assert grads[t].numel() == self.sizes[t] and m_state[t].numel() == self.sizes[t]
            for k in ("param", "grad", "m_code", "v_code"):
                x = self._t[k][t]
                assert x.device.type == "cpu" and x.is_contiguous() and (x.numel() == 0 or x.is_pinned()), \
                    "host tensors must be contiguous pinned CPU memory"
        self._empty = torch.empty(0, dtype=torch.float32)

    @classmethod
    def from_buffers(cls, buf) -> "HostTensors":
        """Views of the flat host buffers of a `workloads.Buffers` (allocated with pin=True)."""
        n = len(buf.spec.sizes)
        return cls(*[[buf.view(k, t) for t in range(n)]
                     for k in ("param", "grad", "m_code", "v_code", "m_absmax", "v_absmax")])

    def view(self, key: str, t: int) -> torch.Tensor:
        x = self._t[key][t]
        if key in ("m_absmax", "v_absmax") and (self.f32[t] or x is None):
            return self._empty
        return x


class _Slot:
    """Device staging for one chunk: flat buffers big enough for the largest chunk."""

    def __init__(self, host: HostTensors, max_elems: int, max_blocks: int, max_f32: int, device):
        spec = host
        kw = dict(device=device)
        self.param = torch.empty(max(max_elems, 1), dtype=spec.param_dtype, **kw)
        self.grad = torch.empty(max(max_elems, 1), dtype=spec.grad_dtype, **kw)
        self.m_code = torch.empty(max(max_elems, 1), dtype=torch.uint8, **kw)
        self.v_code = torch.empty(max(max_elems, 1), dtype=torch.uint8, **kw)
        self.m_absmax = torch.empty(max(max_blocks, 1), dtype=torch.float32, **kw)
        self.v_absmax = torch.empty(max(max_blocks, 1), dtype=torch.float32, **kw)
        self.m_f32 = torch.empty(max(max_f32, 1), dtype=torch.float32, **kw)
        self.v_f32 = torch.empty(max(max_f32, 1), dtype=torch.float32, **kw)
        self.filled = torch.cuda.Event()     # H2D of the chunk in this slot is complete
        self.stepped = torch.cuda.Event()    # the step on this slot is complete
        self.drained = torch.cuda.Event()    # D2H of this slot is complete (slot reusable)
        self.drained.record()


class HostResidentOptimizer:
    def __init__(self, host, block: int, hp: B.HParams, chunks: Sequence[Sequence[int]],
                 device="cuda:0", keep_grads: bool = True, n_slots: int = 3):
        """host: a HostTensors (or a pinned `workloads.Buffers`, wrapped here). chunks: lists of tensor indices,
        updated one chunk at a time under one global clip norm. n_slots device staging buffers (of the largest
        chunk's size) let copy-in, update and copy-out of neighbouring chunks overlap."""
        if not isinstance(host, HostTensors):
            host = HostTensors.from_buffers(host)
        self.host, self.block, self.hp = host, int(block), hp
        self.device = torch.device(device)
        self.chunks = [list(c) for c in chunks if len(c)]
        spec, a = host, 16          # tensors start on 16-element boundaries inside the staging buffers
        # placement of every tensor inside its chunk's staging buffers
        self.place = {}
        max_e = max_b = max_f = 0
        for c in self.chunks:
            e = b = f = e8 = 0
            for t in c:
                s = spec.sizes[t]
                e = (e + a - 1) // a * a; e8 = (e8 + a - 1) // a * a; f = (f + a - 1) // a * a
                nb = 0 if host.f32[t] else (s + block - 1) // block
                self.place[t] = (e, e8, b, f)
                e += s
                if host.f32[t]:
                    f += s
                else:
                    e8 += s; b += nb
            max_e, max_b, max_f = max(max_e, e), max(max_b, b), max(max_f, f)
        self.slots = [_Slot(host, max_e, max_b, max_f, self.device) for _ in range(max(2, int(n_slots)))]
        self.n_slots = len(self.slots)
        self.keep_grads = keep_grads
        self.goff, o = [], 0       # placement of every tensor's gradient in the device-resident gradient buffer
        for sz in spec.sizes:
            o = (o + a - 1) // a * a
            self.goff.append(o)
            o += sz
        self.dev_grad = torch.empty(max(o, 1), dtype=spec.grad_dtype, device=self.device) if keep_grads else None
        self.sqnorm = torch.zeros(1, dtype=torch.float64, device=self.device)
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.workspace = torch.empty(B.lt_workspace_bytes(), dtype=torch.uint8, device=self.device)
        self.result = torch.zeros(2, dtype=torch.float64).pin_memory()
        self.h2d, self.d2h = torch.cuda.Stream(self.device), torch.cuda.Stream(self.device)
        # descriptor lists: norm lists over the resident gradients (or slot gradients), step lists per (chunk, slot)
        self.lists = {}
        for ci, c in enumerate(self.chunks):
            for si, sl in enumerate(self.slots):
                self.lists[(ci, si)] = B.TensorList(*[[self._dev(sl, k, t) for t in c]
                                                      for k in ("param", "grad", "m_code", "v_code", "m_absmax", "v_absmax")])
        # copy plans: per (chunk, slot, key) a few long (device view, host view) pairs instead of one per tensor
        self.plan = {}
        for ci, c in enumerate(self.chunks):
            for si, sl in enumerate(self.slots):
                for k in _KEYS + ("grad",):
                    self.plan[(ci, si, k)] = self._runs(sl, k, c)
        self.t = 0
        self.h2d_bytes = self.d2h_bytes = 0

    def _runs(self, sl: _Slot, key: str, chunk: List[int]):
        """Merges tensors that are adjacent both on the host and in the slot into single copies."""
        out = []
        for t in chunk:
            d, h = self._dev(sl, key, t), self.host.view(key, t)
            if d.numel() == 0:
                continue
            if out:
                pd, ph = out[-1]
                es = d.element_size()
                if (pd.untyped_storage().data_ptr() == d.untyped_storage().data_ptr() and
                        ph.untyped_storage().data_ptr() == h.untyped_storage().data_ptr() and
                        pd.data_ptr() + pd.numel() * es == d.data_ptr() and ph.data_ptr() + ph.numel() * es == h.data_ptr()):
                    n = pd.numel() + d.numel()
                    out[-1] = (pd.as_strided((n,), (1,), pd.storage_offset()), ph.as_strided((n,), (1,), ph.storage_offset()))
                    continue
            out.append((d, h))
        return out

    # device view of tensor t inside a slot
    def _dev(self, sl: _Slot, key: str, t: int) -> torch.Tensor:
        e, e8, b, f = self.place[t]
        s = self.host.sizes[t]
        f32 = self.host.f32[t]
        if key == "grad" and self.keep_grads:
            return self.dev_grad[self.goff[t]: self.goff[t] + s]
        if key in ("param", "grad"):
            return getattr(sl, key)[e: e + s]
        if key in ("m_code", "v_code"):
            return (sl.m_f32 if key == "m_code" else sl.v_f32)[f: f + s] if f32 else getattr(sl, key)[e8: e8 + s]
        nb = 0 if f32 else (s + self.block - 1) // self.block
        return getattr(sl, key)[b: b + nb]

    def _copy(self, dst: torch.Tensor, src: torch.Tensor) -> int:
        if dst.numel():
            dst.copy_(src, non_blocking=True)
        return dst.numel() * dst.element_size()

    def init_state(self) -> None:
        """Value-zero state, produced by the library's kernel on the device and copied out to the host."""
        main = torch.cuda.current_stream(self.device)
        for ci, c in enumerate(self.chunks):
            sl = self.slots[0]
            B.lt_hybrid8_state_init(self.lists[(ci, 0)], self.block)
            for t in c:
                for k in ("m_code", "v_code", "m_absmax", "v_absmax"):
                    self._copy(self.host.view(k, t), self._dev(sl, k, t))
            main.synchronize()

    def step(self) -> None:
        main = torch.cuda.current_stream(self.device)
        host = self.host
        self.t += 1
        self.hp.step = self.t
        self.sqnorm.zero_()
        h2d = d2h = 0
        # pass 1: gradients in, norm
        self.h2d.wait_stream(main)
        for ci, c in enumerate(self.chunks):
            sl = self.slots[ci % self.n_slots]
            with torch.cuda.stream(self.h2d):
                if not self.keep_grads:
                    self.h2d.wait_event(sl.stepped)     # the slot's previous gradients have been read
                for d, h in self.plan[(ci, ci % self.n_slots, "grad")]:
                    h2d += self._copy(d, h)
                sl.filled.record(self.h2d)
            main.wait_event(sl.filled)
            B.lt_grad_sqnorm_multi(self.lists[(ci, ci % self.n_slots)], self.sqnorm, self.workspace)
            sl.stepped.record(main)
        # pass 2: parameters and state in, step, out
        for ci, c in enumerate(self.chunks):
            si = ci % self.n_slots
            sl = self.slots[si]
            with torch.cuda.stream(self.h2d):
                self.h2d.wait_event(sl.drained)         # the slot's previous results have left
                self.h2d.wait_event(sl.stepped)         # and nothing on the compute stream still reads it
                for k in _KEYS + (() if self.keep_grads else ("grad",)):
                    for d, h in self.plan[(ci, si, k)]:
                        h2d += self._copy(d, h)
                sl.filled.record(self.h2d)
            main.wait_event(sl.filled)
            B.lt_hybrid8_step(self.lists[(ci, si)], self.block, self.hp, self.sqnorm, self.status)
            sl.stepped.record(main)
            with torch.cuda.stream(self.d2h):
                self.d2h.wait_event(sl.stepped)
                for k in _KEYS:
                    for d, h in self.plan[(ci, si, k)]:
                        d2h += self._copy(h, d)
                sl.drained.record(self.d2h)
        main.wait_stream(self.d2h)
        self.result[0:1].copy_(self.sqnorm, non_blocking=True)
        self.result[1:2].copy_(self.status.to(torch.float64), non_blocking=True)
        self.h2d_bytes, self.d2h_bytes = h2d, d2h + 16
