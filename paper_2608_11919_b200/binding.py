"""ctypes binding of liblt_hybrid8.so: argument marshalling only. Every step of the optimizer path
runs in the library's CUDA kernels; PyTorch appears here only as the owner of device memory and of
the CUDA stream."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

LT_F32, LT_BF16 = 0, 1
LT_STATE_U8, LT_STATE_F32 = 0, 1
_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liblt_hybrid8.so")


class LtError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__(f"{fn} failed: {lt_status_str(code)} ({code})")


class _LtTensor(C.Structure):
    _fields_ = [("param", C.c_void_p), ("grad", C.c_void_p), ("m_code", C.c_void_p), ("v_code", C.c_void_p),
                ("m_absmax", C.c_void_p), ("v_absmax", C.c_void_p), ("numel", C.c_int64),
                ("param_dtype", C.c_int32), ("grad_dtype", C.c_int32), ("state_dtype", C.c_int32),
                ("reserved", C.c_int32)]


class _LtHParams(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("max_norm", C.c_float), ("step", C.c_int64)]


def library_path() -> str:
    return _SO


def _load():
    if not os.path.exists(_SO):
        raise ImportError(
            f"{_SO} is missing: build it with `python -m paper_2608_11919_b200.build` "
            "(there is no CPU or PyTorch fallback for this path)")
    L = C.CDLL(_SO)
    L.lt_status_str.argtypes = [C.c_int]; L.lt_status_str.restype = C.c_char_p
    L.lt_hybrid8_state_bytes.argtypes = [C.c_int64, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    L.lt_hybrid8_code_table.argtypes = [C.c_int32, C.c_void_p]
    L.lt_workspace_bytes.argtypes = []; L.lt_workspace_bytes.restype = C.c_int64
    L.lt_hybrid8_state_init.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
    L.lt_grad_sqnorm_multi.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
    L.lt_hybrid8_step.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(_LtHParams), C.c_void_p,
                                  C.c_void_p, C.c_void_p]
    L.lt_grad_sqnorm_multi_noalloc.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    L.lt_grad_sqnorm_per_tensor.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    L.lt_skip_count_update.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    L.lt_step_state_advance.argtypes = [C.c_void_p, C.POINTER(_LtHParams), C.c_void_p, C.c_void_p]
    L.lt_hybrid8_step_graph.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(_LtHParams), C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_void_p]
    return L


_lib = _load()


def lt_status_str(code: int) -> str:
    return _lib.lt_status_str(int(code)).decode()


def _check(fn: str, rc: int) -> None:
    if rc != 0:
        raise LtError(fn, rc)


@dataclass
class HParams:
    lr: float = 1e-5
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01
    max_norm: float = 1.0
    step: int = 1

    def c(self) -> _LtHParams:
        return _LtHParams(self.lr, self.beta1, self.beta2, self.eps, self.weight_decay, self.max_norm, self.step)


def _dt(t: torch.dtype) -> int:
    if t == torch.float32:
        return LT_F32
    if t == torch.bfloat16:
        return LT_BF16
    raise TypeError(f"unsupported dtype {t}")


class TensorList:
    """A host array of lt_tensor descriptors over caller-owned device tensors (kept alive here)."""

    def __init__(self, params: Sequence[torch.Tensor], grads: Sequence[torch.Tensor],
                 m_codes: Sequence[torch.Tensor], v_codes: Sequence[torch.Tensor],
                 m_absmax: Sequence[torch.Tensor], v_absmax: Sequence[torch.Tensor]):
        n = len(params)
        assert all(len(x) == n for x in (grads, m_codes, v_codes, m_absmax, v_absmax))
        self.n = n
        self._keep = (list(params), list(grads), list(m_codes), list(v_codes), list(m_absmax), list(v_absmax))
        self.array = (_LtTensor * max(n, 1))()
        for i in range(n):
            p, g = params[i], grads[i]
            assert p.is_contiguous() and g.is_contiguous() and p.numel() == g.numel()
            st32 = m_codes[i].dtype == torch.float32        # plain fp32 moments instead of 8-bit codes
            assert m_codes[i].dtype == v_codes[i].dtype and (st32 or m_codes[i].dtype == torch.uint8)
            self.array[i] = _LtTensor(p.data_ptr(), g.data_ptr(), m_codes[i].data_ptr(), v_codes[i].data_ptr(),
                                      0 if st32 else m_absmax[i].data_ptr(), 0 if st32 else v_absmax[i].data_ptr(),
                                      p.numel(), _dt(p.dtype), _dt(g.dtype), LT_STATE_F32 if st32 else LT_STATE_U8, 0)

    @classmethod
    def from_buffers(cls, buf, indices: Optional[Sequence[int]] = None) -> "TensorList":
        """Descriptors over the flat buffers of a `workloads.Buffers` (all tensors, or a subset)."""
        idx = range(len(buf.spec.sizes)) if indices is None else indices
        return cls(*[[buf.view(k, t) for t in idx]
                     for k in ("param", "grad", "m_code", "v_code", "m_absmax", "v_absmax")])

    @classmethod
    def from_buffer_pieces(cls, buf, pieces) -> "TensorList":
        """Descriptors over block-aligned pieces (tensor index, first block, number of blocks) of the tensors
        of a `workloads.Buffers`, as `sharding.partition_blocks` hands them out."""
        cols = [[] for _ in range(6)]
        for t, b0, nb in pieces:
            size = buf.spec.sizes[t]
            e0, e1 = b0 * buf.block, min(size, (b0 + nb) * buf.block)
            for c, k in zip(cols, ("param", "grad", "m_code", "v_code")):
                c.append(buf.view(k, t)[e0:e1])
            for c, k in zip(cols[4:], ("m_absmax", "v_absmax")):
                c.append(buf.view(k, t)[b0:b0 + nb])
        return cls(*cols)

    def slice(self, start: int, stop: int) -> "TensorList":
        return TensorList(*[x[start:stop] for x in self._keep])

    @property
    def ptr(self):
        return C.cast(self.array, C.c_void_p)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream
    return int(stream)


def lt_hybrid8_state_bytes(numel: int, block: int):
    a, b = C.c_int64(0), C.c_int64(0)
    _check("lt_hybrid8_state_bytes", _lib.lt_hybrid8_state_bytes(numel, block, C.byref(a), C.byref(b)))
    return a.value, b.value


def lt_hybrid8_code_table(is_signed: bool) -> torch.Tensor:
    out = torch.empty(256, dtype=torch.float32)
    _check("lt_hybrid8_code_table", _lib.lt_hybrid8_code_table(int(is_signed), out.data_ptr()))
    return out


def lt_workspace_bytes() -> int:
    return int(_lib.lt_workspace_bytes())


def lt_hybrid8_state_init(tensors: TensorList, block: int, stream=None) -> None:
    _check("lt_hybrid8_state_init", _lib.lt_hybrid8_state_init(tensors.ptr, tensors.n, block, _stream(stream)))


def lt_grad_sqnorm_multi(tensors: TensorList, d_sqnorm: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    assert d_sqnorm.dtype == torch.float64 and d_sqnorm.is_cuda
    _check("lt_grad_sqnorm_multi",
           _lib.lt_grad_sqnorm_multi(tensors.ptr, tensors.n, d_sqnorm.data_ptr(), workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(), _stream(stream)))


def lt_grad_sqnorm_multi_noalloc(tensors: TensorList, d_sqnorm: torch.Tensor, stream=None) -> None:
    """Squared-norm accumulation for callers that cannot provide device scratch: the library's own
    fixed device array is used instead (shared by all calls on the device, so calls must not overlap
    on the GPU; at most 480 non-empty tensors per call; first call before any stream capture)."""
    assert d_sqnorm.dtype == torch.float64 and d_sqnorm.is_cuda
    _check("lt_grad_sqnorm_multi_noalloc",
           _lib.lt_grad_sqnorm_multi_noalloc(tensors.ptr, tensors.n, d_sqnorm.data_ptr(), _stream(stream)))


def lt_grad_sqnorm_per_tensor(tensors: TensorList, d_out: torch.Tensor, stream=None) -> None:
    assert d_out.dtype == torch.float64 and d_out.is_cuda and d_out.numel() >= tensors.n
    _check("lt_grad_sqnorm_per_tensor",
           _lib.lt_grad_sqnorm_per_tensor(tensors.ptr, tensors.n, d_out.data_ptr(), _stream(stream)))


def lt_skip_count_update(d_sqnorm: torch.Tensor, d_skip_count: torch.Tensor, stream=None) -> None:
    assert d_sqnorm.dtype == torch.float64 and d_skip_count.dtype == torch.int32
    _check("lt_skip_count_update",
           _lib.lt_skip_count_update(d_sqnorm.data_ptr(), d_skip_count.data_ptr(), _stream(stream)))


def lt_hybrid8_step(tensors: TensorList, block: int, hp: HParams, d_sqnorm: Optional[torch.Tensor],
                    d_status: Optional[torch.Tensor], stream=None) -> None:
    h = hp.c()
    _check("lt_hybrid8_step",
           _lib.lt_hybrid8_step(tensors.ptr, tensors.n, block, C.byref(h),
                                None if d_sqnorm is None else d_sqnorm.data_ptr(),
                                None if d_status is None else d_status.data_ptr(), _stream(stream)))


def lt_step_state_advance(d_state: torch.Tensor, hp: HParams, d_sqnorm: Optional[torch.Tensor] = None, stream=None) -> None:
    """d_state: 16 bytes of device memory (an lt_step_state), zeroed once by the caller. With d_sqnorm the
    count stays where it is when the norm is not finite (the step that follows is skipped)."""
    assert d_state.is_cuda and d_state.numel() * d_state.element_size() >= 16
    h = hp.c()
    _check("lt_step_state_advance",
           _lib.lt_step_state_advance(d_state.data_ptr(), C.byref(h),
                                      None if d_sqnorm is None else d_sqnorm.data_ptr(), _stream(stream)))


def lt_hybrid8_step_graph(tensors: TensorList, block: int, hp: HParams, d_state: torch.Tensor,
                          d_sqnorm: Optional[torch.Tensor], d_status: Optional[torch.Tensor], stream=None) -> None:
    h = hp.c()
    _check("lt_hybrid8_step_graph",
           _lib.lt_hybrid8_step_graph(tensors.ptr, tensors.n, block, C.byref(h), d_state.data_ptr(),
                                      None if d_sqnorm is None else d_sqnorm.data_ptr(),
                                      None if d_status is None else d_status.data_ptr(), _stream(stream)))


class GraphedHybrid8Optimizer:
    """The whole optimizer step recorded once in a CUDA graph and replayed: zero the norm, norm over all
    chunks, skip bookkeeping, advance the device-resident step state, update all chunks. Between replays the
    caller only writes new gradients into the same buffers."""

    def __init__(self, tensors: TensorList, block: int, hp: HParams, chunks: Optional[Sequence[TensorList]] = None,
                 device=None):
        device = device if device is not None else tensors._keep[0][0].device
        self.tensors, self.block, self.hp = tensors, block, hp
        self.chunks = list(chunks) if chunks is not None else [tensors]
        self.sqnorm = torch.zeros(1, dtype=torch.float64, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.skip_count = torch.zeros(1, dtype=torch.int32, device=device)
        self.state = torch.zeros(2, dtype=torch.int64, device=device)       # an lt_step_state, step 0
        self.workspace = torch.empty(lt_workspace_bytes(), dtype=torch.uint8, device=device)
        self.graph = None

    def init_state(self) -> None:
        lt_hybrid8_state_init(self.tensors, self.block)

    def _enqueue(self) -> None:
        self.sqnorm.zero_()
        for ch in self.chunks:
            lt_grad_sqnorm_multi(ch, self.sqnorm, self.workspace)
        lt_skip_count_update(self.sqnorm, self.skip_count)
        lt_step_state_advance(self.state, self.hp, self.sqnorm)
        for ch in self.chunks:
            lt_hybrid8_step_graph(ch, self.block, self.hp, self.state, self.sqnorm, self.status)

    def step(self) -> None:
        if self.graph is None:
            self._enqueue()                      # first step eagerly: one-time set-up must not be captured
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self._enqueue()
            self.graph = g
            return
        self.graph.replay()


class Hybrid8Optimizer:
    """Convenience driver: owns the norm scalar, the status word and the norm scratch, and enqueues
    zero -> norm (all chunks) -> step (all chunks) on torch's current stream. No host synchronisation."""

    def __init__(self, tensors: TensorList, block: int, hp: HParams, chunks: Optional[Sequence[TensorList]] = None,
                 device=None):
        device = device if device is not None else tensors._keep[0][0].device
        self.tensors, self.block, self.hp = tensors, block, hp
        self.chunks = list(chunks) if chunks is not None else [tensors]
        self.sqnorm = torch.zeros(1, dtype=torch.float64, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.workspace = torch.empty(lt_workspace_bytes(), dtype=torch.uint8, device=device)
        self.skip_count = torch.zeros(1, dtype=torch.int32, device=device)   # consecutive non-finite steps
        self.t = 0

    def init_state(self) -> None:
        lt_hybrid8_state_init(self.tensors, self.block)

    def step(self) -> None:
        self.t += 1
        self.hp.step = self.t
        self.sqnorm.zero_()
        for ch in self.chunks:
            lt_grad_sqnorm_multi(ch, self.sqnorm, self.workspace)
        lt_skip_count_update(self.sqnorm, self.skip_count)
        for ch in self.chunks:
            lt_hybrid8_step(ch, self.block, self.hp, self.sqnorm, self.status)

    def settle_skipped_step(self) -> bool:
        """Reads the status word (a host synchronisation, so the caller picks the moment: typically where it
        reads the loss). If the last step was skipped for a non-finite norm, the step count goes back by one,
        so that skipped steps do not count towards the bias corrections, and the skip bit is cleared.
        Returns whether a step had been skipped. Call it after every step that may have been skipped: the
        host forms the step scalars from this count, and the bit does not say how many steps set it."""
        st = int(self.status.item())
        if st & 1:
            self.t -= 1
            self.status.fill_(st & ~1)
            return True
        return False
