"""ctypes marshalling for the CPU oracle (test infrastructure; holds no arithmetic of the method
beyond bf16 <-> fp32 bit conversions needed to hand numpy arrays across)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from dataclasses import dataclass

import numpy as np

F32, BF16 = 0, 1
_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lt_oracle.cpp")
_SO = os.path.join(_HERE, "liblt_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile lt_oracle.cpp with g++ (no FMA contraction) into liblt_oracle.so beside it."""
    with _lock:
        if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
            tmp = _SO + f".tmp{os.getpid()}"
            cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
                   "-Wall", "-Wextra", "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _SO)
    return _SO


class _Tensor(C.Structure):
    _fields_ = [("param", C.c_void_p), ("grad", C.c_void_p), ("m_code", C.c_void_p), ("v_code", C.c_void_p),
                ("m_absmax", C.c_void_p), ("v_absmax", C.c_void_p), ("numel", C.c_int64),
                ("param_dtype", C.c_int32), ("grad_dtype", C.c_int32), ("state_dtype", C.c_int32),
                ("reserved", C.c_int32)]


class _HParams(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("max_norm", C.c_float), ("step", C.c_int64)]


class _Scalars(C.Structure):
    _fields_ = [(k, C.c_float) for k in
                ("step_size", "inv_sqrt_bc2", "decay", "omb1", "omb2", "beta1", "beta2", "eps")]


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.lto_code_table.argtypes = [C.c_int, C.c_void_p]
        L.lto_nearest.argtypes = [C.c_int, C.c_float]
        L.lto_nearest.restype = C.c_int
        L.lto_nearest_brute.argtypes = [C.c_int, C.c_float]
        L.lto_nearest_brute.restype = C.c_int
        L.lto_state_bytes.argtypes = [C.c_int64, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.lto_sqnorm_accumulate.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.c_double]
        L.lto_sqnorm_accumulate.restype = C.c_double
        L.lto_grad_sqnorm_multi.argtypes = [C.POINTER(_Tensor), C.c_int32, C.c_double]
        L.lto_grad_sqnorm_multi.restype = C.c_double
        L.lto_clip_factor.argtypes = [C.c_double, C.c_float, C.POINTER(C.c_int32)]
        L.lto_clip_factor.restype = C.c_float
        L.lto_step_scalars.argtypes = [C.POINTER(_HParams), C.POINTER(_Scalars)]
        L.lto_state_init.argtypes = [C.POINTER(_Tensor), C.c_int32, C.c_int32]
        L.lto_hybrid8_step.argtypes = [C.POINTER(_Tensor), C.c_int32, C.c_int32, C.POINTER(_HParams),
                                       C.c_double, C.POINTER(C.c_int32), C.c_int32]
        L.lto_hybrid8_step.restype = C.c_int32
        L.lto_step_fp32state.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                         C.POINTER(_HParams), C.c_float]
        L.lto_dequant.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p]
        _lib = L
    return _lib


@dataclass
class HParams:
    lr: float = 1e-5
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01
    max_norm: float = 1.0
    step: int = 1

    def c(self) -> _HParams:
        return _HParams(self.lr, self.beta1, self.beta2, self.eps, self.weight_decay, self.max_norm, self.step)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float32 values (exact)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns, round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


class OracleTensor:
    """One tensor's host arrays: param (float32, or uint16 bf16 bits), grad (uint16 bf16 bits or
    float32), m_code / v_code (uint8), m_absmax / v_absmax (float32, one per block)."""

    def __init__(self, param: np.ndarray, grad: np.ndarray, block: int,
                 m_code=None, v_code=None, m_absmax=None, v_absmax=None, fp32_state: bool = False):
        self.param = np.ascontiguousarray(param).reshape(-1)
        self.grad = np.ascontiguousarray(grad).reshape(-1)
        assert self.param.dtype in (np.float32, np.uint16) and self.grad.dtype in (np.float32, np.uint16)
        assert self.param.size == self.grad.size
        self.numel = int(self.param.size)
        self.block = int(block)
        nb = (self.numel + block - 1) // block
        self.fp32_state = bool(fp32_state) or (m_code is not None and np.asarray(m_code).dtype == np.float32)
        if self.fp32_state:       # plain fp32 moments live in m_code / v_code; the scale arrays are unused
            self.m_code = np.zeros(self.numel, np.float32) if m_code is None else np.ascontiguousarray(m_code, np.float32)
            self.v_code = np.zeros(self.numel, np.float32) if v_code is None else np.ascontiguousarray(v_code, np.float32)
            self.m_absmax = np.zeros(nb, np.float32)
            self.v_absmax = np.zeros(nb, np.float32)
            return
        self.m_code = np.full(self.numel, 127, np.uint8) if m_code is None else np.ascontiguousarray(m_code, np.uint8)
        self.v_code = np.zeros(self.numel, np.uint8) if v_code is None else np.ascontiguousarray(v_code, np.uint8)
        self.m_absmax = np.zeros(nb, np.float32) if m_absmax is None else np.ascontiguousarray(m_absmax, np.float32)
        self.v_absmax = np.zeros(nb, np.float32) if v_absmax is None else np.ascontiguousarray(v_absmax, np.float32)
        assert self.m_code.size == self.numel and self.v_code.size == self.numel
        assert self.m_absmax.size == nb and self.v_absmax.size == nb

    @property
    def param_dtype(self) -> int:
        return F32 if self.param.dtype == np.float32 else BF16

    @property
    def grad_dtype(self) -> int:
        return F32 if self.grad.dtype == np.float32 else BF16

    def set_grad(self, grad: np.ndarray) -> None:
        g = np.ascontiguousarray(grad).reshape(-1)
        assert g.size == self.numel and g.dtype in (np.float32, np.uint16)
        self.grad = g

    def c(self) -> _Tensor:
        p = lambda a: a.ctypes.data_as(C.c_void_p)  # noqa: E731
        return _Tensor(p(self.param), p(self.grad), p(self.m_code), p(self.v_code), p(self.m_absmax),
                       p(self.v_absmax), self.numel, self.param_dtype, self.grad_dtype,
                       1 if self.fp32_state else 0, 0)


def _carray(tensors):
    arr = (_Tensor * max(1, len(tensors)))()
    for i, t in enumerate(tensors):
        arr[i] = t.c()
    return arr


def code_table(is_signed: bool) -> np.ndarray:
    out = np.zeros(256, np.float32)
    lib().lto_code_table(int(is_signed), out.ctypes.data_as(C.c_void_p))
    return out


def nearest(is_signed: bool, x: float) -> int:
    return int(lib().lto_nearest(int(is_signed), float(np.float32(x))))


def nearest_brute(is_signed: bool, x: float) -> int:
    return int(lib().lto_nearest_brute(int(is_signed), float(np.float32(x))))


def state_bytes(numel: int, block: int):
    a, b = C.c_int64(0), C.c_int64(0)
    lib().lto_state_bytes(numel, block, C.byref(a), C.byref(b))
    return a.value, b.value


def sqnorm(tensors, S: float = 0.0) -> float:
    return float(lib().lto_grad_sqnorm_multi(_carray(tensors), len(tensors), S))


def clip_factor(S: float, max_norm: float):
    nf = C.c_int32(0)
    c = lib().lto_clip_factor(S, max_norm, C.byref(nf))
    return float(c), bool(nf.value)


def step_scalars(hp: HParams) -> dict:
    s = _Scalars()
    h = hp.c()
    lib().lto_step_scalars(C.byref(h), C.byref(s))
    return {k: getattr(s, k) for k, _ in _Scalars._fields_}


def state_init(tensors, block: int) -> None:
    lib().lto_state_init(_carray(tensors), len(tensors), block)


def hybrid8_step(tensors, block: int, hp: HParams, S: float, brute: bool = False) -> int:
    """Run one step over `tensors` given the step's total squared gradient norm S. Returns the
    status word (bit 0: skipped because S is not finite)."""
    st = C.c_int32(0)
    h = hp.c()
    lib().lto_hybrid8_step(_carray(tensors), len(tensors), block, C.byref(h), S, C.byref(st), int(brute))
    return st.value


def step_fp32state(param, grad, m, v, hp: HParams, c: float) -> None:
    for a in (param, grad, m, v):
        assert a.dtype == np.float32 and a.flags.c_contiguous
    h = hp.c()
    p = lambda a: a.ctypes.data_as(C.c_void_p)  # noqa: E731
    lib().lto_step_fp32state(p(param), p(grad), p(m), p(v), param.size, C.byref(h), c)


def dequant(is_signed: bool, code: np.ndarray, absmax: np.ndarray, block: int) -> np.ndarray:
    out = np.empty(code.size, np.float32)
    p = lambda a: a.ctypes.data_as(C.c_void_p)  # noqa: E731
    lib().lto_dequant(int(is_signed), p(code), p(absmax), code.size, block, p(out))
    return out
