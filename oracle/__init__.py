"""ctypes front end of the plain-C oracle (TEST INFRASTRUCTURE ONLY).

The oracle is the slow CPU restatement of the SlideDP reduce + AdamW step that the
CUDA library is checked against. Only the tests, the smoke check and the benchmark's
CPU-baseline / reference arm may import this package; the product never does, and
this package never imports the product.

Arrays are numpy arrays on the host: BF16 data as ``uint16`` bit patterns, state as
``float32``. Everything is passed to C by pointer and updated in place.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "slidedp_oracle.c")
_HDR = os.path.join(_HERE, "slidedp_oracle.h")
_LIB = os.path.join(_HERE, "libslidedp_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction, OpenMP)."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


class _HParams(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
                ("eps", ctypes.c_double), ("weight_decay", ctypes.c_double),
                ("inv_R", ctypes.c_double), ("max_norm", ctypes.c_double),
                ("step", ctypes.c_int64)]


@dataclass
class HParams:
    lr: float = 1e-5
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    weight_decay: float = 0.1
    inv_R: float = 1.0
    max_norm: float = 0.0
    step: int = 1

    def _c(self) -> _HParams:
        return _HParams(self.lr, self.beta1, self.beta2, self.eps, self.weight_decay,
                        self.inv_R, self.max_norm, int(self.step))


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        pp = ctypes.POINTER(ctypes.c_void_p)
        L.oracle_state_bytes.restype = ctypes.c_size_t
        L.oracle_state_bytes.argtypes = [ctypes.c_int64, ctypes.POINTER(ctypes.c_int)]
        L.oracle_bf16_to_f32.restype = ctypes.c_float
        L.oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
        L.oracle_f32_to_bf16.restype = ctypes.c_uint16
        L.oracle_f32_to_bf16.argtypes = [ctypes.c_float]
        L.oracle_reduce_mean.restype = None
        L.oracle_reduce_mean.argtypes = [pp, ctypes.c_int, ctypes.c_int64, ctypes.c_double,
                                         ctypes.c_void_p]
        L.oracle_reduce_mean_bf16.restype = None
        L.oracle_reduce_mean_bf16.argtypes = [pp, ctypes.c_int, ctypes.c_int64, ctypes.c_double,
                                              ctypes.c_void_p]
        L.oracle_grad_sumsq.restype = ctypes.c_double
        L.oracle_grad_sumsq.argtypes = [pp, ctypes.c_int, ctypes.c_int64, ctypes.c_double,
                                        ctypes.c_int]
        L.oracle_clip_coef.restype = ctypes.c_double
        L.oracle_clip_coef.argtypes = [ctypes.c_double, ctypes.c_double,
                                       ctypes.POINTER(ctypes.c_double)]
        L.oracle_reduce_adamw_chunk.restype = ctypes.c_int
        L.oracle_reduce_adamw_chunk.argtypes = [pp, ctypes.c_int, ctypes.c_int64,
                                                ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                                ctypes.c_void_p, ctypes.POINTER(_HParams),
                                                ctypes.c_double, ctypes.c_int]
        L.oracle_step.restype = ctypes.c_int
        L.oracle_step.argtypes = [pp, ctypes.c_int, ctypes.c_int64, ctypes.c_void_p,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                  ctypes.c_int64, ctypes.POINTER(_HParams),
                                  ctypes.POINTER(ctypes.c_double),
                                  ctypes.POINTER(ctypes.c_double), ctypes.c_int]
        L.oracle_cast_master_to_bf16.restype = None
        L.oracle_cast_master_to_bf16.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
        L.oracle_max_threads.restype = ctypes.c_int
        L.oracle_max_threads.argtypes = []
        _lib = L
    return _lib


def _check(a: np.ndarray, dtype, n: int | None = None) -> np.ndarray:
    if not isinstance(a, np.ndarray) or a.dtype != dtype or not a.flags.c_contiguous:
        raise TypeError(f"expected a C-contiguous numpy array of {np.dtype(dtype)}")
    if n is not None and a.size != n:
        raise ValueError(f"expected {n} elements, got {a.size}")
    return a


def _grad_ptrs(grads):
    grads = [_check(g, np.uint16) for g in grads]
    n = grads[0].size
    for g in grads:
        _check(g, np.uint16, n)
    arr = (ctypes.c_void_p * len(grads))(*[g.ctypes.data for g in grads])
    return arr, len(grads), n


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def state_bytes(n: int):
    out = (ctypes.c_int * 5)()
    total = lib().oracle_state_bytes(n, out)
    return int(total), list(out)


def bf16_to_f32(bits: int) -> float:
    return float(lib().oracle_bf16_to_f32(bits))


def f32_to_bf16(x) -> int:
    return int(lib().oracle_f32_to_bf16(ctypes.c_float(x)))


def reduce_mean(grads, inv_R: float) -> np.ndarray:
    ptrs, R, n = _grad_ptrs(grads)
    out = np.empty(n, np.float32)
    lib().oracle_reduce_mean(ptrs, R, n, inv_R, out.ctypes.data)
    return out


def reduce_mean_bf16(grads, inv_R: float) -> np.ndarray:
    ptrs, R, n = _grad_ptrs(grads)
    out = np.empty(n, np.uint16)
    lib().oracle_reduce_mean_bf16(ptrs, R, n, inv_R, out.ctypes.data)
    return out


def grad_sumsq(grads, inv_R: float, nthreads: int = 1) -> float:
    ptrs, R, n = _grad_ptrs(grads)
    return float(lib().oracle_grad_sumsq(ptrs, R, n, inv_R, nthreads))


def clip_coef(sumsq: float, max_norm: float):
    norm = ctypes.c_double()
    c = lib().oracle_clip_coef(sumsq, max_norm, ctypes.byref(norm))
    return float(c), float(norm.value)


def cast_master_to_bf16(master: np.ndarray) -> np.ndarray:
    _check(master, np.float32)
    out = np.empty(master.size, np.uint16)
    lib().oracle_cast_master_to_bf16(master.ctypes.data, master.size, out.ctypes.data)
    return out


def reduce_adamw_chunk(grads, master, m, v, param_bf16, hp: HParams, clip: float = 1.0,
                       nthreads: int = 1) -> None:
    ptrs, R, n = _grad_ptrs(grads)
    _check(master, np.float32, n); _check(m, np.float32, n); _check(v, np.float32, n)
    _check(param_bf16, np.uint16, n)
    c = hp._c()
    rc = lib().oracle_reduce_adamw_chunk(ptrs, R, n, master.ctypes.data, m.ctypes.data,
                                         v.ctypes.data, param_bf16.ctypes.data,
                                         ctypes.byref(c), clip, nthreads)
    if rc:
        raise ValueError("oracle_reduce_adamw_chunk rejected its arguments")


def step(grads, master, m, v, param_bf16, hp: HParams, chunk_elems: int = 0,
         nthreads: int = 1):
    """One whole step; returns (norm, clip_coef)."""
    ptrs, R, n = _grad_ptrs(grads)
    _check(master, np.float32, n); _check(m, np.float32, n); _check(v, np.float32, n)
    _check(param_bf16, np.uint16, n)
    c = hp._c()
    norm, coef = ctypes.c_double(), ctypes.c_double()
    rc = lib().oracle_step(ptrs, R, n, master.ctypes.data, m.ctypes.data, v.ctypes.data,
                           param_bf16.ctypes.data, chunk_elems, ctypes.byref(c),
                           ctypes.byref(norm), ctypes.byref(coef), nthreads)
    if rc:
        raise ValueError("oracle_step rejected its arguments")
    return float(norm.value), float(coef.value)
