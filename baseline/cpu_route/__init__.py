"""ctypes front end of the paper-route CPU baseline (``cpu_route.h``): D2H of the gradient,
multi-threaded vectorised CPU AdamW per chunk as the copies land, CPU cast with streaming stores,
BF16 H2D. A timed BASELINE only: libslidedp never imports or links it, it never imports
libslidedp or the oracle, and it shares no code with either.

Host arrays are numpy arrays or torch host tensors (anything with a data pointer); device buffers
are passed as addresses.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cpu_route.cpp")
_HDR = os.path.join(_HERE, "cpu_route.h")
_LIB = os.path.join(_HERE, "libslidedp_cpuroute.so")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")
TIMEOUT = 100001


def build(force: bool = False) -> str:
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        cmd = ["g++", "-std=c++17", "-O3", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-Wall", "-Wextra",
               "-I", os.path.join(CUDA, "include"), "-o", tmp, _SRC,
               "-L", os.path.join(CUDA, "lib64"), "-lcudart",
               f"-Wl,-rpath,{os.path.join(CUDA, 'lib64')}"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


class _HParams(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
                ("eps", ctypes.c_double), ("weight_decay", ctypes.c_double),
                ("inv_R", ctypes.c_double), ("clip_coef", ctypes.c_double),
                ("step", ctypes.c_int64)]


class _Stats(ctypes.Structure):
    _fields_ = [("ms_total", ctypes.c_double), ("ms_wait_d2h", ctypes.c_double),
                ("ms_update", ctypes.c_double), ("ms_d2h_lane", ctypes.c_double),
                ("ms_h2d_lane", ctypes.c_double), ("d2h_bytes", ctypes.c_int64),
                ("h2d_bytes", ctypes.c_int64), ("chunks", ctypes.c_int64)]


@dataclass
class HParams:
    lr: float = 1e-5
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    weight_decay: float = 0.1
    inv_R: float = 1.0
    clip_coef: float = 1.0
    step: int = 1

    def _c(self) -> _HParams:
        return _HParams(self.lr, self.beta1, self.beta2, self.eps, self.weight_decay, self.inv_R,
                        self.clip_coef, int(self.step))


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, pp = ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p)
        L.cpuroute_isa.restype = ctypes.c_char_p
        L.cpuroute_max_threads.restype = ctypes.c_int
        L.cpuroute_limit_isa.restype = ctypes.c_int
        L.cpuroute_limit_isa.argtypes = [ctypes.c_char_p]
        L.cpuroute_cast_bf16.restype = ctypes.c_int
        L.cpuroute_cast_bf16.argtypes = [vp, ctypes.c_int64, vp, ctypes.c_int]
        L.cpuroute_adamw.restype = ctypes.c_int
        L.cpuroute_adamw.argtypes = [pp, ctypes.c_int, ctypes.c_int64, vp, vp, vp, vp,
                                     ctypes.POINTER(_HParams), ctypes.c_int]
        L.cpuroute_step.restype = ctypes.c_int
        L.cpuroute_step.argtypes = [pp, ctypes.c_int, ctypes.c_int64, pp, vp, vp, vp, vp, pp,
                                    ctypes.c_int, ctypes.c_int64, ctypes.POINTER(_HParams),
                                    ctypes.c_int, ctypes.POINTER(_Stats)]
        L.cpuroute_deliver.restype = ctypes.c_int
        L.cpuroute_deliver.argtypes = [vp, ctypes.c_int64, vp, vp, ctypes.c_int64, ctypes.c_int,
                                       ctypes.POINTER(_Stats)]
        _lib = L
    return _lib


def _addr(x) -> int:
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return x.ctypes.data                       # numpy


def _ptrs(xs):
    return (ctypes.c_void_p * len(xs))(*[_addr(x) for x in xs])


def _check(rc: int, what: str):
    if rc == TIMEOUT:
        raise TimeoutError(f"{what}: a bounded wait expired")
    if rc != 0:
        raise RuntimeError(f"{what} failed with status {rc}" + (" (cudaError_t)" if rc > 0 else ""))


def _stats(st: _Stats) -> dict:
    return {f: getattr(st, f) for f, _ in _Stats._fields_}


def isa() -> str:
    return lib().cpuroute_isa().decode()


def limit_isa(name: str) -> bool:
    """Switches to the named code path if this CPU can run it; returns whether it did."""
    rc = lib().cpuroute_limit_isa(name.encode())
    if rc == -1:
        raise ValueError(name)
    return rc == 0


def max_threads() -> int:
    return int(lib().cpuroute_max_threads())


def cast_bf16(master, n: int, out_bf16, nthreads: int = 1) -> None:
    _check(lib().cpuroute_cast_bf16(_addr(master), n, _addr(out_bf16), nthreads), "cpuroute_cast_bf16")


def adamw(grads, n: int, master, m, v, param_bf16, hp: HParams, nthreads: int = 1) -> None:
    c = hp._c()
    _check(lib().cpuroute_adamw(_ptrs(grads), len(grads), n, _addr(master), _addr(m), _addr(v),
                                _addr(param_bf16), ctypes.byref(c), nthreads), "cpuroute_adamw")


def step(dev_grads, n: int, host_grad_staging, master, m, v, host_param_staging, dev_params,
         chunk_elems: int, hp: HParams, nthreads: int) -> dict:
    c, st = hp._c(), _Stats()
    _check(lib().cpuroute_step(_ptrs(dev_grads), len(dev_grads), n, _ptrs(host_grad_staging),
                               _addr(master), _addr(m), _addr(v), _addr(host_param_staging),
                               _ptrs(dev_params), len(dev_params), chunk_elems, ctypes.byref(c),
                               nthreads, ctypes.byref(st)), "cpuroute_step")
    return _stats(st)


def deliver(master, n: int, host_param_staging, dev_params, chunk_elems: int, nthreads: int) -> dict:
    st = _Stats()
    _check(lib().cpuroute_deliver(_addr(master), n, _addr(host_param_staging), _addr(dev_params),
                                  chunk_elems, nthreads, ctypes.byref(st)), "cpuroute_deliver")
    return _stats(st)
