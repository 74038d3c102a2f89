"""Thin ctypes binding over libslidedp (same names as the C ABI in ``include/slidedp.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
Tensors are torch tensors used purely as device / pinned-host memory; their
``data_ptr()`` and the raw ``cudaStream_t`` are what crosses the boundary. There is no CPU
fallback: if the shared library is missing the import of this module fails.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libslidedp.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2609_34162_b200.build` "
        "(nvcc, sm_100a). libslidedp has no CPU fallback.")

_lib = ctypes.CDLL(LIB_PATH)

MAX_RANKS = 16
NORM_TILE = 16384
OK, ERR_INVALID_ARG, ERR_MISALIGNED, ERR_BUDGET, ERR_NOT_PINNED, ERR_CUDA, ERR_TIMEOUT, ERR_NO_NORM = (
    0, -1, -2, -3, -4, -5, -6, -7)
ERR_TOO_LARGE = -8
NOALLOC_MAX_ELEMS = 1 << 30
IPC_HANDLE_BYTES = 80


class _HParams(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
                ("eps", ctypes.c_double), ("weight_decay", ctypes.c_double),
                ("inv_R", ctypes.c_double), ("max_norm", ctypes.c_double),
                ("step", ctypes.c_int64)]


class _Stats(ctypes.Structure):
    _fields_ = [("norm", ctypes.c_double), ("clip_coef", ctypes.c_double),
                ("ms_total", ctypes.c_double), ("ms_norm", ctypes.c_double),
                ("ms_h2d", ctypes.c_double), ("ms_kernel", ctypes.c_double),
                ("ms_d2h", ctypes.c_double), ("gbs_h2d", ctypes.c_double),
                ("gbs_d2h", ctypes.c_double), ("chunks", ctypes.c_int64),
                ("nonfinite", ctypes.c_int32), ("reserved", ctypes.c_int32)]


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


_vp, _pp = ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p)
_lib.slidedp_create.restype = ctypes.c_int
_lib.slidedp_create.argtypes = [ctypes.POINTER(_vp), ctypes.c_int, ctypes.c_size_t]
_lib.slidedp_destroy.restype = ctypes.c_int
_lib.slidedp_destroy.argtypes = [_vp]
_lib.slidedp_strerror.restype = ctypes.c_char_p
_lib.slidedp_strerror.argtypes = [ctypes.c_int]
_lib.slidedp_last_cuda_error.restype = ctypes.c_int
_lib.slidedp_last_cuda_error.argtypes = [_vp]
_lib.slidedp_state_bytes.restype = ctypes.c_size_t
_lib.slidedp_state_bytes.argtypes = [ctypes.c_int64]
_lib.slidedp_grad_norm.restype = ctypes.c_int
_lib.slidedp_grad_norm.argtypes = [_vp, _pp, ctypes.c_int, ctypes.c_int64, ctypes.c_double,
                                   ctypes.c_int, _vp]
_lib.slidedp_grad_norm_finish.restype = ctypes.c_int
_lib.slidedp_grad_norm_finish.argtypes = [_vp, ctypes.c_double, ctypes.POINTER(ctypes.c_double),
                                          ctypes.POINTER(ctypes.c_double), _vp]
_lib.slidedp_grad_norm_tiles.restype = ctypes.c_int
_lib.slidedp_grad_norm_tiles.argtypes = [_vp, _pp, ctypes.c_int, ctypes.c_int64, ctypes.c_double, _vp, _vp]
_lib.slidedp_grad_norm_finish_from.restype = ctypes.c_int
_lib.slidedp_grad_norm_finish_from.argtypes = [_vp, _vp, ctypes.c_int64, ctypes.c_double,
                                               ctypes.POINTER(ctypes.c_double),
                                               ctypes.POINTER(ctypes.c_double), _vp]
_lib.slidedp_reduce_adamw_chunk.restype = ctypes.c_int
_lib.slidedp_reduce_adamw_chunk.argtypes = [_vp, _pp, ctypes.c_int, ctypes.c_int64, _vp, _vp, _vp,
                                            _vp, ctypes.POINTER(_HParams), _vp]
_lib.slidedp_stream_step.restype = ctypes.c_int
_lib.slidedp_stream_step.argtypes = [_vp, _pp, ctypes.c_int, ctypes.c_int64, _vp, _vp, _vp, _vp,
                                     ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                     ctypes.POINTER(_HParams), ctypes.POINTER(_Stats)]
_lib.slidedp_reduce_mean_bf16.restype = ctypes.c_int
_lib.slidedp_reduce_mean_bf16.argtypes = [_vp, _pp, ctypes.c_int, ctypes.c_int64, ctypes.c_double, _vp, _vp]
_lib.slidedp_stream_step_async.restype = ctypes.c_int
_lib.slidedp_stream_step_async.argtypes = [_vp, _pp, ctypes.c_int, ctypes.c_int64, _vp, _vp, _vp, _vp,
                                           ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                           ctypes.POINTER(_HParams)]
class _Layer(ctypes.Structure):
    _fields_ = [("grads_bf16", _pp), ("n", ctypes.c_int64), ("host_master", _vp), ("host_m", _vp),
                ("host_v", _vp), ("param_bf16_out", _vp)]


_lib.slidedp_stream_layers.restype = ctypes.c_int
_lib.slidedp_stream_layers.argtypes = [_vp, ctypes.POINTER(_Layer), ctypes.c_int, ctypes.c_int,
                                       ctypes.c_int64, ctypes.c_int, ctypes.POINTER(_HParams),
                                       ctypes.POINTER(_Stats)]
_lib.slidedp_stream_wait.restype = ctypes.c_int
_lib.slidedp_stream_wait.argtypes = [_vp]
_lib.slidedp_deliver_params.restype = ctypes.c_int
_lib.slidedp_deliver_params.argtypes = [_vp, _vp, ctypes.c_int64, _vp, ctypes.c_int64, ctypes.c_int,
                                        ctypes.POINTER(_Stats)]
_lib.slidedp_link_probe.restype = ctypes.c_int
_lib.slidedp_link_probe.argtypes = [_vp, _vp, _vp, _vp, _vp, ctypes.c_size_t, ctypes.c_size_t,
                                    ctypes.c_int, ctypes.POINTER(ctypes.c_double)]
_lib.slidedp_grad_norm_noalloc.restype = ctypes.c_int
_lib.slidedp_grad_norm_noalloc.argtypes = [_pp, ctypes.c_int, ctypes.c_int64, ctypes.c_double,
                                           ctypes.c_double, _vp, _vp]
_lib.slidedp_kernel_launches.restype = ctypes.c_int64
_lib.slidedp_kernel_launches.argtypes = [_vp]
_lib.slidedp_ipc_export.restype = ctypes.c_int
_lib.slidedp_ipc_export.argtypes = [_vp, _vp, ctypes.c_char_p]
_lib.slidedp_ipc_open.restype = ctypes.c_int
_lib.slidedp_ipc_open.argtypes = [_vp, ctypes.c_char_p, ctypes.POINTER(_vp)]
_lib.slidedp_ipc_close.restype = ctypes.c_int
_lib.slidedp_ipc_close.argtypes = [_vp, _vp]
_lib.slidedp_scatter_tile_sums.restype = ctypes.c_int
_lib.slidedp_scatter_tile_sums.argtypes = [_vp, _vp, ctypes.c_int64, _pp, ctypes.c_int, _vp]
_lib.slidedp_reduce_adamw_chunk_bcast.restype = ctypes.c_int
_lib.slidedp_reduce_adamw_chunk_bcast.argtypes = [_vp, _pp, ctypes.c_int, ctypes.c_int64, _vp, _vp, _vp,
                                                  _pp, ctypes.c_int, ctypes.POINTER(_HParams), _vp]
_lib.slidedp_hbm_mix_probe.restype = ctypes.c_int
_lib.slidedp_hbm_mix_probe.argtypes = [_vp, _pp, ctypes.c_int, ctypes.c_int64, _vp, _vp, _vp, _vp,
                                       ctypes.c_int, ctypes.POINTER(ctypes.c_double), _vp]
_lib.slidedp_set_wait_seconds.restype = ctypes.c_int
_lib.slidedp_set_wait_seconds.argtypes = [_vp, ctypes.c_double]
_lib.slidedp_test_fail_nth_call.restype = ctypes.c_int
_lib.slidedp_test_fail_nth_call.argtypes = [_vp, ctypes.c_int64]


class _Rates(ctypes.Structure):
    _fields_ = [("h2d_gbs", ctypes.c_double), ("d2h_gbs", ctypes.c_double),
                ("update_gparams_s", ctypes.c_double), ("norm_gbs", ctypes.c_double),
                ("per_copy_us", ctypes.c_double)]


_lib.slidedp_model_stream_step.restype = ctypes.c_int
_lib.slidedp_model_stream_step.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.c_int,
                                           ctypes.POINTER(_Rates), ctypes.POINTER(ctypes.c_double),
                                           ctypes.POINTER(ctypes.c_double)]


class SlideDPError(RuntimeError):
    def __init__(self, status: int, cuda_error: int = 0):
        self.status, self.cuda_error = status, cuda_error
        msg = _lib.slidedp_strerror(status).decode()
        if status == ERR_CUDA:
            msg += f" (cudaError_t {cuda_error})"
        super().__init__(f"libslidedp: {msg} [{status}]")


def slidedp_strerror(status: int) -> str:
    return _lib.slidedp_strerror(status).decode()


def slidedp_state_bytes(n: int) -> int:
    return int(_lib.slidedp_state_bytes(n))


def _ptr(x) -> int:
    """Raw address of a tensor's first element (or an int passed through, or None)."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _grad_array(grads):
    return (ctypes.c_void_p * len(grads))(*[_ptr(g) for g in grads])


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Context:
    """Owns a ``slidedp_ctx``. Methods carry the C entry points' names and argument order."""

    def __init__(self, device: int = 0, gpu_budget_bytes: int = 0):
        self._h = _vp()
        rc = _lib.slidedp_create(ctypes.byref(self._h), device, gpu_budget_bytes)
        if rc != OK:
            self._h = _vp()
            raise SlideDPError(rc)
        self.device = device

    def _check(self, rc: int):
        if rc != OK:
            raise SlideDPError(rc, _lib.slidedp_last_cuda_error(self._h))

    def slidedp_destroy(self):
        if self._h:
            rc = _lib.slidedp_destroy(self._h)
            self._h = _vp()
            if rc != OK:
                raise SlideDPError(rc)

    close = slidedp_destroy

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.slidedp_destroy()

    def __del__(self):
        try:
            if self._h:
                _lib.slidedp_destroy(self._h)
                self._h = _vp()
        except Exception:
            pass

    def slidedp_kernel_launches(self) -> int:
        return int(_lib.slidedp_kernel_launches(self._h))

    def slidedp_set_wait_seconds(self, seconds: float) -> None:
        self._check(_lib.slidedp_set_wait_seconds(self._h, seconds))

    def slidedp_test_fail_nth_call(self, nth: int) -> None:
        self._check(_lib.slidedp_test_fail_nth_call(self._h, nth))

    def slidedp_last_cuda_error(self) -> int:
        return int(_lib.slidedp_last_cuda_error(self._h))

    def slidedp_grad_norm(self, grads, n: int, inv_R: float, first_chunk: bool = True,
                          stream=None) -> None:
        self._check(_lib.slidedp_grad_norm(self._h, _grad_array(grads), len(grads), n, inv_R,
                                           int(first_chunk), _stream(stream)))

    def slidedp_grad_norm_finish(self, max_norm: float, fetch: bool = False, stream=None):
        """Returns (norm, coef) if ``fetch`` (synchronises), else None."""
        if fetch:
            norm, coef = ctypes.c_double(), ctypes.c_double()
            self._check(_lib.slidedp_grad_norm_finish(self._h, max_norm, ctypes.byref(norm),
                                                      ctypes.byref(coef), _stream(stream)))
            return norm.value, coef.value
        self._check(_lib.slidedp_grad_norm_finish(self._h, max_norm, None, None, _stream(stream)))
        return None

    def slidedp_grad_norm_tiles(self, grads, n: int, inv_R: float, tile_sums_out, stream=None) -> None:
        self._check(_lib.slidedp_grad_norm_tiles(self._h, _grad_array(grads), len(grads), n, inv_R,
                                                 _ptr(tile_sums_out), _stream(stream)))

    def slidedp_grad_norm_finish_from(self, tile_sums, count: int, max_norm: float,
                                      fetch: bool = False, stream=None):
        if fetch:
            norm, coef = ctypes.c_double(), ctypes.c_double()
            self._check(_lib.slidedp_grad_norm_finish_from(
                self._h, _ptr(tile_sums), count, max_norm, ctypes.byref(norm), ctypes.byref(coef),
                _stream(stream)))
            return norm.value, coef.value
        self._check(_lib.slidedp_grad_norm_finish_from(self._h, _ptr(tile_sums), count, max_norm,
                                                       None, None, _stream(stream)))
        return None

    def slidedp_reduce_adamw_chunk(self, grads, n: int, master, m, v, param_bf16_out,
                                   hp: HParams, stream=None) -> None:
        c = hp._c()
        self._check(_lib.slidedp_reduce_adamw_chunk(
            self._h, _grad_array(grads), len(grads), n, _ptr(master), _ptr(m), _ptr(v),
            _ptr(param_bf16_out), ctypes.byref(c), _stream(stream)))

    def slidedp_reduce_adamw_chunk_bcast(self, grads, n: int, master, m, v, param_bf16_outs,
                                         hp: HParams, stream=None) -> None:
        c = hp._c()
        self._check(_lib.slidedp_reduce_adamw_chunk_bcast(
            self._h, _grad_array(grads), len(grads), n, _ptr(master), _ptr(m), _ptr(v),
            _grad_array(param_bf16_outs), len(param_bf16_outs), ctypes.byref(c), _stream(stream)))

    def slidedp_scatter_tile_sums(self, tile_sums, count: int, dsts, stream=None) -> None:
        self._check(_lib.slidedp_scatter_tile_sums(self._h, _ptr(tile_sums), count,
                                                   _grad_array(dsts), len(dsts), _stream(stream)))

    def slidedp_ipc_export(self, dev_ptr) -> bytes:
        """The 80-byte handle of a device buffer (tensor or address), to send to a peer process."""
        buf = ctypes.create_string_buffer(IPC_HANDLE_BYTES)
        self._check(_lib.slidedp_ipc_export(self._h, _ptr(dev_ptr), buf))
        return buf.raw

    def slidedp_ipc_open(self, handle: bytes) -> int:
        """Maps a peer's handle; returns the device address valid in this process."""
        if len(handle) != IPC_HANDLE_BYTES:
            raise ValueError("not a slidedp_ipc_handle")
        out = _vp()
        self._check(_lib.slidedp_ipc_open(self._h, handle, ctypes.byref(out)))
        return int(out.value)

    def slidedp_ipc_close(self, dev_ptr: int) -> None:
        self._check(_lib.slidedp_ipc_close(self._h, dev_ptr))

    def slidedp_reduce_mean_bf16(self, grads, n: int, inv_R: float, out_bf16, stream=None) -> None:
        self._check(_lib.slidedp_reduce_mean_bf16(self._h, _grad_array(grads), len(grads), n, inv_R,
                                                  _ptr(out_bf16), _stream(stream)))

    def slidedp_stream_step(self, grads, n_total: int, host_master, host_m, host_v,
                            param_bf16_out, chunk_elems: int, nbuf: int, hp: HParams,
                            norm_ready: bool = False, want_stats: bool = True):
        c = hp._c()
        st = _Stats()
        self._check(_lib.slidedp_stream_step(
            self._h, _grad_array(grads), len(grads), n_total, _ptr(host_master), _ptr(host_m),
            _ptr(host_v), _ptr(param_bf16_out), chunk_elems, nbuf, int(norm_ready),
            ctypes.byref(c), ctypes.byref(st) if want_stats else None))
        if not want_stats:
            return None
        return {f: getattr(st, f) for f, _ in _Stats._fields_ if f != "reserved"}

    def slidedp_stream_step_async(self, grads, n_total: int, host_master, host_m, host_v,
                                  param_bf16_out, chunk_elems: int, nbuf: int, hp: HParams,
                                  norm_ready: bool = False) -> None:
        c = hp._c()
        self._check(_lib.slidedp_stream_step_async(
            self._h, _grad_array(grads), len(grads), n_total, _ptr(host_master), _ptr(host_m),
            _ptr(host_v), _ptr(param_bf16_out), chunk_elems, nbuf, int(norm_ready),
            ctypes.byref(c)))

    def slidedp_stream_layers(self, layers, chunk_elems: int, nbuf: int, hp: HParams,
                              want_stats: bool = True):
        """``layers``: sequence of (grads, n, host_master, host_m, host_v, param_bf16_out), every
        ``grads`` a list of the same R device buffers' worth of rank gradients."""
        R = len(layers[0][0]) if layers else 1
        keep = [_grad_array(L[0]) for L in layers]              # the pointer arrays must outlive the call
        arr = (_Layer * max(len(layers), 1))()
        for i, (L, g) in enumerate(zip(layers, keep)):
            if len(L[0]) != R:
                raise ValueError("every layer needs the same number of rank gradients")
            arr[i] = _Layer(ctypes.cast(g, _pp), L[1], _ptr(L[2]), _ptr(L[3]), _ptr(L[4]), _ptr(L[5]))
        c, st = hp._c(), _Stats()
        self._check(_lib.slidedp_stream_layers(self._h, arr, len(layers), R, chunk_elems, nbuf,
                                               ctypes.byref(c), ctypes.byref(st) if want_stats else None))
        if not want_stats:
            return None
        return {f: getattr(st, f) for f, _ in _Stats._fields_ if f != "reserved"}

    def slidedp_stream_wait(self) -> None:
        self._check(_lib.slidedp_stream_wait(self._h))

    def slidedp_deliver_params(self, host_master, n_total: int, param_bf16_out, chunk_elems: int,
                               nbuf: int, want_stats: bool = True):
        st = _Stats()
        self._check(_lib.slidedp_deliver_params(
            self._h, _ptr(host_master), n_total, _ptr(param_bf16_out), chunk_elems, nbuf,
            ctypes.byref(st) if want_stats else None))
        if not want_stats:
            return None
        return {f: getattr(st, f) for f in ("ms_total", "ms_h2d", "gbs_h2d", "chunks")}

    def slidedp_hbm_mix_probe(self, grads, n: int, master, m, v, scratch_bf16_out, reps: int = 5,
                              stream=None) -> float:
        """GB/s of the update kernel's loads and stores with no arithmetic (state unchanged)."""
        out = ctypes.c_double()
        self._check(_lib.slidedp_hbm_mix_probe(self._h, _grad_array(grads), len(grads), n, _ptr(master),
                                               _ptr(m), _ptr(v), _ptr(scratch_bf16_out), reps,
                                               ctypes.byref(out), _stream(stream)))
        return out.value

    def slidedp_link_probe(self, host_a, host_b, dev_a, dev_b, nbytes: int, copy_bytes: int,
                           reps: int = 3):
        out = (ctypes.c_double * 4)()
        self._check(_lib.slidedp_link_probe(self._h, _ptr(host_a), _ptr(host_b), _ptr(dev_a),
                                            _ptr(dev_b), nbytes, copy_bytes, reps, out))
        return {"h2d": out[0], "d2h": out[1], "h2d_bidir": out[2], "d2h_bidir": out[3]}


def slidedp_model_stream_step(n_total: int, R: int, chunk_elems: int, nbuf: int, h2d_gbs: float,
                              d2h_gbs: float, update_gparams_s: float, norm_gbs: float = 0.0,
                              per_copy_us: float = 0.0):
    """(lower_bound_ms, predicted_ms) of a host-resident step from measured rates."""
    r = _Rates(h2d_gbs, d2h_gbs, update_gparams_s, norm_gbs, per_copy_us)
    lo, pred = ctypes.c_double(), ctypes.c_double()
    rc = _lib.slidedp_model_stream_step(n_total, R, chunk_elems, nbuf, ctypes.byref(r),
                                        ctypes.byref(lo), ctypes.byref(pred))
    if rc != OK:
        raise SlideDPError(rc)
    return lo.value, pred.value


def shard_bounds(n: int, shards: int):
    """Contiguous shard bounds [(lo, hi), ...] of a flat space of n parameters over `shards`
    GPUs, every interior bound a multiple of NORM_TILE so that the shards' tile sums, gathered
    in shard order, are the tile sums of the unsharded step (argument arithmetic only)."""
    tiles = -(-n // NORM_TILE)
    bounds, lo_tile = [], 0
    for s in range(shards):
        hi_tile = lo_tile + tiles // shards + (1 if s < tiles % shards else 0)
        bounds.append((min(lo_tile * NORM_TILE, n), min(hi_tile * NORM_TILE, n)))
        lo_tile = hi_tile
    return bounds


def slidedp_create(device: int = 0, gpu_budget_bytes: int = 0) -> Context:
    return Context(device, gpu_budget_bytes)


def slidedp_grad_norm_noalloc(grads, n: int, inv_R: float, max_norm: float, out4, stream=None) -> None:
    """Global norm of one chunk for callers that must not allocate device memory (allocator
    callbacks, processes with a fully committed memory budget, plug-ins that only receive
    pointers): same result as ``slidedp_grad_norm`` + ``slidedp_grad_norm_finish``, but the
    tile sums live in a fixed 512 KiB array inside the library instead of a context.

    ``out4`` is a caller-owned device tensor of four float64 (sumsq, norm, coef, non-finite
    flag). ``n`` may not exceed ``NOALLOC_MAX_ELEMS``. Calls share the array, so only issue
    them ordered on one stream; make the first call on a device outside any stream capture.
    """
    rc = _lib.slidedp_grad_norm_noalloc(_grad_array(grads), len(grads), n, inv_R, max_norm,
                                        _ptr(out4), _stream(stream))
    if rc != OK:
        raise SlideDPError(rc)
