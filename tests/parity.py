"""Comparators and small plumbing shared by the parity tests (no method arithmetic here).

Tolerances (from the benchmark definition):
  FP32 master / m / v : |x - y| <= max(1e-6 * |y|, 1e-12) for EVERY element, y = oracle;
  BF16 parameters     : at most 1 BF16 ulp apart everywhere, and at most 1e-4 of the
                        elements differ at all;
  global norm         : |a - b| <= 1e-6 * b.
"""
from __future__ import annotations

import numpy as np
import torch

FP32_RTOL, FP32_ATOL = 1e-6, 1e-12
BF16_MAX_ULP, BF16_MAX_FRACTION = 1, 1e-4
NORM_RTOL = 1e-6


def u16(t: torch.Tensor) -> np.ndarray:
    """BF16 tensor (any device) -> host uint16 bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().numpy()


def _compare_device() -> str:
    """Where the comparators do their arithmetic: on the GPU when there is one (a 2.6 G-element
    state compares in seconds there), else with torch's threaded CPU ops. The values compared
    are the same either way; only this bookkeeping moves."""
    return "cuda" if torch.cuda.is_available() else "cpu"


def _blocks(a, lo: int, hi: int, dev: str) -> torch.Tensor:
    """Elements [lo, hi) of a numpy array or (host) torch tensor, as a tensor on `dev`."""
    if isinstance(a, np.ndarray):
        a = a[lo:hi]
        t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a)
    else:
        t = a[lo:hi]
    return t.to(dev)


def fp32_violations(got, want, block: int = 1 << 26):
    """(count outside tolerance, worst ratio |x-y| / allowed). `got` / `want`: float32 numpy
    arrays or host tensors (pinned ones copy fastest)."""
    return _fp32_compare(got, want, block)[:2]


def _fp32_compare(got, want, block: int = 1 << 26):
    """(count outside tolerance, worst ratio, count of bitwise different elements). Streams in
    blocks so that multi-billion-element states compare in seconds."""
    assert tuple(got.shape) == tuple(want.shape)
    n, dev = int(np.prod(got.shape)), _compare_device()
    bad, worst, bitdiff = 0, 0.0, 0
    for lo in range(0, n, block):
        x = _blocks(got, lo, lo + block, dev)
        y = _blocks(want, lo, lo + block, dev)
        assert x.dtype == torch.float32 and y.dtype == torch.float32
        bitdiff += int((x.view(torch.int32) != y.view(torch.int32)).sum())
        x, y = x.double(), y.double()
        allowed = torch.clamp(FP32_RTOL * y.abs(), min=FP32_ATOL)
        err = (x - y).abs()
        same_special = (torch.isnan(x) & torch.isnan(y)) | (torch.isinf(x) & (x == y))
        err = torch.where(same_special, torch.zeros_like(err), err)
        err = torch.where(torch.isnan(err), torch.full_like(err, float("inf")), err)
        ratio = err / allowed
        bad += int((ratio > 1.0).sum())
        if ratio.numel():
            worst = max(worst, float(ratio.max()))
    return bad, worst, bitdiff


def count_different(a, b, block: int = 1 << 26) -> int:
    """Number of positions where two equally typed arrays / host tensors differ bitwise-as-values
    (used for "bit-identical" checks between two runs of the CUDA path and for reporting)."""
    assert tuple(a.shape) == tuple(b.shape)
    n, dev, diff = int(np.prod(a.shape)), _compare_device(), 0
    for lo in range(0, n, block):
        x, y = _blocks(a, lo, lo + block, dev), _blocks(b, lo, lo + block, dev)
        if x.dtype in (torch.float32, torch.bfloat16):          # compare the bit patterns
            x = x.view(torch.int32 if x.dtype == torch.float32 else torch.int16)
            y = y.view(x.dtype)
        diff += int((x != y).sum())
    return diff


def assert_fp32_close(name: str, got, want):
    bad, worst, bitdiff = _fp32_compare(got, want)
    n = int(np.prod(got.shape))
    assert bad == 0, f"{name}: {bad} of {n} elements outside tolerance (worst {worst:.3g}x)"
    print(f"PARITY {name}: n={n} worst |x-y|/allowed = {worst:.3g}, "
          f"bitwise different = {bitdiff / max(n, 1):.3g}")             # shown with pytest -s
    return worst


def _bf16_line(bits: torch.Tensor) -> torch.Tensor:
    """Monotone integer line over BF16 patterns (so that adjacent values differ by 1)."""
    i = bits.to(torch.int32) & 0xFFFF
    return torch.where((i & 0x8000) != 0, -(i & 0x7FFF), i)


def _bits16(a, lo: int, hi: int, dev: str) -> torch.Tensor:
    """BF16 bit patterns [lo, hi) as int16 on `dev`, from a uint16 numpy array, an int16 tensor
    or a bfloat16 tensor (host or device)."""
    if isinstance(a, np.ndarray):
        assert a.dtype == np.uint16
        return torch.from_numpy(a[lo:hi].view(np.int16)).to(dev)
    t = a[lo:hi]
    return (t.view(torch.int16) if t.dtype == torch.bfloat16 else t).to(dev)


def bf16_mismatch(got, want, block: int = 1 << 26):
    """(max ulp distance, fraction of elements that differ)."""
    assert tuple(got.shape) == tuple(want.shape)
    n, dev = int(np.prod(got.shape)), _compare_device()
    if n == 0:
        return 0, 0.0
    worst, differ = 0, 0
    for lo in range(0, n, block):
        a, b = _bits16(got, lo, lo + block, dev), _bits16(want, lo, lo + block, dev)
        d = (_bf16_line(a) - _bf16_line(b)).abs()
        worst = max(worst, int(d.max()))
        differ += int((d != 0).sum())
    return worst, differ / n


def assert_bf16_close(name: str, got, want):
    ulp, frac = bf16_mismatch(got, want)
    assert ulp <= BF16_MAX_ULP, f"{name}: BF16 params up to {ulp} ulp apart"
    assert frac <= BF16_MAX_FRACTION, f"{name}: {frac:.3g} of BF16 params differ"
    print(f"PARITY {name}: n={int(np.prod(got.shape))} max ulp = {ulp}, fraction differing = {frac:.3g}")
    return ulp, frac


def assert_norm_close(got: float, want: float):
    assert abs(got - want) <= NORM_RTOL * abs(want), f"norm {got!r} vs oracle {want!r}"
    print(f"PARITY norm: {got!r} vs oracle {want!r}, relative error {abs(got - want) / abs(want):.3g}")


def pinned_f32(n: int, src=None) -> torch.Tensor:
    """A page-locked float32 host tensor of n elements, optionally filled from a numpy array or
    a (host or device) tensor."""
    t = torch.empty(n, dtype=torch.float32, pin_memory=True)
    if src is not None:
        t.copy_(torch.from_numpy(src) if isinstance(src, np.ndarray) else src)
        if torch.cuda.is_available():
            torch.cuda.synchronize()
    return t


class GradStage:
    """Moves BF16 rank gradients from the device to the host for the oracle through reusable
    page-locked buffers, on a side stream: `prefetch(slot, grads)` starts the copies and returns,
    `take(slot)` waits for them and returns uint16 numpy views. With two slots the copy of the
    next layer runs while the oracle (a C call that releases the interpreter lock) works on the
    current one. Plumbing only: no arithmetic."""

    def __init__(self, R: int, n: int, slots: int = 2):
        self.bufs = [[torch.empty(n, dtype=torch.bfloat16, pin_memory=True) for _ in range(R)]
                     for _ in range(slots)]
        self.stream = torch.cuda.Stream()
        self.done = [torch.cuda.Event() for _ in range(slots)]
        self.count = [0] * slots

    def prefetch(self, slot: int, grads) -> None:
        self.stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(self.stream):
            for dst, src in zip(self.bufs[slot], grads):
                dst[:src.numel()].copy_(src, non_blocking=True)
            self.done[slot].record(self.stream)
        self.count[slot] = len(grads), grads[0].numel()

    def take(self, slot: int):
        self.done[slot].synchronize()
        R, n = self.count[slot]
        return [b[:n].view(torch.int16).numpy().view(np.uint16) for b in self.bufs[slot][:R]]

    def fetch(self, grads):
        """Synchronous convenience: one set of gradients through slot 0."""
        self.prefetch(0, grads)
        return self.take(0)
