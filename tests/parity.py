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


def fp32_violations(got: np.ndarray, want: np.ndarray, block: int = 1 << 26):
    """(count outside tolerance, worst ratio |x-y| / allowed). Streams in blocks and uses torch's
    threaded CPU ops so that multi-billion-element states compare in seconds."""
    assert got.shape == want.shape and got.dtype == np.float32 and want.dtype == np.float32
    bad, worst = 0, 0.0
    for lo in range(0, got.size, block):
        x = torch.from_numpy(got[lo:lo + block]).double()
        y = torch.from_numpy(want[lo:lo + block]).double()
        allowed = torch.clamp(FP32_RTOL * y.abs(), min=FP32_ATOL)
        err = (x - y).abs()
        same_special = (torch.isnan(x) & torch.isnan(y)) | (torch.isinf(x) & (x == y))
        err = torch.where(same_special, torch.zeros_like(err), err)
        err = torch.where(torch.isnan(err), torch.full_like(err, float("inf")), err)
        ratio = err / allowed
        bad += int((ratio > 1.0).sum())
        if ratio.numel():
            worst = max(worst, float(ratio.max()))
    return bad, worst


def assert_fp32_close(name: str, got: np.ndarray, want: np.ndarray):
    bad, worst = fp32_violations(got, want)
    assert bad == 0, f"{name}: {bad} of {got.size} elements outside tolerance (worst {worst:.3g}x)"
    print(f"PARITY {name}: n={got.size} worst |x-y|/allowed = {worst:.3g}, "
          f"bitwise different = {float((got != want).mean()):.3g}")    # shown with pytest -s
    return worst


def _bf16_line(bits: torch.Tensor) -> torch.Tensor:
    """Monotone integer line over BF16 patterns (so that adjacent values differ by 1)."""
    i = bits.to(torch.int32) & 0xFFFF
    return torch.where((i & 0x8000) != 0, -(i & 0x7FFF), i)


def bf16_mismatch(got: np.ndarray, want: np.ndarray, block: int = 1 << 26):
    """(max ulp distance, fraction of elements that differ)."""
    assert got.shape == want.shape and got.dtype == np.uint16 and want.dtype == np.uint16
    if got.size == 0:
        return 0, 0.0
    worst, differ = 0, 0
    for lo in range(0, got.size, block):
        a = torch.from_numpy(got[lo:lo + block].view(np.int16))
        b = torch.from_numpy(want[lo:lo + block].view(np.int16))
        d = (_bf16_line(a) - _bf16_line(b)).abs()
        worst = max(worst, int(d.max()))
        differ += int((d != 0).sum())
    return worst, differ / got.size


def assert_bf16_close(name: str, got: np.ndarray, want: np.ndarray):
    ulp, frac = bf16_mismatch(got, want)
    assert ulp <= BF16_MAX_ULP, f"{name}: BF16 params up to {ulp} ulp apart"
    assert frac <= BF16_MAX_FRACTION, f"{name}: {frac:.3g} of BF16 params differ"
    print(f"PARITY {name}: n={got.size} max ulp = {ulp}, fraction differing = {frac:.3g}")
    return ulp, frac


def assert_norm_close(got: float, want: float):
    assert abs(got - want) <= NORM_RTOL * abs(want), f"norm {got!r} vs oracle {want!r}"
    print(f"PARITY norm: {got!r} vs oracle {want!r}, relative error {abs(got - want) / abs(want):.3g}")
