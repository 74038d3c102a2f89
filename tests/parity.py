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


def fp32_violations(got: np.ndarray, want: np.ndarray, block: int = 1 << 24):
    """(count outside tolerance, worst ratio |x-y| / allowed), streaming to bound memory."""
    assert got.shape == want.shape and got.dtype == np.float32 and want.dtype == np.float32
    bad, worst = 0, 0.0
    for lo in range(0, got.size, block):
        x = got[lo:lo + block].astype(np.float64)
        y = want[lo:lo + block].astype(np.float64)
        allowed = np.maximum(FP32_RTOL * np.abs(y), FP32_ATOL)
        err = np.abs(x - y)
        both_nan = np.isnan(x) & np.isnan(y)
        err[both_nan] = 0.0
        err[np.isnan(err)] = np.inf
        same_inf = np.isinf(x) & (x == y)
        err[same_inf] = 0.0
        ratio = err / allowed
        bad += int((ratio > 1.0).sum())
        if ratio.size:
            worst = max(worst, float(ratio.max()))
    return bad, worst


def assert_fp32_close(name: str, got: np.ndarray, want: np.ndarray):
    bad, worst = fp32_violations(got, want)
    assert bad == 0, f"{name}: {bad} of {got.size} elements outside tolerance (worst {worst:.3g}x)"
    return worst


def _bf16_line(bits: np.ndarray) -> np.ndarray:
    """Monotone integer line over BF16 patterns (so that adjacent values differ by 1)."""
    i = bits.astype(np.int32)
    return np.where(i & 0x8000, -(i & 0x7FFF), i)


def bf16_mismatch(got: np.ndarray, want: np.ndarray):
    """(max ulp distance, fraction of elements that differ)."""
    assert got.shape == want.shape and got.dtype == np.uint16 and want.dtype == np.uint16
    if got.size == 0:
        return 0, 0.0
    d = np.abs(_bf16_line(got) - _bf16_line(want))
    return int(d.max()), float((d != 0).sum()) / got.size


def assert_bf16_close(name: str, got: np.ndarray, want: np.ndarray):
    ulp, frac = bf16_mismatch(got, want)
    assert ulp <= BF16_MAX_ULP, f"{name}: BF16 params up to {ulp} ulp apart"
    assert frac <= BF16_MAX_FRACTION, f"{name}: {frac:.3g} of BF16 params differ"
    return ulp, frac


def assert_norm_close(got: float, want: float):
    assert abs(got - want) <= NORM_RTOL * abs(want), f"norm {got!r} vs oracle {want!r}"
