"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test compares the oracle with something other than itself: the paper's Table 1,
hand-worked IEEE cases, exact rational arithmetic, closed forms, torch's own
(independently written) AdamW / clip_grad_norm_ / BF16 cast, and brute force.
"""
import math
import os
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import HParams

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- helpers
def bf16_bits(x: np.ndarray) -> np.ndarray:
    """BF16 bit patterns of float32 values via torch's cast (independent of the oracle)."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_values(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def rand_bf16(rng, n, sigma=1e-3):
    return bf16_bits((rng.standard_normal(n) * sigma).astype(np.float32))


def fp32_round(q: Fraction) -> Fraction:
    """Round an exact rational to the nearest FP32 (ties to even), in exact arithmetic."""
    if q == 0:
        return Fraction(0)
    sign = -1 if q < 0 else 1
    a = abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    e = max(e, -126)                      # subnormals share the exponent of 2^-126
    ulp = Fraction(2) ** (e - 23)
    k, rem = divmod(a, ulp)
    if rem * 2 > ulp or (rem * 2 == ulp and k % 2 == 1):
        k += 1
    return sign * k * ulp


def fresh_state(rng, n, zero_moments=False):
    w = (rng.standard_normal(n) * 0.02).astype(np.float32)
    if zero_moments:
        return w, np.zeros(n, np.float32), np.zeros(n, np.float32)
    m = (rng.standard_normal(n) * 3e-4).astype(np.float32)
    v = (rng.standard_normal(n) ** 2 * 1e-7).astype(np.float32)
    return w, m, v


def ulp_diff(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    def line(x):
        i = x.view(np.int32).astype(np.int64)
        return np.where(i < 0, -(i & 0x7FFFFFFF), i)
    return np.abs(line(a) - line(b))


# ------------------------------------------------------------------ Table 1: 16N bytes
def test_state_accounting_matches_table1():
    rows = {}
    for ln in open(os.path.join(GOLDEN, "table1_state_bytes.txt")):
        if ln.strip() and not ln.startswith("#"):
            name, _, b = ln.split()
            rows[name] = int(b)
    total, parts = oracle.state_bytes(1)
    assert parts == [rows["compute_weights"], rows["gradients"], rows["master_weights"],
                     rows["adam_moments"] // 2, rows["adam_moments"] // 2]
    assert total == rows["total"] == 16
    for n in (0, 7, 192_946_176, 2_642_493_440):
        assert oracle.state_bytes(n)[0] == 16 * n


# ------------------------------------------------------------------- BF16 conversions
def test_bf16_round_to_nearest_even_exhaustive_neighbourhoods():
    b = np.arange(1 << 16, dtype=np.uint32)
    finite = ((b & 0x7FFF) < 0x7F80)
    for low in (0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF):
        x = ((b << 16) | low).astype(np.uint32).view(np.float32)
        got = np.array([oracle.f32_to_bf16(float(v)) for v in x[finite]], dtype=np.uint32)
        bb = b[finite]
        if low < 0x8000:
            want = bb
        elif low > 0x8000:
            want = bb + 1
        else:
            want = bb + (bb & 1)          # the tie goes to the even mantissa
        assert np.array_equal(got, want), hex(low)
        # torch's cast is a separately written implementation of the same rounding
        assert np.array_equal(got.astype(np.uint16), bf16_bits(x[finite])), hex(low)


def test_bf16_specials_and_widening():
    assert oracle.f32_to_bf16(float("inf")) == 0x7F80
    assert oracle.f32_to_bf16(float("-inf")) == 0xFF80
    nan = oracle.f32_to_bf16(float("nan"))
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x007F) != 0
    # the largest finite FP32 rounds up to infinity
    assert oracle.f32_to_bf16(float(np.finfo(np.float32).max)) == 0x7F80
    assert oracle.bf16_to_f32(0x3F80) == 1.0 and oracle.bf16_to_f32(0xC000) == -2.0
    assert oracle.bf16_to_f32(0x0001) == 2.0 ** -133       # smallest subnormal, exact
    for bits in (0x0000, 0x8000, 0x3FC0, 0x0080, 0x7F7F, 0x0001, 0x807F):
        assert oracle.f32_to_bf16(oracle.bf16_to_f32(bits)) == bits


# ----------------------------------------------------------------------- rank reduction
def test_rank_sum_hand_worked_cases():
    n_cases = 0
    for ln in open(os.path.join(GOLDEN, "rank_sum_cases.txt")):
        if not ln.strip() or ln.startswith("#"):
            continue
        R, vals, want = [s.strip() for s in ln.split("|")]
        R = int(R)
        vals = [float.fromhex(s) for s in vals.split()]
        assert len(vals) == R
        grads = [bf16_bits(np.array([x], np.float32)) for x in vals]
        for g, x in zip(grads, vals):
            assert bf16_values(g)[0] == x, "fixture value must be exact in BF16"
        got = oracle.reduce_mean(grads, 1.0 / R)
        assert got[0] == np.float32(float.fromhex(want)), ln
        n_cases += 1
    assert n_cases >= 8


@pytest.mark.parametrize("R", [1, 2, 3, 4, 5, 8, 16])
def test_rank_sum_against_exact_rational_arithmetic(R):
    rng = np.random.default_rng(100 + R)
    n = 96
    # exponent spread around the 24-bit significand: add order and every rounding matter
    scale = 2.0 ** rng.integers(-22, 1, size=(R, n))
    grads = [bf16_bits((rng.standard_normal(n) * scale[r]).astype(np.float32)) for r in range(R)]
    inv = fp32_round(Fraction(1.0 / R))
    got = oracle.reduce_mean(grads, 1.0 / R)
    vals = [bf16_values(g) for g in grads]
    n_order_sensitive = 0
    for i in range(n):
        s = Fraction(float(vals[0][i]))
        for r in range(1, R):
            s = fp32_round(s + Fraction(float(vals[r][i])))
        want = fp32_round(s * inv)
        assert Fraction(float(got[i])) == want
        s2 = Fraction(float(vals[R - 1][i]))
        for r in range(R - 2, -1, -1):
            s2 = fp32_round(s2 + Fraction(float(vals[r][i])))
        n_order_sensitive += (s2 != s)
    if R >= 3:
        assert n_order_sensitive > 0, "the case set must distinguish rank orders"


@pytest.mark.parametrize("R", [1, 2, 4, 8, 16])
def test_identical_rank_gradients_reduce_to_that_gradient(R):
    g = rand_bf16(np.random.default_rng(3), 4096)
    got = oracle.reduce_mean([g.copy() for _ in range(R)], 1.0 / R)
    assert np.array_equal(got, bf16_values(g))      # exact for a power-of-two R


@pytest.mark.parametrize("R", [3, 5, 6, 7])
def test_identical_rank_gradients_other_R_within_one_ulp(R):
    g = rand_bf16(np.random.default_rng(4), 4096)
    got = oracle.reduce_mean([g.copy() for _ in range(R)], 1.0 / R)
    assert ulp_diff(got, bf16_values(g)).max() <= 1  # (float)(1/R) is inexact


# ------------------------------------------------------------- Adam: closed forms
@pytest.mark.parametrize("wd", [0.0, 0.1])
def test_constant_gradient_closed_form(wd):
    """From m = v = 0 a constant gradient gives mhat = g and vhat = g^2 at every step,
    so each update is  w <- w - lr * ( g / (|g| + eps) + wd * w )."""
    rng = np.random.default_rng(5)
    n, T, R = 512, 12, 4
    # magnitudes from far below eps to far above it: pins where eps sits
    mag = 10.0 ** rng.uniform(-11, -1, n)
    g = bf16_bits((np.sign(rng.standard_normal(n)) * mag).astype(np.float32))
    g[:4] = bf16_bits(np.array([1e-8, -1e-8, 0.0, 1e-3], np.float32))
    gv = bf16_values(g).astype(np.float64)
    w, m, v = fresh_state(rng, n, zero_moments=True)
    p = np.zeros(n, np.uint16)
    hp = HParams(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=wd, inv_R=1.0 / R)
    w_closed = w.astype(np.float64)
    for t in range(1, T + 1):
        hp.step = t
        oracle.reduce_adamw_chunk([g] * R, w, m, v, p, hp)
        w_closed = w_closed - hp.lr * (gv / (np.abs(gv) + hp.eps) + wd * w_closed)
        # the oracle stores FP32 state each step: allow that rounding, nothing more
        assert np.allclose(w, w_closed, rtol=1.2e-7 * t, atol=hp.lr * 4e-7 * t)
        assert np.allclose(m, (1 - 0.9 ** t) * gv, rtol=3e-7 * t, atol=0)
        assert np.allclose(v, (1 - 0.95 ** t) * gv * gv, rtol=3e-7 * t, atol=1e-45)
    # g = eps exactly halves the step: u = g/(g+eps) = 1/2 (eps outside the root, after
    # bias correction); first step only, where no state rounding has accumulated
    w1, m1, v1 = fresh_state(rng, n, zero_moments=True)
    w0 = w1.astype(np.float64).copy()
    hp.step = 1
    oracle.reduce_adamw_chunk([g] * R, w1, m1, v1, p, hp)
    ge = gv[0]
    assert abs((w0[0] - w1[0]) - hp.lr * (ge / (ge + 1e-8) + wd * w0[0])) < 1e-10
    assert abs(ge / (ge + 1e-8) - 0.5) < 1e-2
    assert w1[2] == np.float32(w0[2] * (1 - hp.lr * wd))       # g = 0: decay only, no NaN
    assert not np.isnan(w1).any() and m1[2] == 0 and v1[2] == 0


def test_against_textbook_recurrences_in_50_digit_arithmetic():
    """Kingma & Ba Alg. 1 with Loshchilov & Hutter's decoupled decay, in Decimal."""
    getcontext().prec = 50
    rng = np.random.default_rng(6)
    n, R, T = 96, 2, 4
    hp = HParams(lr=1e-5, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1, inv_R=1.0 / R)
    w, m, v = fresh_state(rng, n, zero_moments=True)
    p = np.zeros(n, np.uint16)
    D = Decimal
    b1, b2, lr, eps, wd = (D(x) for x in (hp.beta1, hp.beta2, hp.lr, hp.eps, hp.weight_decay))
    worst, differ = 0, 0
    for t in range(1, T + 1):
        grads = [rand_bf16(rng, n) for _ in range(R)]
        gbar = (bf16_values(grads[0]) + bf16_values(grads[1])) * np.float32(0.5)  # exact for R=2
        w_in, m_in, v_in = w.copy(), m.copy(), v.copy()
        hp.step = t
        oracle.reduce_adamw_chunk(grads, w, m, v, p, hp)
        for i in range(n):
            g, th = D(float(gbar[i])), D(float(w_in[i]))
            mm = b1 * D(float(m_in[i])) + (1 - b1) * g
            vv = b2 * D(float(v_in[i])) + (1 - b2) * g * g
            mhat, vhat = mm / (1 - b1 ** t), vv / (1 - b2 ** t)
            th = th - lr * (mhat / (vhat.sqrt() + eps) + wd * th)
            want = np.array([float(th), float(mm), float(vv)], np.float64).astype(np.float32)
            got = np.array([w[i], m[i], v[i]], np.float32)
            d = ulp_diff(got, want)
            worst, differ = max(worst, int(d.max())), differ + int((d != 0).sum())
    # Double-then-round equals exact-then-round except at near-ties: with beta = 19/20 or
    # 9/10 the exact update (19 v + g^2)/20 often lies within a double ulp of an FP32
    # midpoint, where the double sum cannot tell the side. One FP32 ulp there, no more.
    assert worst <= 1 and differ <= 0.005 * 3 * n * T


@pytest.mark.parametrize("t,wd", [(1, 0.1), (11, 0.1), (11, 0.0), (1000, 0.01)])
def test_single_step_against_torch_adamw_in_float64(t, wd):
    """torch.optim.AdamW (decoupled decay, eps outside the root after bias correction)
    run in float64 from the same FP32 state, rounded once, must agree to one FP32 ulp."""
    rng = np.random.default_rng(7 + t)
    n, R = 4096, 4
    grads = [rand_bf16(rng, n) for _ in range(R)]
    w, m, v = fresh_state(rng, n, zero_moments=(t == 1))
    p = np.zeros(n, np.uint16)
    hp = HParams(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=wd, inv_R=1.0 / R, step=t)
    gbar = oracle.reduce_mean(grads, hp.inv_R)
    param = torch.nn.Parameter(torch.from_numpy(w.astype(np.float64)))
    opt = torch.optim.AdamW([param], lr=hp.lr, betas=(hp.beta1, hp.beta2), eps=hp.eps,
                            weight_decay=wd, foreach=False, fused=False)
    param.grad = torch.from_numpy(gbar.astype(np.float64))
    opt.state[param] = {"step": torch.tensor(float(t - 1)),
                        "exp_avg": torch.from_numpy(m.astype(np.float64)),
                        "exp_avg_sq": torch.from_numpy(v.astype(np.float64))}
    opt.step()
    oracle.reduce_adamw_chunk(grads, w, m, v, p, hp)
    st = opt.state[param]
    assert ulp_diff(w, param.detach().numpy().astype(np.float32)).max() <= 1
    assert ulp_diff(m, st["exp_avg"].numpy().astype(np.float32)).max() <= 1
    assert ulp_diff(v, st["exp_avg_sq"].numpy().astype(np.float32)).max() <= 1
    assert (w != param.detach().numpy().astype(np.float32)).mean() < 1e-3
    # the BF16 copy is the cast of the stored FP32 master
    assert np.array_equal(p, bf16_bits(w))


# ------------------------------------------------------------------------- clipping
def test_norm_against_exact_summation_and_torch_clip():
    rng = np.random.default_rng(8)
    n, R = 20000, 4
    grads = [rand_bf16(rng, n, 3e-2) for _ in range(R)]
    gbar = oracle.reduce_mean(grads, 0.25).astype(np.float64)
    S = oracle.grad_sumsq(grads, 0.25)
    exact = math.fsum((gbar * gbar).tolist())            # correctly rounded sum
    assert abs(S - exact) <= 1e-12 * exact
    c, norm = oracle.clip_coef(S, 1.0)
    assert abs(norm - math.sqrt(exact)) <= 1e-12 * norm and norm > 1.0
    prm = torch.nn.Parameter(torch.zeros(n, dtype=torch.float64))
    prm.grad = torch.from_numpy(gbar.copy())
    total = torch.nn.utils.clip_grad_norm_([prm], max_norm=1.0)   # max/(norm+1e-6), capped at 1
    assert abs(float(total) - norm) <= 1e-12 * norm
    assert np.allclose(prm.grad.numpy(), gbar * c, rtol=1e-13, atol=0)
    assert c == 1.0 / (norm + 1e-6)


def test_clip_inactive_is_bit_identical_and_scaling_identity():
    rng = np.random.default_rng(9)
    n, R = 5000, 2
    grads = [rand_bf16(rng, n, 1e-4) for _ in range(R)]
    S = oracle.grad_sumsq(grads, 0.5)
    c, norm = oracle.clip_coef(S, 1.0)
    assert norm < 1.0 - 1e-6 and c == 1.0
    assert oracle.clip_coef(S, 0.0)[0] == 1.0 and oracle.clip_coef(S, -1.0)[0] == 1.0
    a, b = fresh_state(rng, n), None
    b = tuple(x.copy() for x in a)
    pa, pb = np.zeros(n, np.uint16), np.zeros(n, np.uint16)
    hp_on = HParams(inv_R=0.5, max_norm=1.0, step=3)
    hp_off = HParams(inv_R=0.5, max_norm=0.0, step=3)
    oracle.step(grads, *a, pa, hp_on)
    oracle.step(grads, *b, pb, hp_off)
    assert all(np.array_equal(x, y) for x, y in zip(a, b)) and np.array_equal(pa, pb)
    # doubling every gradient (exact in binary) doubles the norm exactly
    g2 = [bf16_bits(bf16_values(g) * np.float32(2.0)) for g in grads]
    assert oracle.clip_coef(oracle.grad_sumsq(g2, 0.5), 1.0)[1] == 2.0 * norm
    assert math.isnan(oracle.clip_coef(float("nan"), 1.0)[0])
    assert oracle.clip_coef(float("inf"), 1.0)[0] == 0.0


def test_clipped_step_equals_unclipped_step_on_prescaled_gradients():
    """With a power-of-two coefficient, g*c is exact, so clipping must equal feeding the
    pre-multiplied gradients to the unclipped update."""
    rng = np.random.default_rng(10)
    n, R = 3000, 4
    grads = [rand_bf16(rng, n, 1e-3) for _ in range(R)]
    a = fresh_state(rng, n); b = tuple(x.copy() for x in a)
    pa, pb = np.zeros(n, np.uint16), np.zeros(n, np.uint16)
    hp = HParams(inv_R=0.25, step=11)
    oracle.reduce_adamw_chunk(grads, *a, pa, hp, clip=0.125)
    g8 = [bf16_bits(bf16_values(g) * np.float32(0.125)) for g in grads]
    oracle.reduce_adamw_chunk(g8, *b, pb, hp, clip=1.0)
    assert all(np.array_equal(x, y) for x, y in zip(a, b)) and np.array_equal(pa, pb)


def test_global_norm_covers_all_chunks_before_any_update():
    rng = np.random.default_rng(11)
    n, R = 10_000, 4
    grads = [rand_bf16(rng, n, 2e-2) for _ in range(R)]
    hp = HParams(inv_R=0.25, max_norm=1.0, step=2)
    a = fresh_state(rng, n); b = tuple(x.copy() for x in a)
    pa, pb = np.zeros(n, np.uint16), np.zeros(n, np.uint16)
    norm, c = oracle.step(grads, *a, pa, hp, chunk_elems=0)
    gbar = oracle.reduce_mean(grads, 0.25).astype(np.float64)
    assert abs(norm - float(np.linalg.norm(gbar))) <= 1e-12 * norm and c < 1.0
    # chunk by chunk with the GLOBAL coefficient gives the same state; a per-chunk
    # coefficient would not
    for lo in range(0, n, 1536):
        hi = min(n, lo + 1536)
        oracle.reduce_adamw_chunk([g[lo:hi] for g in grads], b[0][lo:hi], b[1][lo:hi],
                                  b[2][lo:hi], pb[lo:hi], hp, clip=c)
    assert all(np.array_equal(x, y) for x, y in zip(a, b)) and np.array_equal(pa, pb)


# ------------------------------------------------- chunking, threading, multi-step
@pytest.mark.parametrize("chunk", [1, 7, 1000, 4096, 10_000_000])
def test_chunk_size_and_threads_do_not_change_the_step(chunk):
    rng = np.random.default_rng(12)
    n, R = 9973, 3
    grads = [rand_bf16(rng, n, 5e-3) for _ in range(R)]
    hp = HParams(inv_R=1.0 / R, max_norm=0.1, step=7)
    a = fresh_state(rng, n); b = tuple(x.copy() for x in a)
    pa, pb = np.zeros(n, np.uint16), np.zeros(n, np.uint16)
    na = oracle.step(grads, *a, pa, hp, chunk_elems=0, nthreads=1)
    nb = oracle.step(grads, *b, pb, hp, chunk_elems=chunk, nthreads=1)
    assert na == nb
    assert all(np.array_equal(x, y) for x, y in zip(a, b)) and np.array_equal(pa, pb)
    c = tuple(x.copy() for x in fresh_state(np.random.default_rng(12), 1))  # unused warm-up
    del c
    # threads: the update is elementwise (bit-identical); only the norm's add order moves
    d = fresh_state(np.random.default_rng(99), n); e = tuple(x.copy() for x in d)
    pd, pe = np.zeros(n, np.uint16), np.zeros(n, np.uint16)
    hp2 = HParams(inv_R=1.0 / R, max_norm=0.0, step=7)
    oracle.step(grads, *d, pd, hp2, nthreads=1)
    oracle.step(grads, *e, pe, hp2, nthreads=4)
    assert all(np.array_equal(x, y) for x, y in zip(d, e)) and np.array_equal(pd, pe)
    s1, s4 = oracle.grad_sumsq(grads, 1.0 / R, 1), oracle.grad_sumsq(grads, 1.0 / R, 4)
    assert abs(s1 - s4) <= 1e-13 * s1


def test_update_uses_each_operand_where_it_belongs():
    """Brute force on a handful of elements, written straight from the definitions with
    Python floats (IEEE double): a transposed operand or a swapped beta shows here."""
    rng = np.random.default_rng(13)
    n, R, t = 16, 2, 5
    grads = [rand_bf16(rng, n, 1e-3) for _ in range(R)]
    w, m, v = fresh_state(rng, n)
    w0, m0, v0 = w.copy(), m.copy(), v.copy()
    p = np.zeros(n, np.uint16)
    hp = HParams(lr=2e-4, beta1=0.8, beta2=0.99, eps=1e-7, weight_decay=0.05, inv_R=0.5, step=t)
    c = 0.37
    oracle.reduce_adamw_chunk(grads, w, m, v, p, hp, clip=c)
    for i in range(n):
        gb = float(np.float32(np.float32(bf16_values(grads[0])[i] + bf16_values(grads[1])[i])
                              * np.float32(0.5)))
        g = gb * c
        m1 = 0.8 * float(m0[i]) + (1 - 0.8) * g
        v1 = 0.99 * float(v0[i]) + (1 - 0.99) * g * g
        u = (m1 / (1 - 0.8 ** t)) / (math.sqrt(v1 / (1 - 0.99 ** t)) + 1e-7)
        w1 = float(w0[i]) - 2e-4 * (u + 0.05 * float(w0[i]))
        assert m[i] == np.float32(m1) and v[i] == np.float32(v1) and w[i] == np.float32(w1)


def test_multi_step_equals_repeated_single_steps_and_empty_chunk():
    rng = np.random.default_rng(14)
    n, R = 2048, 4
    w, m, v = fresh_state(rng, n, zero_moments=True)
    p = np.zeros(n, np.uint16)
    snapshots = []
    for t in range(1, 4):
        grads = [rand_bf16(np.random.default_rng(1000 + 10 * t + r), n) for r in range(R)]
        oracle.step(grads, w, m, v, p, HParams(inv_R=0.25, max_norm=1.0, step=t), chunk_elems=500)
        snapshots.append((w.copy(), m.copy(), v.copy(), p.copy()))
    # resume from the stored state of step 2: same step 3
    w2, m2, v2, _ = (x.copy() for x in snapshots[1])
    p2 = np.zeros(n, np.uint16)
    grads = [rand_bf16(np.random.default_rng(1000 + 30 + r), n) for r in range(R)]
    oracle.step(grads, w2, m2, v2, p2, HParams(inv_R=0.25, max_norm=1.0, step=3))
    assert all(np.array_equal(x, y) for x, y in zip((w2, m2, v2, p2), snapshots[2]))
    z = np.zeros(0, np.float32)
    assert oracle.step([np.zeros(0, np.uint16)] * 2, z, z.copy(), z.copy(),
                       np.zeros(0, np.uint16), HParams(inv_R=0.5, max_norm=1.0)) == (0.0, 1.0)


# -------------------------------------------------------------- parameter delivery cast
def test_delivery_cast_matches_torch_cast_and_keeps_specials():
    rng = np.random.default_rng(15)
    x = (rng.standard_normal(200_000) * 0.02).astype(np.float32)
    x[:8] = [0.0, -0.0, np.inf, -np.inf, 1.00390625, 1.01171875, 1e-40, -3.4e38]
    #        ties: 1 + 2^-8 -> 1.0 (even), 1 + 3*2^-8 -> 1 + 2^-6 (even); subnormal; near max
    got = oracle.cast_master_to_bf16(x)
    assert np.array_equal(got, bf16_bits(x))
    assert got[4] == 0x3F80 and got[5] == 0x3F82 and got[2] == 0x7F80 and got[3] == 0xFF80
    assert got[1] == 0x8000 and got[7] == 0xFF80            # -3.4e38 rounds to -inf in BF16
    nan = oracle.cast_master_to_bf16(np.array([np.nan], np.float32))[0]
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x7F) != 0
    assert oracle.cast_master_to_bf16(np.zeros(0, np.float32)).size == 0


# ------------------------------------------------ rank reduction returned as one BF16 gradient
@pytest.mark.parametrize("R", [1, 2, 3, 8])
def test_reduced_bf16_gradient_is_the_cast_of_the_fp32_mean(R):
    rng = np.random.default_rng(16 + R)
    n = 5000
    grads = [rand_bf16(rng, n, 2e-3) for _ in range(R)]
    got = oracle.reduce_mean_bf16(grads, 1.0 / R)
    assert np.array_equal(got, bf16_bits(oracle.reduce_mean(grads, 1.0 / R)))   # torch's cast
    if R in (1, 2, 8):       # identical ranks and a power-of-two R: the gradient itself comes back
        same = oracle.reduce_mean_bf16([grads[0]] * R, 1.0 / R)
        assert np.array_equal(same, grads[0])
    # hand case: (1 + 2^-7) averaged with 1 is 1 + 2^-8, a BF16 tie that rounds to the even 1.0
    a = bf16_bits(np.array([1.0078125], np.float32)); b = bf16_bits(np.array([1.0], np.float32))
    assert oracle.reduce_mean_bf16([a, b], 0.5)[0] == 0x3F80


# ------------------------------------------------------------ invariants of Adam and of clipping
def test_adam_is_invariant_to_the_gradient_scale_when_eps_is_zero():
    """From zero moments with eps = 0, multiplying every gradient by a power of two scales m by
    it and v by its square exactly, so mhat / sqrt(vhat), and with it the master, must come out
    bit-identical at every step (Kingma & Ba Sec. 2.1: the step is invariant to gradient scale)."""
    rng = np.random.default_rng(17)
    n, R, T = 3000, 1, 5            # one rank: the mean cannot cancel to zero (0/0 with eps = 0)
    a = fresh_state(rng, n, zero_moments=True); b = tuple(x.copy() for x in a)
    pa, pb = np.zeros(n, np.uint16), np.zeros(n, np.uint16)
    for t in range(1, T + 1):
        grads = [rand_bf16(rng, n, 1e-3) for _ in range(R)]
        scaled = [bf16_bits(bf16_values(g) * np.float32(64.0)) for g in grads]
        hp = HParams(lr=1e-4, beta1=0.9, beta2=0.95, eps=0.0, weight_decay=0.1, inv_R=1.0, step=t)
        # gradients that are exactly zero would give 0/0 with eps = 0: nudge them
        for g, s in zip(grads, scaled):
            z = (g & 0x7FFF) == 0
            g[z] = 0x3A80; s[z] = bf16_bits(bf16_values(g[z]) * np.float32(64.0))
        oracle.reduce_adamw_chunk(grads, *a, pa, hp)
        oracle.reduce_adamw_chunk(scaled, *b, pb, hp)
        assert np.array_equal(a[0], b[0]) and np.array_equal(pa, pb)
        assert np.array_equal(b[1], a[1] * np.float32(64.0))
        assert np.array_equal(b[2], a[2] * np.float32(4096.0))


def test_active_clipping_cancels_a_common_gradient_scale():
    """While the norm exceeds max_norm the clipped gradient is g * max_norm / (norm + 1e-6):
    doubling every gradient doubles the norm exactly, so the clipped gradient changes only
    through the 1e-6 in the denominator."""
    rng = np.random.default_rng(18)
    n, R = 8000, 4
    grads = [rand_bf16(rng, n, 5e-2) for _ in range(R)]
    doubled = [bf16_bits(bf16_values(g) * np.float32(2.0)) for g in grads]
    a = fresh_state(rng, n); b = tuple(x.copy() for x in a)
    pa, pb = np.zeros(n, np.uint16), np.zeros(n, np.uint16)
    hp = HParams(inv_R=0.25, max_norm=1.0, step=4)
    na, ca = oracle.step(grads, *a, pa, hp)
    nb, cb = oracle.step(doubled, *b, pb, hp)
    assert na > 1.0 and nb == 2.0 * na
    assert abs(2.0 * cb / ca - 1.0) < 1e-6            # 2 c' = c (1 + O(1e-6 / norm))
    for x, y in zip(a, b):      # equal up to that 1e-6 (absolute scale: m can cancel to near 0)
        assert np.allclose(x, y, rtol=2e-6, atol=2e-6 * float(np.abs(x).max()))
    assert not all(np.array_equal(x, y) for x, y in zip(a, b))     # and the 1e-6 is really there


@pytest.mark.parametrize("R", [3, 4, 8])
def test_permuting_the_ranks_moves_the_fp32_sum_by_rounding_only(R):
    rng = np.random.default_rng(19 + R)
    n = 4096
    grads = [rand_bf16(rng, n, 1e-3 * 2.0 ** (-9 * (r % 3))) for r in range(R)]  # spread exponents
    base = oracle.reduce_mean(grads, 1.0 / R)
    perm = oracle.reduce_mean(grads[::-1], 1.0 / R)
    exact = sum(bf16_values(g).astype(np.float64) for g in grads) / R
    mag = sum(np.abs(bf16_values(g).astype(np.float64)) for g in grads) / R
    assert np.all(np.abs(base.astype(np.float64) - perm) <= 2 * R * 6e-8 * mag)    # rounding only
    assert np.all(np.abs(base - exact) <= R * 6e-8 * mag + 1e-45)       # ... around the exact mean
