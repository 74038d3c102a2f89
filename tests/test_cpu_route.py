"""The paper's own data path as a baseline component (baseline/cpu_route): gradient D2H ->
multi-threaded vectorised CPU AdamW per chunk -> CPU cast with streaming stores -> BF16 H2D
(paper Sec. 3.2 "Gradient return", Sec. 3.3 "Overlap within a layer" and "Reduce -> D2H -> Adam").
It is checked against the oracle, like the CUDA path, but it is NOT the product and shares no code
with it.

The cast is exact (bit for bit against the oracle's cast, every code path). The update is FP32
arithmetic, as a vectorised CPU Adam is, so it agrees with the FP64 oracle only to FP32 rounding.
Tolerances used here, y = oracle, all per element:
  v       |x - y| <= 1e-6 |y|                   (three FP32 roundings, no cancellation)
  m       |x - y| <= 1e-6 (|beta1 m0| + |(1 - beta1) c g|)   (the two terms may cancel)
  master  |x - y| <= 1e-6 |y| + 1e-4 lr         (the step is lr * O(1); a wrong formula moves it
                                                 by lr * O(1), four orders above this bound)
  BF16    <= 1 ulp apart, <= 1e-3 of the elements differ.
"""
import os

import numpy as np
import pytest
import torch

import oracle
import parity
from baseline import cpu_route as cr
from paper_2609_34162_b200 import workloads as W

NTHREADS = max(1, min(16, len(os.sched_getaffinity(0))))
ISAS = ["avx512-bf16", "avx512f", "scalar"]


@pytest.fixture(params=ISAS)
def isa(request):
    if not cr.limit_isa(request.param):
        pytest.skip(f"this CPU cannot run the {request.param} path")
    yield request.param
    for name in ISAS:                       # back to the best the CPU has
        if cr.limit_isa(name):
            break


def specials():
    x = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 1e-40, -1e-45, 3.3895314e38, -3.4e38,
                  1.0, 1.00390625, 1.001953125, 1.005859375, 2.0 ** -126, 2.0 ** -133,
                  1.17e-38, 9.18e-41], np.float32)
    return x


def test_cast_is_bit_exact_on_every_code_path(isa):
    rng = np.random.default_rng(3)
    n = 200_003
    x = (rng.standard_normal(n) * 0.02).astype(np.float32)
    x[:specials().size] = specials()
    bits = rng.integers(0, 1 << 32, 4096, dtype=np.uint64).astype(np.uint32)     # any pattern
    x[1000:1000 + 4096] = bits.view(np.float32)
    want = oracle.cast_master_to_bf16(x)
    nan = np.isnan(x)
    for offset in (0, 1, 31, 32, 33):                     # destination alignment head and tail
        for threads in (1, 3, NTHREADS):
            out = np.full(n + 64, 0xABCD, np.uint16)
            cr.cast_bf16(x, n, out[offset:], threads)
            got = out[offset:offset + n]
            assert np.array_equal(got[~nan], want[~nan]), (isa, offset, threads)
            assert np.all((got[nan] & 0x7F80) == 0x7F80) and np.all((got[nan] & 0x7F) != 0)
            assert np.all(out[:offset] == 0xABCD) and np.all(out[offset + n:] == 0xABCD)
    cr.cast_bf16(x, 0, out, 2)                             # empty: nothing written


def fp32_route_case(n, R, seed, clip=0.37, step=7):
    g = torch.Generator().manual_seed(seed)
    grads = [(torch.randn(n, generator=g) * 1e-3).to(torch.bfloat16) for _ in range(R)]
    w = (torch.randn(n, generator=g) * 0.02).numpy()
    m = (torch.randn(n, generator=g) * 3e-4).numpy()
    v = (torch.randn(n, generator=g).square() * 1e-7).numpy()
    kw = dict(lr=1e-5, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1, step=step)
    return [parity.u16(x) for x in grads], w, m, v, kw, clip


def assert_fp32_route_close(tag, got, want, m0, gbar, kw, clip):
    gw, gm, gv, gp = got
    ow, om, ov, op = want
    d = lambda a, b: np.abs(a.astype(np.float64) - b.astype(np.float64))
    assert np.all(d(gv, ov) <= 1e-6 * np.abs(ov)), tag + "/v"
    scale = np.abs(kw["beta1"] * m0.astype(np.float64)) + np.abs((1 - kw["beta1"]) * clip * gbar.astype(np.float64))
    assert np.all(d(gm, om) <= 1e-6 * scale), tag + "/m"
    assert np.all(d(gw, ow) <= 1e-6 * np.abs(ow) + 1e-4 * kw["lr"]), tag + "/master"
    ulp, frac = parity.bf16_mismatch(gp, op)
    assert ulp <= 1 and frac <= 1e-3, (tag, ulp, frac)
    # the BF16 copy is exactly the cast of the route's OWN FP32 master
    assert np.array_equal(gp, oracle.cast_master_to_bf16(gw)), tag + "/cast"


@pytest.mark.parametrize("R", [1, 4])
@pytest.mark.parametrize("n", [1, 31, 32, 33, 100_003])
def test_fp32_update_matches_the_oracle_to_fp32_rounding(isa, n, R):
    grads, w, m, v, kw, clip = fp32_route_case(n, R, seed=100 * R + n % 97)
    ow, om, ov, op = w.copy(), m.copy(), v.copy(), np.zeros(n, np.uint16)
    oracle.reduce_adamw_chunk(grads, ow, om, ov, op, oracle.HParams(inv_R=1.0 / R, **kw), clip=clip)
    gbar = oracle.reduce_mean(grads, 1.0 / R)
    for threads in (1, NTHREADS):
        gw, gm, gv, gp = w.copy(), m.copy(), v.copy(), np.zeros(n, np.uint16)
        cr.adamw(grads, n, gw, gm, gv, gp, cr.HParams(inv_R=1.0 / R, clip_coef=clip, **kw), threads)
        assert_fp32_route_close(f"{isa} n={n} R={R} t={threads}", (gw, gm, gv, gp), (ow, om, ov, op),
                                m, gbar, kw, clip)
        if threads == 1:
            first = (gw, gm, gv, gp)
        else:                                               # threading never changes a bit
            assert all(np.array_equal(a, b) for a, b in zip(first, (gw, gm, gv, gp)))


def test_code_paths_agree_bit_for_bit_on_the_update():
    """The scalar, AVX-512 and AVX-512-BF16 paths do the same IEEE FP32 operations in the same
    order, so where a CPU has several they produce identical state."""
    n, R = 50_021, 3
    grads, w, m, v, kw, clip = fp32_route_case(n, R, seed=9)
    results = []
    for name in ISAS:
        if not cr.limit_isa(name):
            continue
        gw, gm, gv, gp = w.copy(), m.copy(), v.copy(), np.zeros(n, np.uint16)
        cr.adamw(grads, n, gw, gm, gv, gp, cr.HParams(inv_R=1.0 / R, clip_coef=clip, **kw), 3)
        results.append((gw, gm, gv, gp))
    for name in ISAS:
        if cr.limit_isa(name):
            break
    for r in results[1:]:
        assert all(np.array_equal(a, b) for a, b in zip(results[0], r))


def test_argument_errors():
    x = np.zeros(8, np.float32)
    with pytest.raises(RuntimeError):
        cr.cast_bf16(x, -1, np.zeros(8, np.uint16), 1)
    with pytest.raises(RuntimeError):
        cr.adamw([np.zeros(8, np.uint16)], 8, x, x.copy(), x.copy(), None, cr.HParams(step=0), 1)
    with pytest.raises(ValueError):
        cr.limit_isa("sse9")


@pytest.mark.gpu
@pytest.mark.parametrize("route", ["gpu_reduction", "cpu_reduction"])
def test_pipelined_step_on_a_scaled_layer(route):
    """The whole pipeline on a Qwen3-14B-shaped layer shrunk 16-fold: GPU reduction (one BF16
    gradient produced by libslidedp's slidedp_reduce_mean_bf16, G_l bytes D2H) and CPU reduction
    (all R gradients D2H, R G_l bytes, summed on the host), delivery to two receivers."""
    import paper_2609_34162_b200.slidedp as sd
    wl = W.scaled(W.CONFIGS["qwen3_14b_layer_host"], 16)
    n, R, t = wl.numel, wl.R, 3
    dg = [W.rank_gradient(wl, r, step=t, device="cuda") for r in range(R)]
    hg = [parity.u16(g) for g in dg]
    w0 = parity.f32(W.master_weights(wl, device="cuda")).copy()
    m0 = np.full(n, 1e-4, np.float32)
    v0 = np.full(n, 1e-7, np.float32)
    kw = dict(step=t, **wl.hparams)
    clip = 0.2
    ctx = sd.slidedp_create(0, 0)
    try:
        if route == "gpu_reduction":
            mean = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
            ctx.slidedp_reduce_mean_bf16(dg, n, 1.0 / R, mean)
            torch.cuda.synchronize()
            dev_grads, host_R = [mean], 1
            want_g = [oracle.reduce_mean_bf16(hg, 1.0 / R)]
            assert np.array_equal(parity.u16(mean), want_g[0])
            inv = 1.0
        else:
            dev_grads, host_R, want_g, inv = dg, R, hg, 1.0 / R
        stage = [torch.empty(n, dtype=torch.int16, pin_memory=True) for _ in range(host_R)]
        pstage = torch.empty(n, dtype=torch.int16, pin_memory=True)
        outs = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
        gw, gm, gv = w0.copy(), m0.copy(), v0.copy()
        torch.cuda.synchronize()
        st = cr.step([g.data_ptr() for g in dev_grads], n, stage, gw, gm, gv, pstage,
                     [o.data_ptr() for o in outs], 1 << 20, cr.HParams(inv_R=inv, clip_coef=clip, **kw),
                     NTHREADS)
        torch.cuda.synchronize()
    finally:
        ctx.slidedp_destroy()
    assert st["chunks"] == -(-n // (1 << 20))
    assert st["d2h_bytes"] == 2 * n * host_R and st["h2d_bytes"] == 2 * n * 2
    ow, om, ov, op = w0.copy(), m0.copy(), v0.copy(), np.zeros(n, np.uint16)
    oracle.reduce_adamw_chunk(want_g, ow, om, ov, op, oracle.HParams(inv_R=inv, **kw), clip=clip,
                              nthreads=NTHREADS)
    gbar = oracle.reduce_mean(want_g, inv)
    gp = pstage.numpy().view(np.uint16)
    assert_fp32_route_close(route, (gw, gm, gv, gp), (ow, om, ov, op), m0, gbar, kw, clip)
    for o in outs:                                          # every receiver got the same copy
        assert np.array_equal(parity.u16(o), gp)


@pytest.mark.gpu
def test_cpu_cast_delivery_is_bit_exact():
    """Delivery alone: the CPU casts chunk k+1 into pinned staging while DMA moves chunk k."""
    n = 5 * (1 << 20) + 4099
    g = torch.Generator().manual_seed(12)
    master = (torch.randn(n, generator=g) * 0.02).numpy()
    master[:specials().size] = specials()
    pstage = torch.empty(n, dtype=torch.int16, pin_memory=True)
    out = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()
    st = cr.deliver(master, n, pstage, out.data_ptr(), 1 << 20, NTHREADS)
    torch.cuda.synchronize()
    want = oracle.cast_master_to_bf16(master)
    got = parity.u16(out)
    nan = np.isnan(master)
    assert np.array_equal(got[~nan], want[~nan]) and st["chunks"] == 6 and st["h2d_bytes"] == 2 * n
