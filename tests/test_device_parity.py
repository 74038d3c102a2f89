"""GPU parity, device-resident mode: libslidedp (through its C ABI) against the CPU oracle,
element by element, on the same seeded inputs."""
import os

import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2609_34162_b200 import workloads as W

pytestmark = pytest.mark.gpu

NTHREADS = max(1, min(64, len(os.sched_getaffinity(0))))


@pytest.fixture(scope="module")
def sd():
    import paper_2609_34162_b200.slidedp as sd
    return sd


@pytest.fixture()
def ctx(sd):
    c = sd.slidedp_create(0, 0)
    yield c
    c.slidedp_destroy()


def hp_pair(sd, **kw):
    return sd.HParams(**kw), oracle.HParams(**kw)


def random_case(n, R, seed, zero_moments=False, sigma=1e-3):
    g = torch.Generator().manual_seed(seed)
    grads = [(torch.randn(n, generator=g) * sigma).to(torch.bfloat16) for _ in range(R)]
    w = torch.randn(n, generator=g) * 0.02
    if zero_moments:
        m, v = torch.zeros(n), torch.zeros(n)
    else:
        m = torch.randn(n, generator=g) * 3e-4
        v = torch.randn(n, generator=g).square() * 1e-7
    return grads, w, m, v


def run_both(ctx, sd, grads, w, m, v, hp_kw, clip, chunk=None):
    """One step on the GPU (C ABI) and in the oracle; returns both results on the host."""
    n, R = w.numel(), len(grads)
    hp_g, hp_o = hp_pair(sd, inv_R=1.0 / R, max_norm=clip, **hp_kw)
    dg = [g.cuda() for g in grads]
    dw, dm, dv = w.cuda(), m.cuda(), v.cuda()
    dp = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    norm_g = None
    if clip > 0:
        ctx.slidedp_grad_norm(dg, n, hp_g.inv_R, True)
        norm_g, coef_g = ctx.slidedp_grad_norm_finish(clip, fetch=True)
    if chunk is None:
        ctx.slidedp_reduce_adamw_chunk(dg, n, dw, dm, dv, dp, hp_g)
    else:
        for lo in range(0, n, chunk):
            k = min(chunk, n - lo)
            ctx.slidedp_reduce_adamw_chunk([g[lo:] for g in dg], k, dw[lo:], dm[lo:], dv[lo:],
                                           dp[lo:], hp_g)
    torch.cuda.synchronize()
    ow, om, ov = parity.f32(w).copy(), parity.f32(m).copy(), parity.f32(v).copy()
    op = np.zeros(n, np.uint16)
    norm_o, coef_o = oracle.step([parity.u16(g) for g in grads], ow, om, ov, op, hp_o,
                                 nthreads=NTHREADS)
    return (parity.f32(dw), parity.f32(dm), parity.f32(dv), parity.u16(dp), norm_g), \
           (ow, om, ov, op, norm_o)


def assert_parity(tag, got, want, clip):
    for name, a, b in zip(("master", "m", "v"), got[:3], want[:3]):
        parity.assert_fp32_close(f"{tag}/{name}", a, b)
    parity.assert_bf16_close(f"{tag}/param_bf16", got[3], want[3])
    if clip > 0:
        parity.assert_norm_close(got[4], want[4])


ADAM = dict(lr=1e-5, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)


@pytest.mark.parametrize("R", [1, 2, 3, 4, 5, 8, 16])
@pytest.mark.parametrize("n", [1, 7, 8, 9, 1023, 2048 * 3 + 5, (1 << 20) + 3])
def test_odd_sizes_all_rank_counts(ctx, sd, n, R):
    grads, w, m, v = random_case(n, R, seed=1000 * R + n % 997)
    for clip, step in ((0.0, 1), (0.05, 11)):
        got, want = run_both(ctx, sd, grads, w, m, v, dict(ADAM, step=step), clip)
        assert_parity(f"n={n} R={R} clip={clip}", got, want, clip)


@pytest.mark.parametrize("R", list(range(1, 17)))
def test_every_rank_count_has_its_own_kernel(ctx, sd, R):
    """R = 1..16 each run a kernel with the rank loop unrolled; wide exponent spread between
    ranks so that the left-to-right order of the FP32 adds shows in the result."""
    n = (1 << 16) + 5
    g = torch.Generator().manual_seed(4000 + R)
    scale = 2.0 ** torch.randint(-12, 1, (R, n), generator=g).float()
    grads = [(torch.randn(n, generator=g) * 1e-2 * scale[r]).to(torch.bfloat16) for r in range(R)]
    _, w, m, v = random_case(n, 1, seed=R)
    got, want = run_both(ctx, sd, grads, w, m, v, dict(ADAM, step=4), 0.3)
    assert_parity(f"R={R}", got, want, 0.3)


def test_empty_chunk_is_a_no_op(ctx, sd):
    hp_g, _ = hp_pair(sd, inv_R=0.5, step=1, **ADAM)
    g = [torch.zeros(8, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    w = torch.ones(8, device="cuda")
    p = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    before = ctx.slidedp_kernel_launches()
    ctx.slidedp_reduce_adamw_chunk(g, 0, w, w.clone(), w.clone(), p, hp_g)
    ctx.slidedp_grad_norm(g, 0, 0.5, True)
    norm, coef = ctx.slidedp_grad_norm_finish(1.0, fetch=True)
    assert (norm, coef) == (0.0, 1.0) and torch.all(w == 1.0)
    assert ctx.slidedp_kernel_launches() == before + 1          # only the finish kernel ran


def test_config1_tiny_chunk_first_step(ctx, sd):
    """One flat chunk of 2^20 parameters, R = 2, zero moments, step 1, no clipping."""
    wl = W.CONFIGS["tiny"]
    grads = [W.rank_gradient(wl, r, step=1) for r in range(wl.R)]
    w = W.master_weights(wl)
    z = torch.zeros(wl.numel)
    got, want = run_both(ctx, sd, grads, w, z, z.clone(), dict(wl.hparams, step=1), 0.0)
    assert_parity("tiny", got, want, 0.0)


def prewarmed_state(wl, device="cpu"):
    """m, v (and the master) after `prewarm_steps` seeded ORACLE steps; never the CUDA path."""
    w = parity.f32(W.master_weights(wl, device=device)).copy()
    n = w.size
    m, v, p = np.zeros(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.uint16)
    for t in range(1, wl.prewarm_steps + 1):
        grads = [parity.u16(W.rank_gradient(wl, r, step=t, device=device)) for r in range(wl.R)]
        hp = oracle.HParams(inv_R=1.0 / wl.R, max_norm=wl.max_norm, step=t, **wl.hparams)
        oracle.step(grads, w, m, v, p, hp, nthreads=NTHREADS)
    return w, m, v


@pytest.mark.parametrize("divisor", [16, 1])
def test_config2_qwen3_8b_layer_step11_clipped(ctx, sd, divisor):
    """Qwen3-8B-shaped layer, R = 4, moments pre-warmed by 10 seeded steps, step 11, clip 1.0.
    divisor 1 is the full 192,946,176-parameter layer, compared element by element."""
    wl = W.CONFIGS["qwen3_8b_layer"]
    if divisor > 1:
        wl = W.scaled(wl, divisor)
    dev = "cuda"      # draw on the GPU (fast at full size); both sides get the same bits
    w, m, v = prewarmed_state(wl, dev)
    t = wl.first_step
    grads = [W.rank_gradient(wl, r, step=t, device=dev).cpu() for r in range(wl.R)]
    got, want = run_both(ctx, sd, grads, torch.from_numpy(w), torch.from_numpy(m),
                         torch.from_numpy(v), dict(wl.hparams, step=t), wl.max_norm)
    assert want[4] > 1.5, "clipping must be active in this configuration"
    assert_parity(wl.name, got, want, wl.max_norm)


@pytest.mark.parametrize("R,n", [(4, 16384 * 37 + 4321), (1, 16384 * 37 + 4321), (1, 16384 * 38),
                                 (1, 16384 * 36 + 3), (2, 16384 * 21 + 8), (8, 16384 * 5 + 9)])
def test_norm_is_deterministic_and_chunk_invariant(ctx, sd, R, n):
    """R = 1 runs its own launch shape (two tiles per block): cutting the step into single tiles
    below checks that it produces the bits of one-tile-at-a-time."""
    grads, *_ = random_case(n, R, seed=77, sigma=1e-2)
    dg = [g.cuda() for g in grads]
    ref = None
    for _ in range(3):
        ctx.slidedp_grad_norm(dg, n, 1.0 / R, True)
        out = ctx.slidedp_grad_norm_finish(1.0, fetch=True)
        ref = ref or out
        assert out == ref                                        # bit-identical run to run
    # chunks cut at multiples of the 16384-element tile: bit-identical to the uncut pass
    for cut in (16384, 16384 * 5, 16384 * 36):
        first = True
        for lo in range(0, n, cut):
            ctx.slidedp_grad_norm([g[lo:] for g in dg], min(cut, n - lo), 1.0 / R, first)
            first = False
        assert ctx.slidedp_grad_norm_finish(1.0, fetch=True) == ref
    # any other cut: same value to rounding
    first = True
    for lo in range(0, n, 100_000):
        ctx.slidedp_grad_norm([g[lo:] for g in dg], min(100_000, n - lo), 1.0 / R, first)
        first = False
    other = ctx.slidedp_grad_norm_finish(1.0, fetch=True)
    assert abs(other[0] - ref[0]) <= 1e-12 * ref[0]
    want = oracle.clip_coef(oracle.grad_sumsq([parity.u16(g) for g in grads], 1.0 / R), 1.0)
    parity.assert_norm_close(ref[0], want[1])
    assert abs(ref[1] - want[0]) <= 1e-6 * want[0]


def test_single_rank_norm_kernel_has_the_bits_of_the_generic_one(ctx, sd):
    """The R = 1 launch shape against the generic kernel on the same values: a second rank of
    zeros (g + 0 = g exactly) with the same 1/R argument must give the same norm, bit for bit."""
    for n in (16384 * 9 + 4321, 16384 * 4, 5, 16384 + 7):
        grads, *_ = random_case(n, 1, seed=n % 1000, sigma=3e-3)
        g = grads[0].cuda()
        zero = torch.zeros_like(g)
        ctx.slidedp_grad_norm([g], n, 0.5, True)
        one = ctx.slidedp_grad_norm_finish(0.7, fetch=True)
        ctx.slidedp_grad_norm([g, zero], n, 0.5, True)
        two = ctx.slidedp_grad_norm_finish(0.7, fetch=True)
        assert one == two and one[0] > 0.0


def test_update_is_chunk_invariant_bit_for_bit(ctx, sd):
    n, R = (1 << 18) + 8 * 13, 4
    grads, w, m, v = random_case(n, R, seed=5)
    whole, want = run_both(ctx, sd, grads, w, m, v, dict(ADAM, step=3), 0.02)
    assert_parity("whole", whole, want, 0.02)
    for chunk in (8, 4096, 100_000 - 100_000 % 8):
        parts, _ = run_both(ctx, sd, grads, w, m, v, dict(ADAM, step=3), 0.02, chunk=chunk)
        for a, b in zip(whole[:4], parts[:4]):
            assert np.array_equal(a, b)


def test_hyperparameter_and_value_ranges(ctx, sd):
    """Large lr, tiny and zero gradients, zero state, huge v, denormal-range gradients."""
    n, R = 4096 + 3, 2
    g = torch.Generator().manual_seed(9)
    mag = 10.0 ** (torch.rand(n, generator=g) * 36 - 34)          # 1e-34 .. 1e2
    sign = torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0)
    grads = [(mag * sign).to(torch.bfloat16), (mag * 0.5).to(torch.bfloat16)]
    grads[0][:16] = 0; grads[1][:16] = 0
    w = torch.randn(n, generator=g) * 0.02
    w[:4] = 0
    m = torch.zeros(n); v = torch.zeros(n)
    m[100:200] = torch.randn(100, generator=g) * 1e-20
    v[200:300] = 1e30
    for kw in (dict(lr=1e-2, beta1=0.5, beta2=0.999, eps=1e-6, weight_decay=0.0, step=2),
               dict(lr=1e-5, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1, step=100000),
               dict(lr=3e-4, beta1=0.0, beta2=0.0, eps=1e-8, weight_decay=0.01, step=1)):
        got, want = run_both(ctx, sd, grads, w, m, v, kw, 0.0)
        assert not np.isnan(got[0]).any()
        assert_parity(str(kw), got, want, 0.0)


def test_nonfinite_gradients_propagate_without_trapping(ctx, sd):
    n, R = 64, 2
    grads, w, m, v = random_case(n, R, seed=3)
    grads[0][5] = float("inf"); grads[1][9] = float("nan")
    got, want = run_both(ctx, sd, grads, w, m, v, dict(ADAM, step=2), 0.0)
    for a, b in zip(got[:3], want[:3]):
        assert np.array_equal(np.isfinite(a), np.isfinite(b))
    keep = np.ones(n, bool); keep[[5, 9]] = False
    for a, b in zip(got[:3], want[:3]):
        parity.assert_fp32_close("finite part", a[keep], b[keep])
    dg = [g.cuda() for g in grads]
    ctx.slidedp_grad_norm(dg, n, 0.5, True)
    norm, coef = ctx.slidedp_grad_norm_finish(1.0, fetch=True)
    assert np.isnan(norm) and np.isnan(coef)


def test_argument_errors_are_reported_not_faulted(ctx, sd):
    n = 64
    g = [torch.zeros(n + 8, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    w = torch.zeros(n + 8, device="cuda")
    p = torch.zeros(n + 8, dtype=torch.bfloat16, device="cuda")
    hp = sd.HParams(inv_R=0.5, step=1)

    def status(fn):
        with pytest.raises(sd.SlideDPError) as e:
            fn()
        return e.value.status

    call = ctx.slidedp_reduce_adamw_chunk
    assert status(lambda: call([g[0][1:], g[1]], n, w, w.clone(), w.clone(), p, hp)) == sd.ERR_MISALIGNED
    assert status(lambda: call(g, n, w[1:], w.clone(), w.clone(), p, hp)) == sd.ERR_MISALIGNED
    assert status(lambda: call(g, -1, w, w.clone(), w.clone(), p, hp)) == sd.ERR_INVALID_ARG
    assert status(lambda: call([], n, w, w.clone(), w.clone(), p, hp)) == sd.ERR_INVALID_ARG
    assert status(lambda: call(g * 9, n, w, w.clone(), w.clone(), p, hp)) == sd.ERR_INVALID_ARG
    assert status(lambda: call(g, n, None, w.clone(), w.clone(), p, hp)) == sd.ERR_INVALID_ARG
    assert status(lambda: call(g, n, w, w.clone(), w.clone(), p,
                               sd.HParams(inv_R=0.5, step=0))) == sd.ERR_INVALID_ARG
    assert status(lambda: call(g, n, w, w.clone(), w.clone(), p,
                               sd.HParams(inv_R=0.5, beta1=1.0))) == sd.ERR_INVALID_ARG
    fresh = sd.slidedp_create(0, 0)
    try:
        assert status(lambda: fresh.slidedp_reduce_adamw_chunk(
            g, n, w, w.clone(), w.clone(), p, sd.HParams(inv_R=0.5, max_norm=1.0))) == sd.ERR_NO_NORM
    finally:
        fresh.slidedp_destroy()
    torch.cuda.synchronize()
    assert torch.all(w == 0)


def test_indices_beyond_2_to_31(ctx, sd):
    """A chunk of 2^31 + 4099 parameters (34 GB on the device): 64-bit indexing in both kernels.
    The update is elementwise, so the oracle checks slices (head, around 2^31, ragged tail) with
    the global coefficient; the norm is checked over the whole range."""
    n, R = (1 << 31) + 4099, 1
    free, _ = torch.cuda.mem_get_info()
    if free < 45 << 30:
        pytest.skip("needs 45 GB of free device memory")
    gen = torch.Generator(device="cuda").manual_seed(2031)
    g = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    w = torch.empty(n, device="cuda")
    seg = 1 << 27
    for lo in range(0, n, seg):
        k = min(seg, n - lo)
        g[lo:lo + k] = (torch.randn(k, generator=gen, device="cuda") * 1e-3).to(torch.bfloat16)
        w[lo:lo + k] = torch.randn(k, generator=gen, device="cuda") * 0.02
    m = w * 0.01
    v = w * w * 1e-3
    p = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    slices = [(0, 1 << 20), ((1 << 31) - (1 << 19), (1 << 31) + 2048), (n - (1 << 20), n)]
    before = [[parity.f32(t[a:b]).copy() for t in (w, m, v)] for a, b in slices]
    kw = dict(ADAM, inv_R=1.0, max_norm=1.0, step=11)
    ctx.slidedp_grad_norm([g], n, 1.0, True)
    norm_g, coef_g = ctx.slidedp_grad_norm_finish(1.0, fetch=True)
    ctx.slidedp_reduce_adamw_chunk([g], n, w, m, v, p, sd.HParams(**kw))
    torch.cuda.synchronize()
    hg = parity.u16(g)
    coef_o, norm_o = oracle.clip_coef(oracle.grad_sumsq([hg], 1.0, NTHREADS), 1.0)
    parity.assert_norm_close(norm_g, norm_o)
    assert coef_o < 1.0 and abs(coef_g - coef_o) <= 1e-6 * coef_o
    for (a, b), (ow, om, ov) in zip(slices, before):
        op = np.zeros(b - a, np.uint16)
        oracle.reduce_adamw_chunk([hg[a:b].copy()], ow, om, ov, op, oracle.HParams(**kw),
                                  clip=coef_o, nthreads=NTHREADS)
        tag = f"[{a}:{b}]"
        parity.assert_fp32_close(tag + "/master", parity.f32(w[a:b]), ow)
        parity.assert_fp32_close(tag + "/m", parity.f32(m[a:b]), om)
        parity.assert_fp32_close(tag + "/v", parity.f32(v[a:b]), ov)
        parity.assert_bf16_close(tag + "/param_bf16", parity.u16(p[a:b]), op)
    # nothing outside the chunk was touched and every element inside was written
    assert int((p == 0).sum()) < n // 1000


@pytest.mark.parametrize("n", [1, 3, 4, 5, 1021, 1024, 1027, 16384, 16385, 65536 + 7])
def test_guard_bands_around_every_buffer_stay_intact(ctx, sd, n):
    """Every output (and input) sits between 64-element canary bands; after the norm, the update
    and the delivery cast, the bands are unchanged and every element inside was written once."""
    R, pad = 3, 64
    gen = torch.Generator(device="cuda").manual_seed(n)

    def banded(dtype, fill):
        t = torch.full((n + 2 * pad,), fill, dtype=dtype, device="cuda")
        return t, t[pad:pad + n]

    gfull, grads = zip(*[banded(torch.bfloat16, 123.0) for _ in range(R)])
    for g in grads:
        g.copy_((torch.randn(n, generator=gen, device="cuda") * 1e-3).to(torch.bfloat16))
    wfull, w = banded(torch.float32, -7.0)
    mfull, m = banded(torch.float32, -7.0)
    vfull, v = banded(torch.float32, -7.0)
    pfull, p = banded(torch.bfloat16, -7.0)
    w.copy_(torch.randn(n, generator=gen, device="cuda") * 0.02); m.zero_(); v.zero_()
    snap = [t.clone() for t in gfull]
    ctx.slidedp_grad_norm(list(grads), n, 1.0 / R, True)
    ctx.slidedp_grad_norm_finish(0.01)
    ctx.slidedp_reduce_adamw_chunk(list(grads), n, w, m, v, p, sd.HParams(inv_R=1.0 / R, max_norm=0.01,
                                                                           step=1))
    torch.cuda.synchronize()
    for full, fill in ((wfull, -7.0), (mfull, -7.0), (vfull, -7.0), (pfull, -7.0)):
        assert torch.all(full[:pad] == fill) and torch.all(full[pad + n:] == fill)
    assert all(torch.equal(a, b) for a, b in zip(snap, gfull))          # gradients are read-only
    assert torch.all(p.float() != -7.0) and torch.all(v >= 0) and torch.all(m.abs() < 1.0)
    # delivery cast into a banded output
    host = torch.empty(n, pin_memory=True); host.copy_(w)
    pfull.fill_(-7.0)
    torch.cuda.synchronize()
    ctx.slidedp_deliver_params(host, n, p, 8, 2)
    assert torch.all(pfull[:pad] == -7.0) and torch.all(pfull[pad + n:] == -7.0)
    assert torch.equal(p, w.to(torch.bfloat16))


def test_random_hyperparameters_and_steps(ctx, sd):
    """Forty seeded draws of (lr, betas, eps, weight decay, step, clip, R) on a ragged chunk."""
    rng = np.random.default_rng(2024)
    n = 4099
    for case in range(40):
        R = int(rng.integers(1, 17))
        kw = dict(lr=float(10 ** rng.uniform(-6, -2)), beta1=float(rng.choice([0.0, 0.5, 0.8, 0.9, 0.99])),
                  beta2=float(rng.choice([0.0, 0.9, 0.95, 0.999, 0.9999])),
                  eps=float(10 ** rng.uniform(-12, -5)), weight_decay=float(rng.choice([0.0, 0.01, 0.1, 1.0])),
                  step=int(rng.choice([1, 2, 10, 1000, 10 ** 6])))
        clip = float(rng.choice([0.0, 1e-3, 1.0, 1e3]))
        grads, w, m, v = random_case(n, R, seed=5000 + case, zero_moments=bool(case % 3 == 0),
                                     sigma=float(10 ** rng.uniform(-5, -1)))
        got, want = run_both(ctx, sd, grads, w, m, v, kw, clip)
        assert_parity(f"case {case}: R={R} clip={clip} {kw}", got, want, clip)


def test_whole_step_replays_from_a_cuda_graph(ctx, sd):
    """Norm, finish and update only enqueue work on the caller's stream (no allocation, no
    synchronisation), so a step can be captured once and replayed; the replay gives the bits of
    the eager step."""
    n, R = (1 << 18) + 5, 4
    grads, w, m, v = random_case(n, R, seed=42)
    dg = [g.cuda() for g in grads]
    hp = sd.HParams(inv_R=0.25, max_norm=0.02, step=2)

    def fresh():
        return w.cuda(), m.cuda(), v.cuda(), torch.zeros(n, dtype=torch.bfloat16, device="cuda")

    def step(state):
        ctx.slidedp_grad_norm(dg, n, 0.25, True)
        ctx.slidedp_grad_norm_finish(0.02)
        ctx.slidedp_reduce_adamw_chunk(dg, n, *state, hp)

    eager = fresh()
    step(eager)
    torch.cuda.synchronize()
    replayed = fresh()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step(replayed)
    for t, src in zip(replayed, fresh()):
        t.copy_(src)                      # capture does not execute: start from the same state
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip(eager, replayed):
        assert torch.equal(a, b)


@pytest.mark.parametrize("R", [1, 2, 3, 4, 7, 8, 16])
def test_rank_reduction_alone_returns_the_bf16_mean_bit_exact(ctx, sd, R):
    for n in (0, 5, 8, 4099, (1 << 20) + 7):
        g = torch.Generator().manual_seed(100 * R + n % 89)
        scale = 2.0 ** torch.randint(-10, 1, (R, max(n, 1)), generator=g).float()
        grads = [(torch.randn(max(n, 1), generator=g) * 1e-2 * scale[r]).to(torch.bfloat16)[:n]
                 for r in range(R)]
        out = torch.full((max(n, 8),), 9.0, dtype=torch.bfloat16, device="cuda")
        dg = [x.cuda() for x in grads] if n else [out] * R      # n = 0 still needs real pointers
        ctx.slidedp_reduce_mean_bf16(dg, n, 1.0 / R, out)
        torch.cuda.synchronize()
        want = oracle.reduce_mean_bf16([parity.u16(x) for x in grads], 1.0 / R) if n else np.zeros(0, np.uint16)
        assert np.array_equal(parity.u16(out[:n]), want), (R, n)
        assert torch.all(out[n:] == 9.0)


@pytest.mark.parametrize("seed", range(8))
def test_config2_shape_many_seeds_multi_step(ctx, sd, seed):
    """The benchmark's hyper-parameters on a 3 M-parameter cut of the layer, eight seeds, three
    consecutive clipped steps each, both sides restarted from the oracle's state every step so
    that each step is a single-step comparison on realistic warm moments."""
    import dataclasses
    wl = dataclasses.replace(W.scaled(W.CONFIGS["qwen3_8b_layer"], 64), seed=100 + seed)
    n, R = wl.numel, wl.R
    w = parity.f32(W.master_weights(wl)).copy()
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    for t in range(1, 4):
        grads = [W.rank_gradient(wl, r, step=t) for r in range(R)]
        got, want = run_both(ctx, sd, grads, torch.from_numpy(w), torch.from_numpy(m),
                             torch.from_numpy(v), dict(wl.hparams, step=t), 0.5)
        assert_parity(f"seed {seed} step {t}", got, want, 0.5)
        w, m, v = want[0], want[1], want[2]


@pytest.mark.parametrize("shards", [2, 3, 4, 8])
def test_sharded_step_emulated_on_one_gpu_is_bit_identical(ctx, sd, shards):
    """The multi-GPU form of the step, emulated as one GPU doing every shard in turn: tile-aligned
    shard bounds, per-shard tile sums written to one gathered array in shard order, the fold of
    that array on "every GPU", and the fused update of each shard from all ranks' gradient slices.
    Norm, coefficient, state and BF16 copy must equal the unsharded step bit for bit."""
    n, R = 16384 * 19 + 777, 4
    grads, w, m, v = random_case(n, R, seed=900 + shards, sigma=1e-2)
    dg = [g.cuda() for g in grads]
    hp = sd.HParams(inv_R=0.25, max_norm=0.5, step=3)
    # unsharded reference
    rw, rm, rv = w.cuda(), m.cuda(), v.cuda()
    rp = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    ctx.slidedp_grad_norm(dg, n, 0.25, True)
    ref = ctx.slidedp_grad_norm_finish(0.5, fetch=True)
    ctx.slidedp_reduce_adamw_chunk(dg, n, rw, rm, rv, rp, hp)
    # sharded
    bounds = sd.shard_bounds(n, shards)
    assert bounds[0][0] == 0 and bounds[-1][1] == n
    assert all(a[1] == b[0] for a, b in zip(bounds, bounds[1:]))
    assert all(lo % sd.NORM_TILE == 0 for lo, _ in bounds)
    total_tiles = -(-n // sd.NORM_TILE)
    gathered = torch.full((total_tiles,), float("nan"), dtype=torch.float64, device="cuda")
    at = 0
    for lo, hi in bounds:
        ctx.slidedp_grad_norm_tiles([g[lo:] for g in dg], hi - lo, 0.25, gathered[at:])
        at += -(-(hi - lo) // sd.NORM_TILE)
    assert at == total_tiles
    got = ctx.slidedp_grad_norm_finish_from(gathered, total_tiles, 0.5, fetch=True)
    assert got == ref
    sw, sm, sv = w.cuda(), m.cuda(), v.cuda()
    sp = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    for lo, hi in reversed(bounds):                      # any order: shards are independent
        ctx.slidedp_reduce_adamw_chunk([g[lo:] for g in dg], hi - lo, sw[lo:], sm[lo:], sv[lo:],
                                       sp[lo:], hp)
    torch.cuda.synchronize()
    for a, b in ((sw, rw), (sm, rm), (sv, rv), (sp, rp)):
        assert torch.equal(a, b)


def test_hbm_mix_probe_leaves_the_state_unchanged(ctx, sd):
    """The roofline probe issues the update kernel's loads and stores without arithmetic: the FP32
    state comes back bit for bit, only the scratch output changes, and a rate is reported."""
    n, R = (1 << 22) + 6, 4
    grads, w, m, v = random_case(n, R, seed=8)
    dg = [g.cuda() for g in grads]
    dw, dm, dv = w.cuda(), m.cuda(), v.cuda()
    scratch = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()
    gbs = ctx.slidedp_hbm_mix_probe(dg, n, dw, dm, dv, scratch, 3)
    torch.cuda.synchronize()
    assert gbs > 100.0
    assert torch.equal(dw.cpu(), w) and torch.equal(dm.cpu(), m) and torch.equal(dv.cpu(), v)
    assert all(torch.equal(a.cpu(), b) for a, b in zip(dg, grads))
    assert scratch.view(torch.int16).count_nonzero() > n // 2
    assert not scratch[-2:].view(torch.int16).any()          # the ragged tail is not touched
    with pytest.raises(sd.SlideDPError) as e:
        ctx.slidedp_hbm_mix_probe(dg, 2, dw, dm, dv, scratch, 3)
    assert e.value.status == sd.ERR_INVALID_ARG
