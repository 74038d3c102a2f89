"""Failure handling of libslidedp, exercised on the HOST only: nothing here faults, traps or hangs
the GPU. (Paper Sec. 3.3 "Completion and buffer reuse" is the only related passage; the bounded
waits and the error contract are this library's.)

  * a wait bound of a millisecond makes slidedp_stream_wait / slidedp_stream_step give up with
    SLIDEDP_ERR_TIMEOUT while perfectly healthy copies are still running; they simply finish, a
    later wait succeeds, and the step's results are complete and correct;
  * the host-side hook slidedp_test_fail_nth_call makes the nth runtime call of an entry point
    report failure without issuing it; every entry point then returns SLIDEDP_ERR_CUDA, leaves
    nothing running on the caller's buffers, and the context computes a correct step afterwards.
"""
import numpy as np
import pytest
import torch

import oracle
import parity

pytestmark = pytest.mark.gpu

CUDA_ERROR_UNKNOWN = 999


@pytest.fixture(scope="module")
def sd():
    import paper_2609_34162_b200.slidedp as sd
    return sd


@pytest.fixture()
def ctx(sd):
    c = sd.slidedp_create(0, 0)
    yield c
    c.slidedp_destroy()


def pinned(a: np.ndarray) -> torch.Tensor:
    t = torch.empty(a.shape, dtype=torch.float32, pin_memory=True)
    t.numpy()[...] = a
    return t


class Case:
    """A small clipped step with its oracle result, replayable on any context."""

    def __init__(self, sd, n=5 * 4096 + 37, R=3, seed=5, nthreads=1):
        g = torch.Generator().manual_seed(seed)
        self.sd, self.n, self.R = sd, n, R
        self.grads = [(torch.randn(n, generator=g) * 1e-2).to(torch.bfloat16) for _ in range(R)]
        self.w0 = (torch.randn(n, generator=g) * 0.02).numpy()
        self.m0 = (torch.randn(n, generator=g) * 1e-3).numpy()
        self.v0 = (torch.randn(n, generator=g).square() * 1e-6).numpy()
        self.kw = dict(inv_R=1.0 / R, max_norm=0.05, step=4, lr=1e-3, beta1=0.9, beta2=0.95,
                       eps=1e-8, weight_decay=0.1)
        self.ow, self.om, self.ov = self.w0.copy(), self.m0.copy(), self.v0.copy()
        self.op = np.zeros(n, np.uint16)
        self.norm, self.coef = oracle.step([parity.u16(x) for x in self.grads], self.ow, self.om,
                                           self.ov, self.op, oracle.HParams(**self.kw),
                                           nthreads=nthreads)
        self.dg = [x.cuda() for x in self.grads]
        torch.cuda.synchronize()

    def check_host_step(self, ctx, chunk=4096, nbuf=3):
        """One synchronous host-resident step on `ctx`, checked against the oracle."""
        hw, hm, hv = pinned(self.w0), pinned(self.m0), pinned(self.v0)
        dp = torch.zeros(self.n, dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        st = ctx.slidedp_stream_step(self.dg, self.n, hw, hm, hv, dp, chunk, nbuf,
                                     self.sd.HParams(**self.kw))
        self.check_state(hw.numpy(), hm.numpy(), hv.numpy(), parity.u16(dp))
        parity.assert_norm_close(st["norm"], self.norm)

    def check_state(self, w, m, v, p):
        parity.assert_fp32_close("master", w, self.ow)
        parity.assert_fp32_close("m", m, self.om)
        parity.assert_fp32_close("v", v, self.ov)
        parity.assert_bf16_close("param_bf16", p, self.op)


def test_a_wait_that_runs_out_returns_timeout_and_the_work_still_completes(ctx, sd):
    """A large asynchronous step (about 1.5 GB each way over the host link, tens of ms) and a wait
    bound of one millisecond: TIMEOUT, nothing cancelled; with the bound restored the wait
    succeeds, the result is the oracle's, and the context runs another correct step."""
    case = Case(sd, n=(1 << 27) + 4099, R=2, seed=9, nthreads=16)
    hw, hm, hv = pinned(case.w0), pinned(case.m0), pinned(case.v0)
    dp = torch.zeros(case.n, dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()
    ctx.slidedp_set_wait_seconds(1e-3)
    ctx.slidedp_stream_step_async(case.dg, case.n, hw, hm, hv, dp, 1 << 22, 3, sd.HParams(**case.kw))
    with pytest.raises(sd.SlideDPError) as e:
        ctx.slidedp_stream_wait()
    assert e.value.status == sd.ERR_TIMEOUT
    with pytest.raises(sd.SlideDPError) as e:              # still running: still a timeout,
        ctx.slidedp_stream_wait()                          # and still nothing broken
    assert e.value.status == sd.ERR_TIMEOUT
    ctx.slidedp_set_wait_seconds(300.0)
    ctx.slidedp_stream_wait()
    case.check_state(hw.numpy(), hm.numpy(), hv.numpy(), parity.u16(dp))
    # the synchronous call times out the same way and completes the same way
    hw, hm, hv = pinned(case.w0), pinned(case.m0), pinned(case.v0)
    dp.zero_()
    torch.cuda.synchronize()
    ctx.slidedp_set_wait_seconds(1e-3)
    with pytest.raises(sd.SlideDPError) as e:
        ctx.slidedp_stream_step(case.dg, case.n, hw, hm, hv, dp, 1 << 22, 3, sd.HParams(**case.kw))
    assert e.value.status == sd.ERR_TIMEOUT
    ctx.slidedp_set_wait_seconds(300.0)
    ctx.slidedp_stream_wait()
    case.check_state(hw.numpy(), hm.numpy(), hv.numpy(), parity.u16(dp))
    Case(sd).check_host_step(ctx)


def test_wait_bound_argument_errors(ctx, sd):
    for bad in (0.0, -1.0, float("nan"), 1e6):
        with pytest.raises(sd.SlideDPError) as e:
            ctx.slidedp_set_wait_seconds(bad)
        assert e.value.status == sd.ERR_INVALID_ARG


def _sweep(ctx, sd, call, after_failure, limit=400):
    """Fails the 1st, 2nd, ... guarded runtime call of `call` in turn until it gets through
    untouched; returns how many distinct failure points were hit."""
    failures = 0
    for nth in range(1, limit):
        ctx.slidedp_test_fail_nth_call(nth)
        try:
            call()
        except sd.SlideDPError as e:
            assert e.status == sd.ERR_CUDA and e.cuda_error == CUDA_ERROR_UNKNOWN, (nth, e)
            assert ctx.slidedp_last_cuda_error() == CUDA_ERROR_UNKNOWN
            failures += 1
            ctx.slidedp_test_fail_nth_call(0)
            after_failure(nth)
            continue
        ctx.slidedp_test_fail_nth_call(0)
        return failures
    raise AssertionError("the call never got through")


def test_every_streaming_entry_point_survives_a_failed_runtime_call(ctx, sd):
    case = Case(sd)
    n = case.n
    state = {}

    def fresh():
        state["h"] = [pinned(case.w0), pinned(case.m0), pinned(case.v0)]
        state["p"] = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()

    def usable(nth):
        # whatever was queued has finished (nothing touches the buffers any more): every chunk
        # of the failed step holds either its old or its new values, never anything else
        torch.cuda.synchronize()
        for got, old, new in zip(state["h"], (case.w0, case.m0, case.v0), (case.ow, case.om, case.ov)):
            g = got.numpy()
            is_new = np.abs(g.astype(np.float64) - new) <= np.maximum(1e-6 * np.abs(new), 1e-12)
            assert np.all((g == old) | is_new)
        if nth % 7 == 1:                      # and the context still computes a correct step
            case.check_host_step(ctx)

    hp = sd.HParams(**case.kw)

    def sync_step():
        fresh()
        ctx.slidedp_stream_step(case.dg, n, *state["h"], state["p"], 4096, 3, hp)

    hits = _sweep(ctx, sd, sync_step, usable)
    assert hits >= 6 * 15                     # six chunks, some fifteen calls each
    case.check_state(*(h.numpy() for h in state["h"]), parity.u16(state["p"]))

    def async_step():
        fresh()
        ctx.slidedp_stream_step_async(case.dg, n, *state["h"], state["p"], 8192, 2, hp)
        ctx.slidedp_stream_wait()

    assert _sweep(ctx, sd, async_step, usable) >= 3 * 12
    case.check_state(*(h.numpy() for h in state["h"]), parity.u16(state["p"]))

    # the multi-layer step: two layers (the two halves of the case), one global norm
    half = (n // 2) // 8 * 8

    def layers_step():
        fresh()
        h, p = state["h"], state["p"]
        ctx.slidedp_stream_layers(
            [([g[:half] for g in case.dg], half, h[0][:half], h[1][:half], h[2][:half], p[:half]),
             ([g[half:] for g in case.dg], n - half, h[0][half:], h[1][half:], h[2][half:], p[half:])],
            4096, 3, hp)

    assert _sweep(ctx, sd, layers_step, usable) >= 6 * 14
    case.check_state(*(h.numpy() for h in state["h"]), parity.u16(state["p"]))

    # parameter delivery
    master = pinned(case.ow)
    out = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()
    assert _sweep(ctx, sd, lambda: ctx.slidedp_deliver_params(master, n, out, 4096, 2),
                  lambda nth: case.check_host_step(ctx) if nth % 9 == 1 else None) >= 6 * 4
    assert np.array_equal(parity.u16(out), case.op)

    # link probe
    ha, hb = (torch.empty(1 << 20, dtype=torch.uint8, pin_memory=True) for _ in range(2))
    da, db = (torch.empty(1 << 20, dtype=torch.uint8, device="cuda") for _ in range(2))
    assert _sweep(ctx, sd, lambda: ctx.slidedp_link_probe(ha, hb, da, db, 1 << 20, 1 << 18, 1),
                  lambda nth: None) >= 4
    case.check_host_step(ctx)


def test_every_device_resident_entry_point_survives_a_failed_runtime_call(ctx, sd):
    """A failed launch queues nothing: the state is untouched and the call can simply be repeated."""
    case = Case(sd)
    n = case.n
    dw, dm, dv = (torch.from_numpy(x).cuda() for x in (case.w0, case.m0, case.v0))
    dp = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    tiles = torch.zeros(-(-n // sd.NORM_TILE), dtype=torch.float64, device="cuda")
    out = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()
    hp = sd.HParams(**case.kw)
    nothing = lambda nth: None

    assert _sweep(ctx, sd, lambda: ctx.slidedp_grad_norm(case.dg, n, case.kw["inv_R"], True), nothing) == 1
    got = {}
    def finish():
        got["nc"] = ctx.slidedp_grad_norm_finish(case.kw["max_norm"], fetch=True)
    assert _sweep(ctx, sd, finish, nothing) == 3          # launch, copy of the scalars, event
    parity.assert_norm_close(got["nc"][0], case.norm)

    def untouched(nth):
        torch.cuda.synchronize()
        assert np.array_equal(parity.f32(dw), case.w0) and np.array_equal(parity.f32(dm), case.m0)
        assert np.array_equal(parity.f32(dv), case.v0) and not parity.u16(dp).any()

    assert _sweep(ctx, sd, lambda: ctx.slidedp_reduce_adamw_chunk(case.dg, n, dw, dm, dv, dp, hp),
                  untouched) == 1
    torch.cuda.synchronize()
    case.check_state(parity.f32(dw), parity.f32(dm), parity.f32(dv), parity.u16(dp))

    assert _sweep(ctx, sd, lambda: ctx.slidedp_reduce_mean_bf16(case.dg, n, case.kw["inv_R"], out),
                  nothing) == 1
    torch.cuda.synchronize()
    assert np.array_equal(parity.u16(out), oracle.reduce_mean_bf16([parity.u16(g) for g in case.grads],
                                                                   case.kw["inv_R"]))
    assert _sweep(ctx, sd, lambda: ctx.slidedp_grad_norm_tiles(case.dg, n, case.kw["inv_R"], tiles),
                  nothing) == 1
    def finish_from():
        got["nc2"] = ctx.slidedp_grad_norm_finish_from(tiles, tiles.numel(), case.kw["max_norm"], fetch=True)
    assert _sweep(ctx, sd, finish_from, nothing) == 3
    assert got["nc2"] == got["nc"]
    # the sharded step's entry points and the roofline probe
    dsts = [torch.zeros_like(tiles), torch.zeros_like(tiles)]
    assert _sweep(ctx, sd, lambda: ctx.slidedp_scatter_tile_sums(tiles, tiles.numel(), dsts), nothing) == 1
    torch.cuda.synchronize()
    assert all(torch.equal(d, tiles) for d in dsts)
    b = [torch.from_numpy(x).cuda() for x in (case.w0, case.m0, case.v0)]
    outs = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    torch.cuda.synchronize()
    assert _sweep(ctx, sd, lambda: ctx.slidedp_reduce_adamw_chunk_bcast(case.dg, n, *b, outs, hp),
                  nothing) == 1
    torch.cuda.synchronize()
    case.check_state(*(parity.f32(x) for x in b), parity.u16(outs[1]))
    assert _sweep(ctx, sd, lambda: ctx.slidedp_ipc_export(outs[0]), nothing) == 2
    assert len(ctx.slidedp_ipc_export(outs[0])) == sd.IPC_HANDLE_BYTES
    assert _sweep(ctx, sd, lambda: ctx.slidedp_hbm_mix_probe(case.dg, n, *b, outs[0], 1), nothing) >= 1
    torch.cuda.synchronize()
    case.check_state(*(parity.f32(x) for x in b), parity.u16(outs[1]))      # the probe left the state alone


def test_non_finite_hyper_parameters_are_rejected(ctx, sd):
    n = 64
    g = [torch.zeros(n, dtype=torch.bfloat16, device="cuda")]
    w, m, v = (torch.zeros(n, device="cuda") for _ in range(3))
    p = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    for field in ("lr", "eps", "weight_decay", "inv_R"):
        for bad in (float("inf"), float("-inf"), float("nan")):
            with pytest.raises(sd.SlideDPError) as e:
                ctx.slidedp_reduce_adamw_chunk(g, n, w, m, v, p, sd.HParams(**{field: bad}))
            assert e.value.status == sd.ERR_INVALID_ARG, (field, bad)
    with pytest.raises(sd.SlideDPError) as e:
        ctx.slidedp_reduce_adamw_chunk(g, n, w, m, v, p, sd.HParams(max_norm=float("nan")))
    assert e.value.status == sd.ERR_INVALID_ARG
    ctx.slidedp_reduce_adamw_chunk(g, n, w, m, v, p, sd.HParams())       # and a finite set passes
    torch.cuda.synchronize()
