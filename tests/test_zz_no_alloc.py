"""slidedp_grad_norm_noalloc: the global norm for callers that must not allocate device
memory (allocator callbacks, processes whose memory budget is fully committed, plug-ins that
only receive pointers). It keeps its tile sums in a fixed array inside the library, so it is
checked here against the context-based entry points, which allocate theirs: same kernels and
summation tree, so the results must agree (the tolerance of the other norm tests, 1e-6
relative, is the bar; in practice the bits are equal).

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test. It passes alone in a fresh process and after the other tests."""
import numpy as np
import pytest
import torch

import oracle
import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sd():
    import paper_2609_34162_b200.slidedp as sd
    return sd


def reference(sd, grads, n, inv_R, max_norm):
    ctx = sd.slidedp_create(0, 0)
    try:
        ctx.slidedp_grad_norm(grads, n, inv_R, True)
        return ctx.slidedp_grad_norm_finish(max_norm, fetch=True)
    finally:
        ctx.slidedp_destroy()


def test_two_calls_in_a_row_match_the_allocating_entry_point(sd):
    g = torch.Generator(device="cuda").manual_seed(123)
    out = torch.full((4,), -1.0, dtype=torch.float64, device="cuda")
    # a large call first, then a smaller one with other data: the second must not see what the
    # first left in the shared array
    for n, R, sigma, max_norm in ((16384 * 41 + 777, 4, 1e-2, 1.0), (16384 * 3 + 5, 2, 3e-4, 0.5)):
        grads = [(torch.randn(n, generator=g, device="cuda") * sigma).to(torch.bfloat16)
                 for _ in range(R)]
        sd.slidedp_grad_norm_noalloc(grads, n, 1.0 / R, max_norm, out)
        torch.cuda.synchronize()
        sumsq, norm, coef, nonfinite = out.tolist()
        want_norm, want_coef = reference(sd, grads, n, 1.0 / R, max_norm)
        assert abs(norm - want_norm) <= 1e-6 * want_norm
        assert abs(coef - want_coef) <= 1e-6 * want_coef
        assert abs(sumsq - want_norm ** 2) <= 1e-6 * sumsq and nonfinite == 0.0
        assert (norm, coef) == (want_norm, want_coef)          # same tree, same bits
        # and directly against the CPU oracle, at the tolerance of the other norm tests
        S = oracle.grad_sumsq([parity.u16(x) for x in grads], 1.0 / R, 4)
        coef_o, norm_o = oracle.clip_coef(S, max_norm)
        parity.assert_norm_close(norm, norm_o)
        assert abs(coef - coef_o) <= 1e-6 * coef_o and abs(sumsq - S) <= 2e-6 * S


def test_calls_after_the_first_take_no_device_memory(sd):
    """The point of the entry point: once the set-up call on this device has been made (it may
    load the library's device image), further calls must not move the device's free memory.
    Every buffer is created before the measurement, so torch's own allocator is quiet too."""
    g = torch.Generator(device="cuda").manual_seed(7)
    n, R = 16384 * 9 + 11, 3
    grads = [(torch.randn(n, generator=g, device="cuda") * 1e-3).to(torch.bfloat16) for _ in range(R)]
    out = torch.zeros(4, dtype=torch.float64, device="cuda")
    sd.slidedp_grad_norm_noalloc(grads, 0, 1.0 / R, 1.0, out)       # set-up call, n = 0
    torch.cuda.synchronize()
    assert out.tolist() == [0.0, 0.0, 1.0, 0.0]
    torch.cuda.mem_get_info()
    free_before, _ = torch.cuda.mem_get_info()
    seen = set()
    for _ in range(5):
        sd.slidedp_grad_norm_noalloc(grads, n, 1.0 / R, 1.0, out)
        torch.cuda.synchronize()
        seen.add(tuple(out.tolist()))
        assert torch.cuda.mem_get_info()[0] == free_before
    assert len(seen) == 1 and next(iter(seen))[1] > 0.0              # and the same bits every time


def test_limits_and_argument_errors(sd):
    out = torch.zeros(4, dtype=torch.float64, device="cuda")
    g = [torch.zeros(64, dtype=torch.bfloat16, device="cuda")]

    def status(fn):
        with pytest.raises(sd.SlideDPError) as e:
            fn()
        return e.value.status

    call = sd.slidedp_grad_norm_noalloc
    assert status(lambda: call(g, sd.NOALLOC_MAX_ELEMS + 1, 1.0, 1.0, out)) == sd.ERR_TOO_LARGE
    assert "capacity" in sd.slidedp_strerror(sd.ERR_TOO_LARGE)
    assert status(lambda: call(g, -1, 1.0, 1.0, out)) == sd.ERR_INVALID_ARG
    assert status(lambda: call(g, 64, 1.0, 1.0, None)) == sd.ERR_INVALID_ARG
    assert status(lambda: call([g[0][1:]], 8, 1.0, 1.0, out)) == sd.ERR_MISALIGNED
    call(g, 0, 1.0, 1.0, out)                                   # empty chunk: norm 0, coef 1
    torch.cuda.synchronize()
    assert out.tolist() == [0.0, 0.0, 1.0, 0.0]
