"""GPU parity of slidedp_deliver_params (the BF16 copy of a host-resident FP32 master, the step
before the update path): bit-exact against the oracle's cast."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2609_34162_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sd():
    import paper_2609_34162_b200.slidedp as sd
    return sd


@pytest.fixture()
def ctx(sd):
    c = sd.slidedp_create(0, 0)
    yield c
    c.slidedp_destroy()


def same_bf16(got: np.ndarray, want: np.ndarray) -> bool:
    """Bit-exact, except that any NaN pattern matches any NaN pattern (payloads are not part
    of the definition: a NaN stays a NaN)."""
    def is_nan(b):
        return ((b & 0x7F80) == 0x7F80) & ((b & 0x007F) != 0)
    nan = is_nan(got)
    return bool(np.array_equal(nan, is_nan(want)) and np.array_equal(got[~nan], want[~nan]))


def deliver(ctx, host, chunk, nbuf):
    n = host.numel()
    out = torch.full((max(n, 8),), 7.0, dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()          # the fill ran on torch's stream, the library uses its own
    st = ctx.slidedp_deliver_params(host, n, out, chunk, nbuf)
    return parity.u16(out[:n]), st


@pytest.mark.parametrize("n", [0, 1, 7, 8, 9, 4099, (1 << 20) + 3])
def test_ragged_sizes_and_specials_bit_exact(ctx, n):
    g = torch.Generator().manual_seed(n)
    host = torch.empty(n, pin_memory=True)
    host.copy_(torch.randn(n, generator=g) * 0.02)
    if n >= 9:
        host[:9] = torch.tensor([0.0, -0.0, float("inf"), float("-inf"), 1.00390625, 1.01171875,
                                 1e-40, -3.4e38, float("nan")])
    want = oracle.cast_master_to_bf16(host.numpy().copy())
    for chunk, nbuf in ((8, 2), (1024, 3), (1 << 18, 2), (1 << 22, 3)):
        if n > 100_000 and chunk == 8:
            continue
        got, st = deliver(ctx, host, chunk, nbuf)
        assert same_bf16(got, want), (n, chunk, nbuf)
        assert st["chunks"] == -(-n // chunk)


def test_config3_layer_full_size_and_agreement_with_the_update_path(ctx, sd):
    """The 330,311,680-parameter Qwen3-14B-shaped layer in 64 MiB chunks: bit-exact against the
    oracle, and delivering the master that slidedp_stream_step just wrote gives exactly the BF16
    copy that step emitted."""
    wl = W.CONFIGS["qwen3_14b_layer_host"]
    n, R = wl.numel, wl.R
    hw = torch.empty(n, pin_memory=True)
    hw.copy_(W.master_weights(wl, device="cuda"))
    got, st = deliver(ctx, hw, W.chunk_elems(64), 3)
    assert np.array_equal(got, oracle.cast_master_to_bf16(hw.numpy()))
    assert st["chunks"] == 20 and st["gbs_h2d"] > 1.0
    hm, hv = torch.zeros(n, pin_memory=True), torch.zeros(n, pin_memory=True)
    dg = [W.rank_gradient(wl, r, step=1, device="cuda") for r in range(R)]
    dp = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()
    ctx.slidedp_stream_step(dg, n, hw, hm, hv, dp, W.chunk_elems(64), 3,
                            sd.HParams(inv_R=1.0 / R, max_norm=1.0, step=1, **wl.hparams))
    again, _ = deliver(ctx, hw, W.chunk_elems(16), 2)
    assert np.array_equal(again, parity.u16(dp))


def test_argument_errors(ctx, sd):
    out = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    pinned, pageable = torch.zeros(64, pin_memory=True), torch.zeros(64)

    def status(fn):
        with pytest.raises(sd.SlideDPError) as e:
            fn()
        return e.value.status

    call = ctx.slidedp_deliver_params
    assert status(lambda: call(pageable, 64, out, 8, 2)) == sd.ERR_NOT_PINNED
    assert status(lambda: call(pinned, 64, out, 12, 2)) == sd.ERR_INVALID_ARG
    assert status(lambda: call(pinned, 64, out, 8, 1)) == sd.ERR_INVALID_ARG
    assert status(lambda: call(pinned, -1, out, 8, 2)) == sd.ERR_INVALID_ARG
    assert status(lambda: call(pinned, 64, None, 8, 2)) == sd.ERR_INVALID_ARG
    assert status(lambda: call(pinned, 64, out[1:], 8, 2)) == sd.ERR_MISALIGNED
    tight = sd.slidedp_create(0, 2 * 16 * 4 - 1)
    try:
        assert status(lambda: tight.slidedp_deliver_params(pinned, 64, out, 16, 2)) == sd.ERR_BUDGET
    finally:
        tight.slidedp_destroy()
