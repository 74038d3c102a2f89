"""The sharded multi-rank step with real process plumbing, on ONE GPU: two processes, both on
cuda:0, each holding its rank-local BF16 gradients; buffer handles exchanged over gloo, the
peers' buffers mapped with slidedp_ipc_open, every byte of data moved by libslidedp's own
kernels (paper Sec. 3.2 "Gradient return" / "Parameter dispatch").

The ranks' kernels never wait on one another on the device (there are no flags or spins in this
library); the ranks are ordered by host-side barriers only, so sharing one GPU is safe.

Checked: norm, coefficient, FP32 state and the BF16 copy held by EVERY rank are bit-identical to
the unsharded single-context step over the same R gradients, and within the benchmark's
tolerances of the CPU oracle, over two consecutive steps (clipped, then unclipped)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import parity
from paper_2609_34162_b200 import workloads as W

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def workload():
    return W.scaled(W.CONFIGS["qwen3_8b_layer"], 48)        # ~4 M parameters, ragged, 246 tiles


def hparams(sd_or_oracle, wl, t, R):
    return sd_or_oracle.HParams(inv_R=1.0 / R, max_norm=wl.max_norm if t == 1 else 0.0, step=t,
                                **wl.hparams)


def _rank_main(rank, port, out, WORLD, K_LOCAL):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import paper_2609_34162_b200.slidedp as sd
    from paper_2609_34162_b200.sharded import ShardedStep
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=WORLD)
    ctx = sd.slidedp_create(0, 0)
    try:
        wl = workload()
        n, R = wl.numel, WORLD * K_LOCAL
        grads = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(K_LOCAL)]
        param = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
        sh = ShardedStep(ctx, grads, n, param)
        lo, hi = sh.bounds[rank]
        w = W.master_weights(wl, device="cuda")[lo:hi].clone()
        m, v = torch.zeros(hi - lo, device="cuda"), torch.zeros(hi - lo, device="cuda")
        results = []
        for t in (1, 2):
            for i in range(K_LOCAL):          # global rank-major order: buffer i of rank r is K*r + i
                W.rank_gradient(wl, K_LOCAL * rank + i, step=t, device="cuda", out=grads[i])
            torch.cuda.synchronize()
            nc = sh.step(w, m, v, hparams(sd, wl, t, R))
            torch.cuda.synchronize()
            results.append({"nc": nc, "w": w.cpu().numpy(), "m": m.cpu().numpy(), "v": v.cpu().numpy(),
                            "p": parity.u16(param)})
        launches = ctx.slidedp_kernel_launches()
        sh.close()
        out.put((rank, {"bounds": sh.bounds, "steps": results, "launches": launches}))
    finally:
        ctx.slidedp_destroy()
        dist.destroy_process_group()


@pytest.mark.parametrize("WORLD,K_LOCAL", [(2, 2), (3, 1)])
def test_processes_sharing_one_gpu_match_the_unsharded_step_bit_for_bit(WORLD, K_LOCAL):
    """Two processes with two gradient buffers each (R = 4), and three processes with one each
    (R = 3: 1/R is not exact in FP32, and 246 tiles over 3 shards)."""
    import paper_2609_34162_b200.slidedp as sd
    mpc = mp.get_context("spawn")
    out = mpc.Queue()
    port = free_port()
    procs = [mpc.Process(target=_rank_main, args=(r, port, out, WORLD, K_LOCAL)) for r in range(WORLD)]
    for p in procs:
        p.start()
    try:
        res = dict(out.get(timeout=300) for _ in procs)
    finally:
        for p in procs:
            p.join(timeout=120)
    assert all(p.exitcode == 0 for p in procs)

    # the unsharded step on one context, and the oracle, over the same R gradients
    wl = workload()
    n, R = wl.numel, WORLD * K_LOCAL
    ctx = sd.slidedp_create(0, 0)
    try:
        dw = W.master_weights(wl, device="cuda")
        dm, dv = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        dp = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
        ow, om, ov = parity.f32(dw).copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
        op = np.zeros(n, np.uint16)
        bounds = res[0]["bounds"]
        assert all(res[r]["bounds"] == bounds for r in range(WORLD))
        assert bounds[0][0] == 0 and bounds[-1][1] == n
        for ti, t in enumerate((1, 2)):
            dg = [W.rank_gradient(wl, r, step=t, device="cuda") for r in range(R)]
            hp = hparams(sd, wl, t, R)
            nc = None
            if hp.max_norm > 0:
                ctx.slidedp_grad_norm(dg, n, hp.inv_R, True)
                nc = ctx.slidedp_grad_norm_finish(hp.max_norm, fetch=True)
            ctx.slidedp_reduce_adamw_chunk(dg, n, dw, dm, dv, dp, hp)
            torch.cuda.synchronize()
            norm_o, coef_o = oracle.step([parity.u16(g) for g in dg], ow, om, ov, op,
                                         hparams(oracle, wl, t, R), nthreads=8)
            for rank in range(WORLD):
                got = res[rank]["steps"][ti]
                lo, hi = bounds[rank]
                assert got["nc"] == nc                                  # same bits on every rank
                for name, dev in (("w", dw), ("m", dm), ("v", dv)):
                    assert np.array_equal(got[name], parity.f32(dev[lo:hi])), (t, rank, name)
                assert np.array_equal(got["p"], parity.u16(dp)), (t, rank)   # EVERY rank holds all shards
            # and the sharded result against the oracle, assembled from the shards
            for name, want in (("w", ow), ("m", om), ("v", ov)):
                whole = np.concatenate([res[r]["steps"][ti][name] for r in range(WORLD)])
                parity.assert_fp32_close(f"sharded step {t}/{name}", whole, want)
            parity.assert_bf16_close(f"sharded step {t}/param_bf16", res[1]["steps"][ti]["p"], op)
            if nc is not None:
                parity.assert_norm_close(nc[0], norm_o)
                assert abs(nc[1] - coef_o) <= 1e-6 * coef_o and coef_o < 1.0
        # per rank: tiles + scatter + finish + update at step 1, update at step 2
        assert [res[r]["launches"] for r in range(WORLD)] == [5] * WORLD
    finally:
        ctx.slidedp_destroy()


def test_ipc_argument_errors():
    import paper_2609_34162_b200.slidedp as sd
    ctx = sd.slidedp_create(0, 0)
    try:
        t = torch.zeros(1 << 16, dtype=torch.bfloat16, device="cuda")
        h = ctx.slidedp_ipc_export(t[1024:])
        assert len(h) == sd.IPC_HANDLE_BYTES
        base = ctx.slidedp_ipc_export(t)
        assert h[:64] == base[:64]                                   # same allocation,
        off = int.from_bytes(h[64:72], "little") - int.from_bytes(base[64:72], "little")
        assert off == 2048                                           # other offset
        with pytest.raises(sd.SlideDPError) as e:
            ctx.slidedp_ipc_export(0)
        assert e.value.status == sd.ERR_INVALID_ARG
        with pytest.raises(sd.SlideDPError) as e:
            ctx.slidedp_ipc_close(t.data_ptr())                      # never mapped by this context
        assert e.value.status == sd.ERR_INVALID_ARG
        with pytest.raises(ValueError):
            ctx.slidedp_ipc_open(b"short")
        # the broadcast update with ONE output is the plain update, bit for bit
        n = 40_003
        g = torch.Generator(device="cuda").manual_seed(3)
        dg = [(torch.randn(n, generator=g, device="cuda") * 1e-3).to(torch.bfloat16) for _ in range(3)]
        w = torch.randn(n, generator=g, device="cuda") * 0.02
        a = [w.clone(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")]
        b = [w.clone(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")]
        pa, pb, pc = (torch.zeros(n, dtype=torch.bfloat16, device="cuda") for _ in range(3))
        hp = sd.HParams(inv_R=1.0 / 3, step=2)
        ctx.slidedp_reduce_adamw_chunk(dg, n, *a, pa, hp)
        ctx.slidedp_reduce_adamw_chunk_bcast(dg, n, *b, [pb, pc], hp)
        torch.cuda.synchronize()
        assert all(torch.equal(x, y) for x, y in zip(a, b))
        assert torch.equal(pa, pb) and torch.equal(pa, pc)
        with pytest.raises(sd.SlideDPError) as e:
            ctx.slidedp_reduce_adamw_chunk_bcast(dg, n, *b, [], hp)
        assert e.value.status == sd.ERR_INVALID_ARG
    finally:
        ctx.slidedp_destroy()


@pytest.mark.parametrize("R,n,n_outs", [(1, 5, 3), (4, 4 * 128 * 3 + 3, 16), (16, 100_001, 2), (3, 8, 1)])
def test_broadcast_update_equals_the_plain_update_for_every_output(R, n, n_outs):
    """Every output of slidedp_reduce_adamw_chunk_bcast, ragged tail included, carries the bits
    of the plain update; the state does too; guard bands around every output stay intact."""
    import paper_2609_34162_b200.slidedp as sd
    ctx = sd.slidedp_create(0, 0)
    try:
        g = torch.Generator(device="cuda").manual_seed(100 * R + n_outs)
        dg = [(torch.randn(n, generator=g, device="cuda") * 1e-3).to(torch.bfloat16) for _ in range(R)]
        w = torch.randn(n, generator=g, device="cuda") * 0.02
        m = torch.randn(n, generator=g, device="cuda") * 3e-4
        v = torch.randn(n, generator=g, device="cuda").square() * 1e-7
        a, b = [w.clone(), m.clone(), v.clone()], [w.clone(), m.clone(), v.clone()]
        pa = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
        pad = 8                                             # keeps every output 16-byte aligned
        banded = [torch.full((n + 2 * pad,), -7.0, dtype=torch.bfloat16, device="cuda")
                  for _ in range(n_outs)]
        hp = sd.HParams(inv_R=1.0 / R, max_norm=0.02, step=9)
        ctx.slidedp_grad_norm(dg, n, 1.0 / R, True)
        ctx.slidedp_grad_norm_finish(0.02)
        ctx.slidedp_reduce_adamw_chunk(dg, n, *a, pa, hp)
        ctx.slidedp_reduce_adamw_chunk_bcast(dg, n, *b, [x[pad:] for x in banded], hp)
        torch.cuda.synchronize()
        assert all(torch.equal(x, y) for x, y in zip(a, b))
        for x in banded:
            assert torch.equal(x[pad:pad + n], pa)
            assert torch.all(x[:pad] == -7.0) and torch.all(x[pad + n:] == -7.0)
    finally:
        ctx.slidedp_destroy()
