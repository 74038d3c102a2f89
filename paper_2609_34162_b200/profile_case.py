"""A small, self-ending run of one kernel of libslidedp, for profiling under ncu.

  python -m paper_2609_34162_b200.profile_case --kernel update --params 50331648 --R 4 --launches 4

Inputs are larger than the 126 MB L2 (so DRAM counters mean something) but only a few GB.
Kernels: update (fused reduce + AdamW + BF16 emit), norm (tile sums + finish),
stream (host-resident step through pinned memory).
"""
from __future__ import annotations

import argparse

import torch

from . import slidedp as sd


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", choices=["update", "norm", "stream"], default="update")
    ap.add_argument("--params", type=int, default=48 << 20)
    ap.add_argument("--R", type=int, default=4)
    ap.add_argument("--launches", type=int, default=4)
    ap.add_argument("--clip", type=float, default=1.0)
    args = ap.parse_args()
    n, R = args.params, args.R
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev).manual_seed(0)
    grads = [(torch.randn(n, generator=g, device=dev) * 1e-3).to(torch.bfloat16) for _ in range(R)]
    w = torch.randn(n, generator=g, device=dev) * 0.02
    m = torch.randn(n, generator=g, device=dev) * 3e-4
    v = torch.randn(n, generator=g, device=dev).square() * 1e-7
    p = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    ctx = sd.slidedp_create(0, 0)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.launches + 1)]
    st = torch.cuda.current_stream()
    if args.kernel == "stream":
        hw, hm, hv = (torch.empty(n, pin_memory=True) for _ in range(3))
        hw.copy_(w); hm.copy_(m); hv.copy_(v)
    ctx.slidedp_grad_norm(grads, n, 1.0 / R, True)
    ctx.slidedp_grad_norm_finish(args.clip)
    for i in range(args.launches):
        ev[i].record(st)
        hp = sd.HParams(inv_R=1.0 / R, max_norm=args.clip, step=11 + i)
        if args.kernel == "update":
            ctx.slidedp_reduce_adamw_chunk(grads, n, w, m, v, p, hp)
        elif args.kernel == "norm":
            ctx.slidedp_grad_norm(grads, n, 1.0 / R, True)
            ctx.slidedp_grad_norm_finish(args.clip)
        else:
            ctx.slidedp_stream_step(grads, n, hw, hm, hv, p, 16 << 20, 3, hp, want_stats=False)
    ev[args.launches].record(st)
    torch.cuda.synchronize()
    ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.launches)]
    per = {"update": 26 + 2 * R, "norm": 2 * R, "stream": 24}[args.kernel]
    print(f"{args.kernel}: n={n} R={R} ms/launch={['%.4f' % x for x in ms]} "
          f"best {per * n / (min(ms) * 1e6):.1f} GB/s ({per} B/param)")
    ctx.slidedp_destroy()


if __name__ == "__main__":
    main()
