#!/usr/bin/env python
"""Benchmark of the SlideDP reduce + AdamW hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W]            # libslidedp (CUDA)
  python bench.py --impl reference [--steps K] [--warmup W]      # the CPU oracle, as it stands

One "step" is one pass of the whole hot path over one Qwen3-8B-shaped decoder layer
(192,946,176 parameters, R = 4 BF16 rank gradients, step 11, clip 1.0): the global-norm
pass over all gradients, then the fused rank-reduce + AdamW + BF16-emit kernel.
`value` is whole-job G-params/s with everything resident in HBM; `e2e` is the same step
through slidedp_stream_step with the FP32 state in pinned HOST memory, host<->device copies
inside the timed region. With --gpus N every rank updates its own layer (independent
partitions, no data-path collective): weak scaling. Under a launcher (torchrun) the ranks are the
launcher's; without one, --gpus N > 1 starts the N ranks itself. Prints ONE JSON line on rank 0.

  python bench.py --sharded --gpus N          # one layer sharded over N ranks (peer-mapped buffers)
  python bench.py --report sweep              # the other configurations and the by-R table
  python bench.py --report kernel --kernel update --params 50331648 --R 4   # one small case for ncu
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "G-params/s per reduce+AdamW step"
UNIT = "G-params/s"
WORKLOAD = "qwen3_8b_layer"
HOST_WORKLOAD = "qwen3_14b_layer_host"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per parameter of the fused update kernel, from an
# ncu capture of a 50 M-parameter, R = 4 launch (a full-size launch is above the size an ncu
# capture should hold); scaled to a full launch by the parameter count.
NCU_TRAFFIC_BYTES_PER_PARAM = 32.96


def measured_peak_hbm():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while running."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()          # this exact child, nothing else
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            if self.thread:
                self.thread.join(timeout=2)
        sm, smax, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                sm.append(float(r[0])); smax = float(r[1])
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": smax, "reasons": [], "samples": 0}
        busy = [x for x in sm if x >= 0.5 * max(sm)]
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": smax,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------- reference arm
def run_reference(args):
    """Times the CPU oracle, unchanged, on the host cores: each step is the whole path (norm +
    update) over a bounded sample (the first 2^25 parameters) of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import numpy as np
    import torch

    import oracle
    from paper_2609_34162_b200 import workloads as W
    wl = W.CONFIGS[WORKLOAD]
    n = min(wl.numel, 1 << 25)
    cores = min(len(os.sched_getaffinity(0)), oracle.max_threads())

    def u16(t):
        return t.view(torch.int16).numpy().view(np.uint16)
    grads = [u16(W.rank_gradient(wl, r, step=wl.first_step)[:n].contiguous()) for r in range(wl.R)]
    w = W.master_weights(wl)[:n].contiguous().numpy()
    m, v, p = np.zeros(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.uint16)
    t = 1
    for _ in range(args.warmup):
        oracle.step(grads, w, m, v, p, oracle.HParams(inv_R=1.0 / wl.R, max_norm=wl.max_norm,
                                                      step=t, **wl.hparams), nthreads=cores)
        t += 1
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.step(grads, w, m, v, p, oracle.HParams(inv_R=1.0 / wl.R, max_norm=wl.max_norm,
                                                      step=t, **wl.hparams), nthreads=cores)
        t += 1
    dt = time.perf_counter() - t0
    value = n * args.steps / dt / 1e9
    sample = f"first {n} of {wl.numel} parameters per step, R={wl.R}, norm + update"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "params": wl.numel, "R": wl.R, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))
    return 0


class ResultChannel:
    """The contract is ONE JSON line on stdout. Libraries underneath (NCCL prints its version
    banner on stdout when a communicator is created) must not add to it: the real stdout is kept
    aside for the result line and file descriptor 1 points at stderr for everything else."""

    def __init__(self):
        sys.stdout.flush()
        self._fd = os.dup(1)
        os.dup2(2, 1)

    def emit(self, obj) -> None:
        sys.stdout.flush()
        with os.fdopen(os.dup(self._fd), "w") as out:
            out.write(json.dumps(obj) + "\n")

    def close(self) -> None:
        sys.stdout.flush()
        os.dup2(self._fd, 1)
        os.close(self._fd)


# ------------------------------------------------------------------ multi-rank plumbing
def layer_of_rank(rank: int) -> int:
    """Every rank owns a different layer (an independent partition of the model)."""
    return rank


def max_over_ranks(x: float, world: int, device="cuda") -> float:
    """The slowest rank's time: multi-GPU numbers are device times, max over ranks."""
    import torch.distributed as dist
    if world == 1 and not (dist.is_available() and dist.is_initialized()):
        return x
    import torch
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world: int, params_per_rank: int, steps: int, total_ms: float) -> float:
    """Whole-job G-params/s: the parameters all ranks updated over the slowest rank's time."""
    return world * params_per_rank * steps / (total_ms * 1e-3) / 1e9


# --------------------------------------------------------------------------------- CUDA arm
def run_cuda(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2609_34162_b200.slidedp as sd          # raises if libslidedp.so is missing
    from paper_2609_34162_b200 import workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available() or local >= torch.cuda.device_count():
        raise SystemExit("bench.py needs a CUDA device per rank: libslidedp has no CPU path "
                         "(use --impl reference for the CPU oracle)")
    channel = ResultChannel()
    torch.cuda.set_device(local)
    # under a launcher (torchrun sets RANK and MASTER_ADDR) the process group is used even for
    # one rank, so that the N = 1 run exercises the same barrier / reduction code as N > 1
    grouped = world > 1 or ("RANK" in os.environ and "MASTER_ADDR" in os.environ)
    if grouped:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if grouped:
            dist.barrier()
        torch.cuda.synchronize()

    wl = W.CONFIGS[WORKLOAD]
    n, R = wl.numel, wl.R
    layer = layer_of_rank(rank)
    ctx = sd.slidedp_create(local, 0)
    stream = torch.cuda.current_stream()
    dev = torch.device("cuda", local)

    # ---- inputs, resident in HBM: R gradients of the measured step, FP32 state, BF16 out
    t_meas = wl.first_step
    grads = [W.rank_gradient(wl, r, step=t_meas, layer=layer, device=dev) for r in range(R)]
    w = W.master_weights(wl, layer=layer, device=dev)
    m = torch.zeros(n, device=dev)
    v = torch.zeros(n, device=dev)
    p = torch.zeros(n, dtype=torch.bfloat16, device=dev)

    def hp(t):
        return sd.HParams(inv_R=1.0 / R, max_norm=wl.max_norm, step=t, **wl.hparams)

    def device_step(t, ev=None):
        if ev: ev[0].record(stream)
        ctx.slidedp_grad_norm(grads, n, 1.0 / R, True)
        ctx.slidedp_grad_norm_finish(wl.max_norm)
        if ev: ev[1].record(stream)
        ctx.slidedp_reduce_adamw_chunk(grads, n, w, m, v, p, hp(t))
        if ev: ev[2].record(stream)

    # moments pre-warmed by the seeded steps that precede the measured one (timing only: the
    # parity tests pre-warm with the oracle); fresh gradients each pre-warm step
    tmp = [torch.empty(n, dtype=torch.bfloat16, device=dev) for _ in range(R)]
    keep = grads
    for t in range(1, wl.prewarm_steps + 1):
        for r in range(R):
            W.rank_gradient(wl, r, step=t, layer=layer, device=dev, out=tmp[r])
        grads = tmp
        device_step(t)
    grads = keep
    del tmp
    torch.cuda.synchronize()
    torch.cuda.empty_cache()

    for i in range(max(args.warmup, 3)):
        device_step(t_meas + i)
    t_next = t_meas + max(args.warmup, 3)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = ctx.slidedp_kernel_launches()
    barrier()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record(stream)
    for i in range(args.steps):
        device_step(t_next + i, events[i])
    stop.record(stream)
    barrier()
    launches = ctx.slidedp_kernel_launches() - launches0
    total_ms = max_over_ranks(start.elapsed_time(stop), world)
    norm_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in events)
    upd_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in events)
    upd_best = min(e[1].elapsed_time(e[2]) for e in events)
    t_next += args.steps

    # the same loads and stores with no arithmetic, on the same buffers (state unchanged): what
    # this access mix can reach on this device, beside the plain-copy peak
    mix_gbs = ctx.slidedp_hbm_mix_probe(grads, n, w, m, v, p, 8)

    ms_per_step = total_ms / args.steps
    value = job_value(world, n, args.steps, total_ms)
    peak, peak_kind = measured_peak_hbm()
    upd_bytes = (26 + 2 * R) * n
    achieved = upd_bytes / (upd_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "reduce_adamw_kernel<R=4>", "achieved": achieved,
                "peak": peak, "peak_source": f"of {peak_kind}", "unit": "GB/s",
                "frac": achieved / peak,
                "traffic": (NCU_TRAFFIC_BYTES_PER_PARAM * n
                            if NCU_TRAFFIC_BYTES_PER_PARAM is not None else None),
                "algorithmic_bytes_per_launch": upd_bytes, "ms_per_launch": upd_ms,
                "ms_per_launch_best": upd_best,
                "frac_of_nominal_8000": achieved / 8000.0,
                "access_mix_peak": mix_gbs, "frac_of_access_mix_peak": achieved / mix_gbs,
                "access_mix_peak_source": "slidedp_hbm_mix_probe in this run: the kernel's loads and "
                                          "stores with no arithmetic, same buffers, best of 8",
                "norm_pass": {"ms": norm_ms, "algorithmic_bytes": 2 * R * n,
                              "achieved": 2 * R * n / (norm_ms * 1e-3) / 1e9,
                              "frac": 2 * R * n / (norm_ms * 1e-3) / 1e9 / peak}}

    # ---- e2e: the same step with the FP32 state in pinned host memory ------------------
    ce = W.chunk_elems(16)      # a 12-chunk layer at 64 MiB would spend 8 % draining the last chunk
    hw = torch.empty(n, pin_memory=True); hm = torch.empty(n, pin_memory=True)
    hv = torch.empty(n, pin_memory=True)
    hw.copy_(w); hm.copy_(m); hv.copy_(v)
    torch.cuda.synchronize()
    for i in range(2):
        ctx.slidedp_stream_step(grads, n, hw, hm, hv, p, ce, 3, hp(t_next + i), want_stats=False)
    t_next += 2
    e2e_steps = max(1, min(args.steps, 10))
    barrier()
    e2e_ms, wall0, last, per_step = 0.0, time.perf_counter(), None, []
    for i in range(e2e_steps):
        last = ctx.slidedp_stream_step(grads, n, hw, hm, hv, p, ce, 3, hp(t_next + i))
        e2e_ms += last["ms_total"]
        per_step.append(last["ms_total"])
    wall = time.perf_counter() - wall0
    barrier()
    t_next += e2e_steps
    e2e_ms = max_over_ranks(e2e_ms, world)
    e2e = {"value": job_value(world, n, e2e_steps, e2e_ms), "unit": UNIT,
           "h2d_bytes_per_step": 12 * n, "d2h_bytes_per_step": 12 * n + 32,
           "ms_per_step": e2e_ms / e2e_steps, "wall_ms_per_step": wall / e2e_steps * 1e3,
           "ms_per_step_median": statistics.median(per_step), "ms_per_step_best": min(per_step),
           "steps": e2e_steps, "chunk_mib": 16, "nbuf": 3,
           "note": "FP32 master/m/v in pinned host memory, copied H2D and back D2H every step; "
                   "gradients and the BF16 copy stay on the device where backward/forward use them",
           "link_gbs_h2d": last["gbs_h2d"], "link_gbs_d2h": last["gbs_d2h"]}
    del hw, hm, hv
    # the sampler ran through the device-timed region and the e2e region
    clocks = sampler.stop() if rank == 0 else None

    out = None
    if rank == 0:
        # ---- host-resident configuration proper + the measured host-link roofline ------
        host = None
        try:
            host = host_resident_report(ctx, sd, W, torch, dev)
        except Exception as exc:                       # report, never hide
            host = {"error": repr(exc)}
        try:
            route = cpu_route_report(ctx, sd, W, torch, dev)
        except Exception as exc:
            route = {"error": repr(exc)}
        # both delivery routes side by side where the host-resident configuration is reported
        if isinstance(host, dict) and isinstance(route, dict) and "delivery" in host and "delivery" in route:
            host["delivery"]["routes"] = {
                "fp32_h2d_gpu_cast (slidedp_deliver_params)": route["delivery"]["fp32_h2d_gpu_cast"],
                "cpu_cast_bf16_h2d (the paper's route, baseline/cpu_route)": route["delivery"]["cpu_cast_bf16_h2d"]}
        cpu = cpu_baseline(W, torch, np, wl, grads, layer)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "params_per_gpu": n, "R": R, "step": t_meas,
                       "clip_max_norm": wl.max_norm, "mode": "device-resident",
                       "parallelism": f"{world} independent layer(s), one per GPU, no collective",
                       "l2": "inputs (8.1 GB touched per step) exceed the 126 MB L2"},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches,
            "clocks": clocks, "host_resident": host, "cpu_route": route,
            "host_placement": host_placement(torch, local),
        }
    ctx.slidedp_destroy()
    if grouped:
        dist.barrier()
        dist.destroy_process_group()
    if out is not None:
        channel.emit(out)
    channel.close()
    return 0


def run_sharded(args):
    """`--sharded`: ONE Qwen3-8B-shaped layer updated by all ranks together. Every rank holds its
    own rank-local BF16 gradient of the whole layer (R = number of ranks), owns 1/N of the FP32
    state, reads its slice of every peer's gradient through mapped pointers inside the norm and
    update kernels, and stores its shard of the BF16 copy into every rank's parameter buffer
    (paper_2609_34162_b200/sharded.py). Strong scaling: the layer is fixed, the ranks split it.
    The timed region includes the three host-side barriers of each step."""
    import torch
    import torch.distributed as dist

    import paper_2609_34162_b200.slidedp as sd
    from paper_2609_34162_b200 import workloads as W
    from paper_2609_34162_b200.sharded import ShardedStep

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available() or local >= torch.cuda.device_count():
        raise SystemExit("bench.py --sharded needs one CUDA device per rank: libslidedp has no CPU path")
    channel = ResultChannel()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if "MASTER_ADDR" not in os.environ:
        os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    wl = W.CONFIGS[WORKLOAD]
    n, R = wl.numel, world
    ctx = sd.slidedp_create(local, 0)
    grad = W.rank_gradient(wl, rank, step=wl.first_step, device=dev)
    param = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    sh = ShardedStep(ctx, [grad], n, param)
    lo, hi = sh.bounds[rank]
    w = W.master_weights(wl, device=dev)[lo:hi].clone()
    m, v = torch.zeros(hi - lo, device=dev), torch.zeros(hi - lo, device=dev)
    stream = torch.cuda.current_stream()

    def hp(t):
        return sd.HParams(inv_R=1.0 / R, max_norm=wl.max_norm, step=t, **wl.hparams)

    t = 1
    for _ in range(max(args.warmup, 3)):
        sh.step(w, m, v, hp(t), stream)
        t += 1
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = ctx.slidedp_kernel_launches()
    dist.barrier(); torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record(stream)
    for _ in range(args.steps):
        sh.step(w, m, v, hp(t), stream)
        t += 1
    stop.record(stream)
    dist.barrier(); torch.cuda.synchronize()
    launches = ctx.slidedp_kernel_launches() - launches0
    total_ms = max_over_ranks(start.elapsed_time(stop), world)
    clocks = sampler.stop() if rank == 0 else None
    sh.close()
    ctx.slidedp_destroy()
    if rank == 0:
        # per parameter and rank: (12 + 14)/N state bytes locally, 2 (R - 1)/N gradient bytes
        # and 2 (N - 1)/N parameter bytes over the GPU interconnect, plus the norm's re-read
        channel.emit({
            "metric": METRIC, "value": n * args.steps / (total_ms * 1e-3) / 1e9, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "mode": "sharded",
            "config": {"workload": WORKLOAD, "params": n, "R": R, "clip_max_norm": wl.max_norm,
                       "parallelism": f"one layer sharded over {world} rank(s): peer-mapped gradient "
                                      "reads, BF16 copy stored to every rank, host barriers"},
            "gpu_launches": launches, "clocks": clocks,
            "interconnect_bytes_per_rank_per_step": (4 * (R - 1) + 2 * (world - 1)) * (hi - lo)})
    dist.barrier()
    dist.destroy_process_group()
    channel.close()
    return 0


def run_sweep(args):
    """`--report sweep`: one JSON line with the other benchmark configurations on one GPU:
    the tiny chunk (L2-resident and rotating over buffer sets larger than L2), the chunk-size
    sweep of the Qwen2.5-72B-shaped layer (16/64/256 MiB, 2 and 3 slots) and the eight-layer,
    R = 8 host-resident step with one global norm. Not the contract line; for the tables."""
    import torch

    import paper_2609_34162_b200.slidedp as sd
    from paper_2609_34162_b200 import workloads as W
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    ctx = sd.slidedp_create(0, 0)
    st = torch.cuda.current_stream()
    peak, peak_kind = measured_peak_hbm()
    out = {"report": "sweep", "hbm_peak_gbs": peak, "hbm_peak_source": peak_kind}

    def hp(wl, t):
        return sd.HParams(inv_R=1.0 / wl.R, max_norm=wl.max_norm, step=t, **wl.hparams)

    # ---- tiny chunk: 31.5 MB of traffic fits the 126 MB L2, so time it both ways
    wl = W.CONFIGS["tiny"]
    n, R, sets = wl.numel, wl.R, 16
    bufs = []
    for i in range(sets):
        g = [W.rank_gradient(wl, r, step=1 + i, device=dev) for r in range(R)]
        bufs.append((g, W.master_weights(wl, device=dev), torch.zeros(n, device=dev),
                     torch.zeros(n, device=dev), torch.zeros(n, dtype=torch.bfloat16, device=dev)))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    res = {}
    reps = sets * 20
    for name, pick in (("l2_resident", lambda i: 0), ("rotating_16_sets", lambda i: i % sets)):
        for i in range(sets * 2):
            g, w, m, v, p = bufs[pick(i)]
            ctx.slidedp_reduce_adamw_chunk(g, n, w, m, v, p, hp(wl, 1))
        torch.cuda.synchronize()
        # a 5 us kernel is launch-bound from Python: capture the launches in a CUDA graph
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(reps):
                g, w, m, v, p = bufs[pick(i)]
                ctx.slidedp_reduce_adamw_chunk(g, n, w, m, v, p, hp(wl, 1))
        graph.replay()
        torch.cuda.synchronize()
        ev[0].record(st)
        graph.replay()
        ev[1].record(st)
        torch.cuda.synchronize()
        us = ev[0].elapsed_time(ev[1]) / reps * 1e3
        res[name] = {"us_per_launch": us, "g_params_per_s": n / us / 1e3,
                     "algorithmic_gbs": (26 + 2 * R) * n / us / 1e3}
        del graph
    res["note"] = ("320 launches replayed from one CUDA graph; the rotating case touches 16 x 31.5 MB = 504 MB "
                   "(4 x L2) between reuses, the resident case is a cache number, not HBM")
    out["tiny"] = res
    del bufs

    # ---- by rank count: update kernel, norm pass, rank reduction alone (100 M parameters)
    n = 100_000_000
    gen = torch.Generator(device=dev).manual_seed(11)
    pool = [(torch.randn(n, generator=gen, device=dev) * 1e-3).to(torch.bfloat16) for _ in range(16)]
    w = torch.randn(n, generator=gen, device=dev) * 0.02
    m = torch.randn(n, generator=gen, device=dev) * 3e-4
    v = torch.randn(n, generator=gen, device=dev).square() * 1e-7
    p = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    by_R = []
    reps = 12
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]

    def timed(fn):
        for _ in range(3):
            fn()
        for i in range(reps):
            evs[i].record(st)
            fn()
        evs[reps].record(st)
        torch.cuda.synchronize()
        ms = sorted(evs[i].elapsed_time(evs[i + 1]) for i in range(reps))
        return statistics.median(ms), ms[0]

    for R in (1, 2, 3, 4, 8, 16):
        g = pool[:R]
        h = sd.HParams(inv_R=1.0 / R, max_norm=1.0, step=11)
        ctx.slidedp_grad_norm(g, n, 1.0 / R, True)
        ctx.slidedp_grad_norm_finish(1.0)

        def norm_pass():
            ctx.slidedp_grad_norm(g, n, 1.0 / R, True)
            ctx.slidedp_grad_norm_finish(1.0)
        row = {"R": R}
        for name, fn, per in (("update", lambda: ctx.slidedp_reduce_adamw_chunk(g, n, w, m, v, p, h), 26 + 2 * R),
                              ("norm", norm_pass, 2 * R),
                              ("reduce_mean_bf16", lambda: ctx.slidedp_reduce_mean_bf16(g, n, 1.0 / R, p), 2 * R + 2)):
            med, best = timed(fn)
            row[name] = {"ms": med, "ms_best": best, "bytes_per_param": per,
                         "gbs": per * n / (med * 1e6), "frac_of_measured_peak": per * n / (med * 1e6) / peak}
        by_R.append(row)
    # the sharded step's update with its BF16 copy stored to G buffers (all local here: the HBM
    # cost of the stores alone; on real ranks G - 1 of them cross the GPU interconnect)
    g4 = pool[:4]
    h4 = sd.HParams(inv_R=0.25, max_norm=1.0, step=11)
    extra = [torch.zeros(n, dtype=torch.bfloat16, device=dev) for _ in range(7)]
    bcast = []
    for G in (1, 2, 4, 8):
        outs = [p] + extra[:G - 1]
        med, best = timed(lambda: ctx.slidedp_reduce_adamw_chunk_bcast(g4, n, w, m, v, outs, h4))
        per = 26 + 2 * 4 + 2 * (G - 1)
        bcast.append({"outputs": G, "ms": med, "bytes_per_param": per, "gbs": per * n / (med * 1e6),
                      "frac_of_measured_peak": per * n / (med * 1e6) / peak})
    out["broadcast_update_R4"] = {"params": n, "rows": bcast,
                                  "note": "all outputs in local HBM; one GPU cannot show the interconnect"}
    del extra
    out["by_rank_count"] = {"params": n, "timing": f"median of {reps} launches, CUDA events, inputs >> L2",
                            "rows": by_R}
    del pool, w, m, v, p
    torch.cuda.empty_cache()

    def pinned_state(n):
        return [torch.empty(n, pin_memory=True) for _ in range(3)]

    # ---- chunk-size sweep on the Qwen2.5-72B-shaped layer
    wl = W.CONFIGS["qwen25_72b_layer_host"]
    n, R = wl.numel, wl.R
    grads = [W.rank_gradient(wl, r, step=wl.first_step, device=dev) for r in range(R)]
    p = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    hw, hm, hv = pinned_state(n)
    hw.copy_(W.master_weights(wl, device=dev)); hm.zero_(); hv.zero_()
    dbuf = torch.empty(2 << 28, dtype=torch.float32, device=dev)
    probes = {}
    for mib in (16, 64, 256):
        probes[str(mib)] = ctx.slidedp_link_probe(hm, hv, dbuf[:1 << 28], dbuf[1 << 28:],
                                                  1 << 30, mib << 20, 3)
    del dbuf
    hm.zero_(); hv.zero_()
    sweep, t = [], 1
    for mib in wl.chunk_mib:
        for nbuf in (2, 3):
            runs = []
            for i in range(4):
                r_ = ctx.slidedp_stream_step(grads, n, hw, hm, hv, p, W.chunk_elems(mib), nbuf,
                                             hp(wl, t))
                t += 1
                if i >= 1:
                    runs.append(r_)
            ms = statistics.mean(r_["ms_total"] for r_ in runs)
            pr = probes[str(mib)]
            bound = max(12.0 * n / (pr["h2d_bidir"] * 1e6), 12.0 * n / (pr["d2h_bidir"] * 1e6))
            lanes = {k: statistics.mean(r_[k] for r_ in runs)
                     for k in ("ms_norm", "ms_h2d", "ms_kernel", "ms_d2h")}
            # the paper's dependency model fed with rates measured in this run
            lo_ms, pred_ms = sd.slidedp_model_stream_step(
                n, R, W.chunk_elems(mib), nbuf, pr["h2d_bidir"], pr["d2h_bidir"],
                n / (lanes["ms_kernel"] * 1e6), 2.0 * R * n / (lanes["ms_norm"] * 1e6), 3.0)
            sweep.append({"chunk_mib": mib, "nbuf": nbuf, "ms_per_step": ms,
                          "model_lower_bound_ms": lo_ms, "model_predicted_ms": pred_ms,
                          "g_params_per_s": n / ms / 1e6,
                          "link_gbs_each_way": 12.0 * n / (ms * 1e6), "frac_of_link": bound / ms,
                          "lanes_ms": lanes})
    out["qwen25_72b_layer_host"] = {"params": n, "R": R, "link_probe_gbs": probes, "sweep": sweep}
    del grads, p, hw, hm, hv
    torch.cuda.empty_cache()

    # ---- eight layers, R = 8: global norm over all layers, then every layer streamed
    wl = W.CONFIGS["qwen3_14b_8layers_host"]
    L, R, nl = wl.layers, wl.R, wl.layer_numel
    grads = [[W.rank_gradient(wl, r, step=1, layer=l, device=dev) for r in range(R)]
             for l in range(L)]
    ps = [torch.zeros(nl, dtype=torch.bfloat16, device=dev) for _ in range(L)]
    state = []
    for l in range(L):
        hw, hm, hv = pinned_state(nl)
        hw.copy_(W.master_weights(wl, layer=l, device=dev)); hm.zero_(); hv.zero_()
        state.append((hw, hm, hv))
    ce = W.chunk_elems(64)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_ms, norm_ms = [], []
    for t in range(1, wl.steps + 1):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e0.record(st)
        for l in range(L):
            ctx.slidedp_grad_norm(grads[l], nl, 1.0 / R, l == 0)
        ctx.slidedp_grad_norm_finish(wl.max_norm)
        e1.record(st)
        torch.cuda.synchronize()
        for l in range(L):
            ctx.slidedp_stream_step(grads[l], nl, *state[l], ps[l], ce, 3, hp(wl, t),
                                    norm_ready=True, want_stats=False)
        torch.cuda.synchronize()
        step_ms.append((time.perf_counter() - t0) * 1e3)
        norm_ms.append(e0.elapsed_time(e1))
    ms = statistics.mean(step_ms[2:])
    nm = statistics.mean(norm_ms[2:])
    # the same step with the layers enqueued back to back (one wait at the end)
    async_ms = []
    for t in range(wl.steps + 1, wl.steps + 6):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for l in range(L):
            ctx.slidedp_grad_norm(grads[l], nl, 1.0 / R, l == 0)
        ctx.slidedp_grad_norm_finish(wl.max_norm)
        torch.cuda.synchronize()
        for l in range(L):
            ctx.slidedp_stream_step_async(grads[l], nl, *state[l], ps[l], ce, 3, hp(wl, t),
                                          norm_ready=True)
        ctx.slidedp_stream_wait()
        async_ms.append((time.perf_counter() - t0) * 1e3)
    ams = statistics.mean(async_ms[1:])
    # and as ONE call: norm over all layers + every layer streamed (slidedp_stream_layers)
    one_call = []
    for t in range(wl.steps + 6, wl.steps + 11):
        torch.cuda.synchronize()
        one_call.append(ctx.slidedp_stream_layers(
            [(grads[l], nl, *state[l], ps[l]) for l in range(L)], ce, 3, hp(wl, t)))
    oms = statistics.mean(r_["ms_total"] for r_ in one_call[1:])
    out["qwen3_14b_8layers_host"] = {
        "async_layers": {"ms_per_step": ams, "g_params_per_s": wl.numel / ams / 1e6,
                         "link_gbs_each_way": 12.0 * wl.numel / (ams * 1e6)},
        "one_call_stream_layers": {"ms_per_step": oms, "g_params_per_s": wl.numel / oms / 1e6,
                                   "link_gbs_each_way": 12.0 * wl.numel / (oms * 1e6),
                                   "ms_norm": statistics.mean(r_["ms_norm"] for r_ in one_call[1:]),
                                   "timing": "CUDA events inside the call, norm pass included"},
        "params": wl.numel, "R": R, "layers": L, "steps": wl.steps, "chunk_mib": 64, "nbuf": 3,
        "ms_per_step": ms, "g_params_per_s": wl.numel / ms / 1e6,
        "link_gbs_each_way": 12.0 * wl.numel / (ms * 1e6),
        "norm_pass_ms": nm, "norm_pass_gbs": 2.0 * R * wl.numel / (nm * 1e6),
        "norm_pass_frac_of_hbm": 2.0 * R * wl.numel / (nm * 1e6) / peak,
        "timing": "host wall clock per step bracketed by synchronize (the calls are synchronous)"}
    ctx.slidedp_destroy()
    print(json.dumps(out))
    return 0


def host_resident_report(ctx, sd, W, torch, dev):
    """Qwen3-14B-shaped layer with pinned host state, 64 MiB chunks, 3 slots, against the
    pinned-copy bandwidth measured in the same run."""
    wl = W.CONFIGS[HOST_WORKLOAD]
    n, R = wl.numel, wl.R
    grads = [W.rank_gradient(wl, r, step=wl.first_step, device=dev) for r in range(R)]
    p = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    hw = torch.empty(n, pin_memory=True); hm = torch.empty(n, pin_memory=True)
    hv = torch.empty(n, pin_memory=True)
    hw.copy_(W.master_weights(wl, device=dev)); hm.zero_(); hv.zero_()
    # link probe on 1 GiB per direction in 64 MiB copies, reusing hw/hm as the pinned buffers
    dbuf = torch.empty(2 << 28, dtype=torch.float32, device=dev)
    probe = ctx.slidedp_link_probe(hw, hm, dbuf[:1 << 28], dbuf[1 << 28:], 1 << 30, 64 << 20, 3)
    del dbuf
    hw.copy_(W.master_weights(wl, device=dev)); hm.zero_()
    torch.cuda.synchronize()
    ce = W.chunk_elems(64)
    runs = []
    for i in range(5):
        st = ctx.slidedp_stream_step(grads, n, hw, hm, hv, p, ce, 3,
                                     sd.HParams(inv_R=1.0 / R, max_norm=wl.max_norm, step=1 + i,
                                                **wl.hparams))
        if i >= 2:
            runs.append(st)
    ms = statistics.mean(r["ms_total"] for r in runs)
    link_bytes = 12.0 * n
    bound_ms = max(link_bytes / (probe["h2d_bidir"] * 1e6), link_bytes / (probe["d2h_bidir"] * 1e6))
    # parameter delivery (the step before the path): BF16 copy of the pinned FP32 master
    dl = [ctx.slidedp_deliver_params(hw, n, p, ce, 3) for _ in range(4)][1:]
    dl_ms = statistics.mean(r["ms_total"] for r in dl)
    delivery = {"ms": dl_ms, "g_params_per_s": n / dl_ms / 1e6, "h2d_bytes": 4 * n,
                "roofline": {"bound": "host-link", "unit": "GB/s", "achieved": 4.0 * n / (dl_ms * 1e6),
                             "peak": probe["h2d"], "frac": 4.0 * n / (dl_ms * 1e6) / probe["h2d"],
                             "peak_source": "pinned-copy probe in this run, H2D alone"}}
    return {"workload": HOST_WORKLOAD, "delivery": delivery, "params": n, "R": R, "chunk_mib": 64, "nbuf": 3,
            "value": n / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
            "link_probe_gbs": probe,
            "link_gbs_effective_each_way": link_bytes / (ms * 1e6),
            "roofline": {"bound": "host-link", "unit": "GB/s",
                         "achieved": link_bytes / (ms * 1e6),
                         "peak": min(probe["h2d_bidir"], probe["d2h_bidir"]),
                         "frac": bound_ms / ms,
                         "peak_source": "pinned-copy probe in this run, both directions at once"},
            "lanes_ms": {k: statistics.mean(r[k] for r in runs)
                         for k in ("ms_norm", "ms_h2d", "ms_kernel", "ms_d2h")}}


def cpu_route_report(ctx, sd, W, torch, dev):
    """The paper's OWN data path on this machine, beside the fused GPU path (baseline/cpu_route; not
    the product): the Qwen3-14B-shaped layer of the host-resident configuration, gradient return
    by GPU reduction (ONE BF16 gradient, G_l bytes D2H, produced by slidedp_reduce_mean_bf16) or
    by CPU reduction (R G_l bytes D2H, summed on the host), the multi-threaded FP32 CPU AdamW per
    64 MiB-of-FP32 chunk as the copies land, the CPU cast with streaming stores, and the BF16
    delivery sent once ("sharded") or R times ("replicated"): the four datapaths of the paper's
    host-traffic table (Sec. 2.4), with q_l = 1."""
    import numpy as np

    from baseline import cpu_route as cr
    wl = W.CONFIGS[HOST_WORKLOAD]
    n, R = wl.numel, wl.R
    threads = min(len(os.sched_getaffinity(0)), cr.max_threads())
    grads = [W.rank_gradient(wl, r, step=wl.first_step, device=dev) for r in range(R)]
    mean = torch.empty(n, dtype=torch.bfloat16, device=dev)
    outs = [torch.empty(n, dtype=torch.bfloat16, device=dev) for _ in range(R)]
    stage = [torch.empty(n, dtype=torch.int16, pin_memory=True) for _ in range(R)]
    pstage = torch.empty(n, dtype=torch.int16, pin_memory=True)
    w = W.master_weights(wl, device=dev).cpu().numpy()
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    ce = W.chunk_elems(64)
    # the clip coefficient comes from the GPU norm pass in every route (the paper has no clipping)
    ctx.slidedp_grad_norm(grads, n, 1.0 / R, True)
    _, coef = ctx.slidedp_grad_norm_finish(wl.max_norm, fetch=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    st = torch.cuda.current_stream()
    rows, t = [], 1
    for reduction in ("gpu", "cpu"):
        for delivery, copies in (("sharded", 1), ("replicated", R)):
            runs = []
            for i in range(4):
                red_ms = 0.0
                if reduction == "gpu":
                    e0.record(st)
                    ctx.slidedp_reduce_mean_bf16(grads, n, 1.0 / R, mean)
                    e1.record(st)
                    torch.cuda.synchronize()
                    red_ms = e0.elapsed_time(e1)
                    src, inv = [mean.data_ptr()], 1.0
                else:
                    src, inv = [g.data_ptr() for g in grads], 1.0 / R
                hp = cr.HParams(inv_R=inv, clip_coef=coef, step=t, **wl.hparams)
                r_ = cr.step(src, n, stage[:len(src)], w, m, v, pstage,
                             [o.data_ptr() for o in outs[:copies]], ce, hp, threads)
                t += 1
                r_["ms_reduce_kernel"] = red_ms
                if i >= 1:
                    runs.append(r_)
            ms = statistics.mean(r_["ms_total"] + r_["ms_reduce_kernel"] for r_ in runs)
            upd = statistics.mean(r_["ms_update"] for r_ in runs)
            host_bytes = (2 * len(src) + 12 + 14) * n          # gradients + state read, state + BF16 written
            rows.append({"delivery": delivery, "reduction": reduction + " reduction",
                         "h2d_bytes": runs[0]["h2d_bytes"], "d2h_bytes": runs[0]["d2h_bytes"],
                         "ms_per_step": ms, "g_params_per_s": n / ms / 1e6,
                         "ms_cpu_update": upd, "cpu_update_gbs": host_bytes / (upd * 1e6),
                         "ms_waiting_for_d2h": statistics.mean(r_["ms_wait_d2h"] for r_ in runs),
                         "ms_d2h_lane": statistics.mean(r_["ms_d2h_lane"] for r_ in runs),
                         "ms_h2d_lane": statistics.mean(r_["ms_h2d_lane"] for r_ in runs),
                         "ms_gpu_reduce_kernel": statistics.mean(r_["ms_reduce_kernel"] for r_ in runs)})
    # delivery alone, both ways: CPU cast + 2 B/param H2D against FP32 H2D + GPU cast
    hw = torch.empty(n, pin_memory=True)
    hw.copy_(torch.from_numpy(w))
    cpu_runs = [cr.deliver(w, n, pstage, outs[0].data_ptr(), ce, threads) for _ in range(4)][1:]
    gpu_runs = [ctx.slidedp_deliver_params(hw, n, outs[0], ce, 3) for _ in range(4)][1:]
    cpu_ms = statistics.mean(r_["ms_total"] for r_ in cpu_runs)
    gpu_ms = statistics.mean(r_["ms_total"] for r_ in gpu_runs)
    delivery = {"params": n, "chunk_mib": 64,
                "cpu_cast_bf16_h2d": {"ms": cpu_ms, "link_bytes": 2 * n, "link_gbs": 2.0 * n / (cpu_ms * 1e6),
                                      "ms_inside_cast": statistics.mean(r_["ms_update"] for r_ in cpu_runs),
                                      "host_cores": threads, "isa": cr.isa(),
                                      "host_dram_bytes": 6 * n},
                "fp32_h2d_gpu_cast": {"ms": gpu_ms, "link_bytes": 4 * n, "link_gbs": 4.0 * n / (gpu_ms * 1e6),
                                      "host_cores": 0, "host_dram_bytes": 4 * n}}
    return {"workload": HOST_WORKLOAD, "params": n, "R": R, "chunk_mib": 64, "host_cores": threads,
            "isa": cr.isa(), "arithmetic": "FP32 (vectorised CPU AdamW), BF16 gradients",
            "clip_coef": coef, "datapaths": rows, "delivery": delivery,
            "note": "baseline: the paper's route on this box; the product's host-resident step is "
                    "host_resident.value"}


def host_placement(torch, local: int):
    """Where the pinned state and the GPU sit (the paper keeps pinned buffers and the update
    worker on a fixed NUMA node, Sec. 3.2 "Routes and physical resources"): NUMA nodes visible to
    this process, the GPU's node as sysfs reports it, and the CPUs this process may run on."""
    def read(path):
        try:
            with open(path) as f:
                return f.read().strip()
        except OSError:
            return None
    nodes = [d for d in os.listdir("/sys/devices/system/node")
             if d.startswith("node") and d[4:].isdigit()] if os.path.isdir("/sys/devices/system/node") else []
    bdf = None
    try:
        bdf = torch.cuda.get_device_properties(local).pci_bus_id
        bdf = f"{torch.cuda.get_device_properties(local).pci_domain_id:04x}:{bdf:02x}:" \
              f"{torch.cuda.get_device_properties(local).pci_device_id:02x}.0"
    except Exception:
        bdf = None
    mems = None
    status = read("/proc/self/status") or ""
    for line in status.splitlines():
        if line.startswith("Mems_allowed_list"):
            mems = line.split(":", 1)[1].strip()
    return {"numa_nodes": len(nodes), "mems_allowed": mems,
            "gpu_numa_node": read(f"/sys/bus/pci/devices/{bdf}/numa_node") if bdf else None,
            "cpus": len(os.sched_getaffinity(0))}


def cpu_baseline(W, torch, np, wl, grads, layer):
    """The oracle as it stands, one whole step (norm + update) of the same layer on the host
    cores of this machine."""
    import oracle
    cores = min(len(os.sched_getaffinity(0)), oracle.max_threads())
    n = wl.numel if cores >= 4 else wl.numel // 4
    hg = [g[:n].cpu().view(torch.int16).numpy().view(np.uint16) for g in grads]
    w = W.master_weights(wl, layer=layer)[:n].contiguous().numpy()
    m, v, p = np.zeros(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.uint16)
    kw = dict(inv_R=1.0 / wl.R, max_norm=wl.max_norm, **wl.hparams)
    oracle.step([g[:1 << 20] for g in hg], w[:1 << 20], m[:1 << 20], v[:1 << 20], p[:1 << 20],
                oracle.HParams(step=1, **kw), nthreads=cores)           # warm the threads
    t0 = time.perf_counter()
    oracle.step(hg, w, m, v, p, oracle.HParams(step=2, **kw), nthreads=cores)
    dt = time.perf_counter() - t0
    # the same oracle on ONE thread, on the first 2^24 parameters
    k = min(n, 1 << 24)
    t0 = time.perf_counter()
    oracle.step([g[:k] for g in hg], w[:k], m[:k], v[:k], p[:k], oracle.HParams(step=3, **kw),
                nthreads=1)
    dt1 = time.perf_counter() - t0
    return {"value": n / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"one whole step (norm + update) over {n} of {wl.numel} parameters, R={wl.R}",
            "seconds": dt, "single_thread_value": k / dt1 / 1e9,
            "single_thread_sample": f"one whole step over the first {k} parameters"}


def run_kernel_case(args):
    """`--report kernel`: a small, self-ending run of ONE kernel, for profiling under ncu
    (inputs larger than the 126 MB L2 so DRAM counters mean something, but about a GB):

      python bench.py --report kernel --kernel update --params 50331648 --R 4 --launches 4

    Kernels: update (fused reduce + AdamW + BF16 emit), norm (tile sums + finish), reduce (rank
    reduction alone), stream (host-resident step through pinned memory), deliver (FP32 H2D + BF16
    cast)."""
    import torch

    import paper_2609_34162_b200.slidedp as sd
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
    if args.kernel in ("stream", "deliver"):
        hw, hm, hv = (torch.empty(n, pin_memory=True) for _ in range(3))
        hw.copy_(w); hm.copy_(m); hv.copy_(v)
    ctx.slidedp_grad_norm(grads, n, 1.0 / R, True)
    ctx.slidedp_grad_norm_finish(args.clip)
    torch.cuda.synchronize()
    for i in range(args.launches):
        ev[i].record(st)
        hp = sd.HParams(inv_R=1.0 / R, max_norm=args.clip, step=11 + i)
        if args.kernel == "update":
            ctx.slidedp_reduce_adamw_chunk(grads, n, w, m, v, p, hp)
        elif args.kernel == "norm":
            ctx.slidedp_grad_norm(grads, n, 1.0 / R, True)
            ctx.slidedp_grad_norm_finish(args.clip)
        elif args.kernel == "reduce":
            ctx.slidedp_reduce_mean_bf16(grads, n, 1.0 / R, p)
        elif args.kernel == "deliver":
            ctx.slidedp_deliver_params(hw, n, p, 16 << 20, 3, want_stats=False)
        else:
            ctx.slidedp_stream_step(grads, n, hw, hm, hv, p, 16 << 20, 3, hp, want_stats=False)
    ev[args.launches].record(st)
    torch.cuda.synchronize()
    ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.launches)]
    per = {"update": 26 + 2 * R, "norm": 2 * R, "reduce": 2 * R + 2, "stream": 24, "deliver": 4}[args.kernel]
    print(json.dumps({"report": "kernel", "kernel": args.kernel, "params": n, "R": R,
                      "ms_per_launch": ms, "bytes_per_param": per,
                      "best_gbs": per * n / (min(ms) * 1e6)}))
    ctx.slidedp_destroy()
    return 0


# ------------------------------------------------------------------- launching the ranks
def _free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_entry(rank, world, port, worker, args):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.exit(worker(args))


def launch_ranks(world: int, worker, args) -> int:
    """Runs `worker(args)` as `world` processes of this node, one per GPU, with the launcher
    environment (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, MASTER_PORT) set as an
    outer launcher would set it. Returns the first non-zero exit code, else 0."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    port = _free_port()
    procs = [ctx.Process(target=_rank_entry, args=(r, world, port, worker, args))
             for r in range(world)]
    for p in procs:
        p.start()
    # a rank that dies (no device, a failed check) must not leave the others waiting at the
    # rendezvous: stop exactly the processes started here as soon as one exits non-zero
    failed = None
    while failed is None and any(p.is_alive() for p in procs):
        for p in procs:
            p.join(timeout=0.2)
            if p.exitcode not in (None, 0):
                failed = p.exitcode
                break
    if failed is not None:
        for p in procs:
            if p.is_alive():
                p.terminate()
        for p in procs:
            p.join(timeout=10)
        return failed if failed > 0 else 1
    for p in procs:
        p.join()
        if p.exitcode != 0:
            return p.exitcode if p.exitcode and p.exitcode > 0 else 1
    return 0


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--report", choices=["contract", "sweep", "kernel"], default="contract")
    ap.add_argument("--sharded", action="store_true",
                    help="one layer sharded over the ranks (peer-mapped gradients, BF16 copy stored "
                         "to every rank) instead of one independent layer per rank")
    ap.add_argument("--kernel", choices=["update", "norm", "reduce", "stream", "deliver"],
                    default="update")
    ap.add_argument("--params", type=int, default=48 << 20)
    ap.add_argument("--R", type=int, default=4)
    ap.add_argument("--launches", type=int, default=4)
    ap.add_argument("--clip", type=float, default=1.0)
    args = ap.parse_args(argv)
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    launched = "RANK" in os.environ and "WORLD_SIZE" in os.environ
    if launched and int(os.environ["WORLD_SIZE"]) != args.gpus:
        print(f"bench.py: --gpus {args.gpus} disagrees with WORLD_SIZE={os.environ['WORLD_SIZE']} "
              "set by the launcher", file=sys.stderr)
        return 2
    if args.impl == "reference":
        return run_reference(args)
    if args.report == "sweep":
        return run_sweep(args)
    if args.report == "kernel":
        return run_kernel_case(args)
    worker = run_sharded if args.sharded else run_cuda
    if not launched and args.gpus > 1:
        return launch_ranks(args.gpus, worker, args)      # no outer launcher: start the ranks here
    return worker(args)


if __name__ == "__main__":
    sys.exit(main())
