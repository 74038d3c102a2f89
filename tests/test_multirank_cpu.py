"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, rendezvous on 127.0.0.1.

The path shards into independent layers (one per rank, no data-path collective); what the ranks
share is only the timing reduction (max over ranks) and the whole-job aggregate."""
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_34162_b200 import workloads as W
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
        slowest = bench.max_over_ranks(local_ms, world, device="cpu")
        layer = bench.layer_of_rank(rank)
        wl = W.scaled(W.CONFIGS["qwen3_8b_layer"], 4096)
        g = W.rank_gradient(wl, 0, step=11, layer=layer)
        gathered = [torch.zeros_like(g, dtype=torch.float32) for _ in range(world)]
        dist.all_gather(gathered, g.float())
        out.put((rank, slowest, layer, bool(torch.equal(gathered[0], gathered[1])),
                 bench.job_value(world, 1000, 4, slowest)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_max_time_and_distinct_layers():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]           # both see the slowest rank's time
    assert [r[2] for r in res] == [0, 1]                 # different layers ...
    assert res[0][3] is False                            # ... with different gradients
    assert res[0][4] == 2 * 1000 * 4 / 15e-3 / 1e9       # whole-job aggregate over all ranks


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.job_value(1, 192_946_176, 50, 50 * 1.2167) > 158


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def _gloo_rank(args):
    """A stand-in for bench.py's per-rank worker: joins a gloo group from the environment that
    bench.launch_ranks prepared and proves that both ranks met."""
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert os.environ["MASTER_ADDR"] == "127.0.0.1" and os.environ["LOCAL_RANK"] == str(rank)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        t = torch.tensor([float(rank + 1)])
        dist.all_reduce(t)
        with open(os.path.join(args["dir"], f"rank{rank}.txt"), "w") as f:
            f.write(f"{world} {t.item()}")
    finally:
        dist.destroy_process_group()
    return args["codes"][rank]


def test_bench_starts_its_own_ranks_when_no_launcher_did(tmp_path):
    sys.path.insert(0, ROOT)
    import bench
    assert bench.launch_ranks(2, _gloo_rank, {"dir": str(tmp_path), "codes": [0, 0]}) == 0
    assert sorted(os.listdir(tmp_path)) == ["rank0.txt", "rank1.txt"]
    for r in range(2):
        assert open(tmp_path / f"rank{r}.txt").read() == "2 3.0"     # world 2, 1 + 2
    # a failing rank is reported
    assert bench.launch_ranks(2, _gloo_rank, {"dir": str(tmp_path), "codes": [0, 7]}) == 7


def test_gpus_flag_reaches_the_rank_spawn_and_must_agree_with_a_launcher():
    exe = [sys.executable, os.path.join(ROOT, "bench.py")]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    if not torch.cuda.is_available():
        r = subprocess.run(exe + ["--gpus", "2", "--steps", "1", "--warmup", "0"], env=env,
                           capture_output=True, text=True, timeout=300)
        # the ranks were started and stopped where the CUDA path must: no device, no fallback
        # (the first rank to fail takes its sibling down, so one or two messages)
        assert r.returncode != 0 and 1 <= r.stderr.count("needs a CUDA device") <= 2, r.stderr
    r = subprocess.run(exe + ["--gpus", "2"], env=dict(env, RANK="0", WORLD_SIZE="4"),
                       capture_output=True, text=True, timeout=120)
    assert r.returncode == 2 and "disagrees with WORLD_SIZE" in r.stderr


def _one_rank_dies(args):
    """Rank 1 fails at once; rank 0 would wait a long time (as it would at a rendezvous)."""
    if int(os.environ["RANK"]) == 1:
        return 7
    import time
    time.sleep(120)
    return 0


def test_a_failed_rank_does_not_leave_the_others_waiting():
    import time
    sys.path.insert(0, ROOT)
    import bench
    t0 = time.perf_counter()
    assert bench.launch_ranks(2, _one_rank_dies, None) == 7
    assert time.perf_counter() - t0 < 60


def test_only_the_result_line_reaches_stdout():
    """Whatever a library underneath writes to file descriptor 1 (NCCL prints a version banner
    there) ends up on stderr; stdout carries the one JSON line."""
    code = ("import os, sys; sys.path.insert(0, %r); import bench\n"
            "ch = bench.ResultChannel()\n"
            "os.write(1, b'banner from a C library\\n'); print('a stray print')\n"
            "ch.emit({'value': 1.5}); ch.close()\n") % ROOT
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout == '{"value": 1.5}\n', (r.stdout, r.stderr)
    assert "banner from a C library" in r.stderr and "a stray print" in r.stderr
