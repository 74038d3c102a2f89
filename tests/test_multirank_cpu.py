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
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
