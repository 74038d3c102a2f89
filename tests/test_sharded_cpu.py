"""Host-side logic of the sharded multi-rank step (paper Sec. 3.2 "Gradient return" /
"Parameter dispatch"), on CPU with two gloo ranks and a recording stand-in for the library:
the shard bounds, the rank-major gradient order, which pointer is local and which is mapped,
the byte offsets every kernel is given, the position of each shard's tile sums in the gathered
array, and the order of the calls between the barriers. No arithmetic is involved: the real
kernels behind the same calls are covered by the GPU tests."""
import os
import socket
import struct
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TILE = 16384


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def fake_address(rank: int, ptr: int) -> int:
    """What the stand-in's slidedp_ipc_open returns for a buffer exported by `rank`."""
    return ((rank + 1) << 52) | (ptr & ((1 << 48) - 1))


class RecordingCtx:
    def __init__(self, rank):
        self.rank, self.calls, self.closed = rank, [], []

    def slidedp_ipc_export(self, t):
        return struct.pack("<qq", self.rank, t.data_ptr()).ljust(80, b"\0")

    def slidedp_ipc_open(self, handle):
        rank, ptr = struct.unpack("<qq", handle[:16])
        assert rank != self.rank, "a handle cannot be opened by the process that exported it"
        return fake_address(rank, ptr)

    def slidedp_ipc_close(self, p):
        self.closed.append(p)

    def slidedp_grad_norm_tiles(self, grads, k, inv_R, out, stream=None):
        self.calls.append(("tiles", list(grads), k, inv_R, out.data_ptr()))

    def slidedp_scatter_tile_sums(self, src, count, dsts, stream=None):
        self.calls.append(("scatter", src.data_ptr(), count, list(dsts)))

    def slidedp_grad_norm_finish_from(self, tiles, count, max_norm, fetch=False, stream=None):
        self.calls.append(("finish", tiles.data_ptr(), count, max_norm))
        return (2.0, 0.5)

    def slidedp_reduce_adamw_chunk_bcast(self, grads, k, w, m, v, outs, hp, stream=None):
        self.calls.append(("update", list(grads), k, w.data_ptr(), list(outs), hp.step))


class NoStream:
    cuda_stream = 0

    def synchronize(self):
        pass


def _worker(rank, world, port, n, k_local, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2609_34162_b200.sharded import ShardedStep
    from paper_2609_34162_b200.slidedp import HParams
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        grads = [torch.zeros(n, dtype=torch.bfloat16) for _ in range(k_local)]
        param = torch.zeros(n, dtype=torch.bfloat16)
        ctx = RecordingCtx(rank)
        sh = ShardedStep(ctx, grads, n, param)
        ptrs = [None] * world
        dist.all_gather_object(ptrs, {"g": [g.data_ptr() for g in grads], "p": param.data_ptr(),
                                      "t": sh.gathered.data_ptr()})
        lo, hi = sh.bounds[rank]
        shard = [torch.zeros(hi - lo) for _ in range(3)]
        res = sh.step(*shard, HParams(inv_R=1.0 / (world * k_local), max_norm=1.0, step=3),
                      stream=NoStream())
        sh.step(*shard, HParams(inv_R=1.0 / (world * k_local), max_norm=0.0, step=4), stream=NoStream())
        sh.close()
        out.put((rank, {"bounds": sh.bounds, "counts": sh.counts, "offsets": sh.offsets,
                        "total": sh.total_tiles, "calls": ctx.calls, "closed": ctx.closed,
                        "ptrs": ptrs, "res": res, "local_tiles": sh.local_tiles.data_ptr(),
                        "shard_w": shard[0].data_ptr()}))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("n,k_local", [(5 * TILE + 123, 1), (3 * TILE, 2), (100, 1)])
def test_two_ranks_give_every_kernel_the_right_pointers(n, k_local):
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n, k_local, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank in range(world):
        r = res[rank]
        ptrs, (lo, hi) = r["ptrs"], r["bounds"][rank]
        assert r["bounds"] == res[0]["bounds"] and r["total"] == -(-n // TILE)
        assert r["offsets"] == [0, r["counts"][0]]
        where = lambda owner, p: p if owner == rank else fake_address(owner, p)
        want_grads = [where(o, g) + 2 * lo for o in range(world) for g in ptrs[o]["g"]]
        order = [rank] + [o for o in range(world) if o != rank]
        want_outs = [where(o, ptrs[o]["p"]) + 2 * lo for o in order]
        want_dsts = [where(o, ptrs[o]["t"]) + 8 * r["offsets"][rank] for o in order]
        kinds = [c[0] for c in r["calls"]]
        assert kinds == ["tiles", "scatter", "finish", "update", "update"]     # clipped, then not
        tiles, scatter, finish, upd, upd2 = r["calls"]
        assert tiles[1] == want_grads and tiles[2] == hi - lo and tiles[4] == r["local_tiles"]
        assert tiles[3] == 1.0 / (world * k_local)
        assert scatter[1] == r["local_tiles"] and scatter[2] == r["counts"][rank] and scatter[3] == want_dsts
        assert finish[1] == ptrs[rank]["t"] and finish[2] == r["total"] and finish[3] == 1.0
        assert upd[1] == want_grads and upd[2] == hi - lo and upd[3] == r["shard_w"]
        assert upd[4] == want_outs and upd[5] == 3 and upd2[5] == 4
        assert r["res"] == (2.0, 0.5)
        # every peer buffer that was mapped is unmapped again: k gradients, the parameter
        # buffer and the tile array of the one peer
        peer = 1 - rank
        assert sorted(r["closed"]) == sorted([fake_address(peer, g) for g in ptrs[peer]["g"]] +
                                             [fake_address(peer, ptrs[peer]["p"]),
                                              fake_address(peer, ptrs[peer]["t"])])


def test_shard_bounds_tile_aligned_cover():
    sys.path.insert(0, ROOT)
    from paper_2609_34162_b200.slidedp import shard_bounds
    for n in (0, 1, TILE - 1, TILE, TILE + 1, 7 * TILE + 5, 192_946_176, 330_311_680):
        for shards in (1, 2, 3, 4, 8, 16):
            b = shard_bounds(n, shards)
            assert len(b) == shards and b[0][0] == 0 and b[-1][1] == n
            for (lo, hi), (lo2, _) in zip(b, b[1:]):
                assert hi == lo2 and lo <= hi
            assert all(lo % TILE == 0 or lo == n for lo, _ in b)
            sizes = [-(-(hi - lo) // TILE) for lo, hi in b]
            assert sum(sizes) == -(-n // TILE) and max(sizes) - min(sizes) <= 1
