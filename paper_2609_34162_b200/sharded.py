"""The sharded multi-rank step: one process per GPU, each holding its rank-local BF16 gradient.

Orchestration only; there is no arithmetic in this module. Every number is produced by
libslidedp's kernels, every byte of data moves through those kernels' plain loads and stores on
buffers mapped between the processes; ``torch.distributed`` carries the 80-byte buffer handles
once and the barriers that order the ranks.

What the ranks do (paper Sec. 3.2: "Gradient return" sums the rank-local gradients into one
result; "Parameter dispatch", sharded delivery, lets every rank hold 1/R of a layer and
reconstructs it with an all-gather). With G ranks the flat parameter space of n parameters is
cut into G contiguous shards at multiples of the norm tile (``shard_bounds``); rank s

  1. maps every peer's gradient buffer(s), BF16 parameter buffer and tile-sum array (once);
  2. computes the tile sums of its shard over ALL ranks' gradients (``slidedp_grad_norm_tiles``
     reads the peers' slices in rank order) and stores them into every rank's gathered array
     (``slidedp_scatter_tile_sums``);                                             -- barrier --
  3. folds the gathered array (``slidedp_grad_norm_finish_from``): every rank gets the norm and
     the clip coefficient of the unsharded step, bit for bit;
  4. updates its shard of master / m / v, the kernel storing the BF16 copy of the shard into
     every rank's parameter buffer (``slidedp_reduce_adamw_chunk_bcast``).         -- barrier --

The gradients cross the GPU interconnect once (each rank reads the 1/G it needs), the BF16
parameters once (each rank writes its 1/G to the others), the norm costs 8 bytes per 16384
parameters. Rank order of the reduction: rank-major, then the order of a rank's own buffers.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from .slidedp import NORM_TILE, HParams, shard_bounds


def tile_count(n: int) -> int:
    return -(-n // NORM_TILE)


class ShardedStep:
    """One layer's sharded update across the ranks of a process group.

    ctx          a ``slidedp.Context`` on this rank's device (anything with the same methods).
    local_grads  this rank's BF16 gradient buffers (device tensors of n elements, usually one).
    param_bf16   this rank's BF16 parameter buffer (device, n): receives EVERY shard.
    The FP32 state is not held here: ``step`` takes this rank's shard of master / m / v
    (``hi - lo`` elements each, see ``bounds``).
    """

    def __init__(self, ctx, local_grads, n: int, param_bf16, group=None, tile_sums=None):
        self.ctx, self.n, self.group = ctx, n, group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.bounds = shard_bounds(n, self.world)
        self.lo, self.hi = self.bounds[self.rank]
        self.counts = [tile_count(hi - lo) for lo, hi in self.bounds]
        self.offsets = [sum(self.counts[:s]) for s in range(self.world)]
        self.total_tiles = sum(self.counts)
        assert self.total_tiles == tile_count(n)
        dev = param_bf16.device
        # every rank's gathered tile sums, and this shard's own
        self.gathered = tile_sums if tile_sums is not None else torch.zeros(
            max(self.total_tiles, 1), dtype=torch.float64, device=dev)
        self.local_tiles = torch.zeros(max(self.counts[self.rank], 1), dtype=torch.float64, device=dev)
        self._keep = (list(local_grads), param_bf16)

        # ---- exchange the buffer handles (control plane, once)
        mine = {"grads": [ctx.slidedp_ipc_export(g) for g in local_grads],
                "param": ctx.slidedp_ipc_export(param_bf16),
                "tiles": ctx.slidedp_ipc_export(self.gathered)}
        everyone = [None] * self.world
        dist.all_gather_object(everyone, mine, group=group)
        self._mapped = []

        def address(rank, handle, own):
            if rank == self.rank:
                return own
            p = ctx.slidedp_ipc_open(handle)
            self._mapped.append(p)
            return p

        self.grad_ptrs, self.param_ptrs, self.tile_ptrs = [], [], []
        for r, h in enumerate(everyone):
            own_g = [g.data_ptr() for g in local_grads]
            for i, hg in enumerate(h["grads"]):
                self.grad_ptrs.append(address(r, hg, own_g[i] if r == self.rank else None))
            self.param_ptrs.append(address(r, h["param"], param_bf16.data_ptr()))
            self.tile_ptrs.append(address(r, h["tiles"], self.gathered.data_ptr()))
        self.R = len(self.grad_ptrs)
        # this rank first among the outputs (its own copy is the local store)
        order = [self.rank] + [r for r in range(self.world) if r != self.rank]
        self.param_ptrs = [self.param_ptrs[r] for r in order]
        self.tile_ptrs = [self.tile_ptrs[r] for r in order]

    def _barrier(self, stream):
        """Everything this rank queued is complete, then every rank is here."""
        stream.synchronize()
        dist.barrier(group=self.group)
        if dist.get_backend(self.group) == "nccl":
            # an NCCL barrier is itself stream work on torch's current stream: wait for it on
            # the host, so that the ordering holds whatever stream the step's kernels use
            torch.cuda.current_stream().synchronize()

    def step(self, master_shard, m_shard, v_shard, hp: HParams, stream=None):
        """One update. The rank-local gradients must already be complete on every rank's device
        and no rank may still read the previous BF16 copy (the first barrier below orders both,
        given that each rank calls ``step`` only after its own backward / forward is done).
        Returns (norm, coef) when clipping, else None."""
        ctx, lo, hi = self.ctx, self.lo, self.hi
        stream = stream if stream is not None else torch.cuda.current_stream()
        k = hi - lo
        grads = [p + 2 * lo for p in self.grad_ptrs]                     # BF16: 2 bytes each
        self._barrier(stream)
        out = None
        if hp.max_norm > 0.0:
            ctx.slidedp_grad_norm_tiles(grads, k, hp.inv_R, self.local_tiles, stream=stream)
            dsts = [p + 8 * self.offsets[self.rank] for p in self.tile_ptrs]
            ctx.slidedp_scatter_tile_sums(self.local_tiles, self.counts[self.rank], dsts, stream=stream)
            self._barrier(stream)
            out = ctx.slidedp_grad_norm_finish_from(self.gathered, self.total_tiles, hp.max_norm,
                                                    fetch=True, stream=stream)
        outs = [p + 2 * lo for p in self.param_ptrs]
        ctx.slidedp_reduce_adamw_chunk_bcast(grads, k, master_shard, m_shard, v_shard, outs, hp,
                                             stream=stream)
        self._barrier(stream)
        return out

    def close(self):
        """Unmaps the peers' buffers (after a barrier: no peer kernel may still use ours)."""
        if self._mapped is None:
            return
        if torch.cuda.is_available():
            torch.cuda.synchronize()
        dist.barrier(group=self.group)
        for p in self._mapped:
            self.ctx.slidedp_ipc_close(p)
        self._mapped = None
        dist.barrier(group=self.group)
