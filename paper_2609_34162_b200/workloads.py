"""Seeded synthetic inputs for the five benchmark configurations.

This module only draws random numbers and lays tensors out flat; it contains none of
the method's arithmetic (no reduction, no Adam, no clipping), so that the CUDA path
and the CPU oracle can both be fed from it without sharing any of their own code.

The inputs stand in for the real gradients and weights of the paper's workloads
(Qwen3-8B / Qwen3-14B / Qwen2.5-72B decoder layers, paper Sec. 4.1), which are not
needed to exercise the update path: the shapes are the per-layer projection shapes,
gradients are N(0, sigma=1e-3) rounded to BF16 (config 4 mixes in 1% Student-t(3)
values of scale 1e-2), masters are N(0, sigma=0.02) in FP32 with RMSNorm weights 1.0.

Every draw is made in fixed segments of ``SEGMENT`` elements, each from its own
generator seeded by (config seed, kind, layer, rank, step, segment), so a piece of a
tensor can be regenerated alone and temporary memory stays bounded at full size.
A torch generator's stream depends on its device, so the two sides of a comparison
must be fed the SAME generated bits (generate once, copy), not regenerate per side.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

SEGMENT = 1 << 24  # elements per independently seeded draw

_KIND_GRAD, _KIND_MASTER = 1, 2


@dataclass(frozen=True)
class Workload:
    name: str
    mode: str                  # "device" | "host"
    tensors: tuple             # ((name, numel, init), ...) for ONE layer; init: "normal" | "ones"
    R: int
    layers: int = 1
    seed: int = 0
    first_step: int = 1        # step index of the measured update
    prewarm_steps: int = 0     # seeded steps run before the measured one
    steps: int = 1             # consecutive measured steps
    max_norm: float = 0.0
    heavy_tail: bool = False
    chunk_mib: tuple = (64,)   # bytes of ONE FP32 state array per chunk, in MiB
    nbuf: int = 3
    hparams: dict = field(default_factory=lambda: dict(lr=1e-5, beta1=0.9, beta2=0.95,
                                                       eps=1e-8, weight_decay=0.1))

    @property
    def layer_numel(self) -> int:
        return sum(t[1] for t in self.tensors)

    @property
    def numel(self) -> int:
        return self.layer_numel * self.layers


def _decoder(hidden, kv, inter, norms=True, kv_bias=False):
    t = [("q", hidden * hidden, "normal"), ("k", hidden * kv, "normal")]
    if kv_bias:
        t.append(("k_bias", kv, "normal"))
    t.append(("v", hidden * kv, "normal"))
    if kv_bias:
        t.append(("v_bias", kv, "normal"))
    t += [("o", hidden * hidden, "normal"), ("gate", hidden * inter, "normal"),
          ("up", hidden * inter, "normal"), ("down", inter * hidden, "normal")]
    if norms:
        t += [("input_norm", hidden, "ones"), ("post_attn_norm", hidden, "ones")]
    return tuple(t)


CONFIGS = {
    # one flat chunk, device-resident, first step from zero moments, no clipping
    "tiny": Workload("tiny", "device", (("chunk", 1 << 20, "normal"),), R=2, seed=0),
    # Qwen3-8B-shaped layer, device-resident, step 11 after 10 seeded steps, clip 1.0
    "qwen3_8b_layer": Workload("qwen3_8b_layer", "device", _decoder(4096, 1024, 12288), R=4,
                               seed=1, first_step=11, prewarm_steps=10, max_norm=1.0),
    # Qwen3-14B-shaped layer, host-resident, 64 MiB chunks, triple buffering
    "qwen3_14b_layer_host": Workload("qwen3_14b_layer_host", "host",
                                     _decoder(5120, 1024, 17408), R=4, seed=2, first_step=11,
                                     prewarm_steps=10, max_norm=1.0),
    # Qwen2.5-72B-shaped layer (k/v biases, no norms), heavy-tailed gradients, chunk sweep
    "qwen25_72b_layer_host": Workload("qwen25_72b_layer_host", "host",
                                      _decoder(8192, 1024, 29568, norms=False, kv_bias=True),
                                      R=4, seed=3, first_step=11, prewarm_steps=10, max_norm=1.0,
                                      heavy_tail=True, chunk_mib=(16, 64, 256)),
    # eight Qwen3-14B-shaped layers, host-resident, 10 steps from zero moments
    "qwen3_14b_8layers_host": Workload("qwen3_14b_8layers_host", "host",
                                       _decoder(5120, 1024, 17408), R=8, layers=8, seed=4,
                                       steps=10, max_norm=1.0),
}


def scaled(w: Workload, divisor: int, name: str | None = None) -> Workload:
    """The same workload with every tensor shrunk ``divisor``-fold (ragged sizes kept)."""
    tensors = tuple((n, max(1, numel // divisor) + (3 if init == "normal" else 0), init)
                    for n, numel, init in w.tensors)
    return Workload(name or f"{w.name}/{divisor}", w.mode, tensors, w.R, w.layers, w.seed,
                    w.first_step, w.prewarm_steps, w.steps, w.max_norm, w.heavy_tail,
                    w.chunk_mib, w.nbuf, dict(w.hparams))


def _seed(w: Workload, kind: int, layer: int, rank: int, step: int, segment: int) -> int:
    s = w.seed
    for x in (kind, layer, rank, step, segment):
        s = (s * 1_000_003 + x + 0x9E37) % (1 << 62)
    return s


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def rank_gradient(w: Workload, rank: int, step: int, layer: int = 0, device="cpu",
                  out: torch.Tensor | None = None) -> torch.Tensor:
    """BF16 gradient of one rank for one layer at one step (flat, ``layer_numel`` long)."""
    n = w.layer_numel
    if out is None:
        out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for si, lo in enumerate(range(0, n, SEGMENT)):
        k = min(SEGMENT, n - lo)
        g = _gen(device, _seed(w, _KIND_GRAD, layer, rank, step, si))
        x = torch.randn(k, generator=g, device=device, dtype=torch.float32) * 1e-3
        if w.heavy_tail:
            # 1% of the elements, chosen independently, are 1e-2 * Student-t(nu=3):
            # a standard normal over the root of a chi-square(3)/3.
            pick = torch.rand(k, generator=g, device=device) < 0.01
            z = torch.randn(k, generator=g, device=device, dtype=torch.float32)
            chi = torch.randn(3, k, generator=g, device=device, dtype=torch.float32)
            t3 = z / torch.sqrt((chi * chi).sum(0) / 3.0)
            x = torch.where(pick, 1e-2 * t3, x)
        out[lo:lo + k] = x.to(torch.bfloat16)
    return out


def master_weights(w: Workload, layer: int = 0, device="cpu",
                   out: torch.Tensor | None = None) -> torch.Tensor:
    """FP32 master of one layer: N(0, 0.02) for matrices and biases, 1.0 for norm weights."""
    n = w.layer_numel
    if out is None:
        out = torch.empty(n, dtype=torch.float32, device=device)
    for si, lo in enumerate(range(0, n, SEGMENT)):
        k = min(SEGMENT, n - lo)
        g = _gen(device, _seed(w, _KIND_MASTER, layer, 0, 0, si))
        out[lo:lo + k] = torch.randn(k, generator=g, device=device, dtype=torch.float32) * 0.02
    off = 0
    for _, numel, init in w.tensors:
        if init == "ones":
            out[off:off + numel] = 1.0
        off += numel
    return out


def chunk_elems(chunk_mib: int) -> int:
    """A chunk size quoted in MiB counts the bytes of ONE FP32 state array."""
    return chunk_mib * (1 << 20) // 4
