"""CPU-side checks of the C ABI: the library builds, loads and exports what the header
declares; the host-only entry points behave; the comparators in parity.py are sane."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_34162_b200.build import build
    return ctypes.CDLL(build())


def declared_symbols():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"SLIDEDP_API\s+[\w\s\*]+?\b(slidedp_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert {"slidedp_grad_norm", "slidedp_reduce_adamw_chunk", "slidedp_stream_step",
            "slidedp_create", "slidedp_destroy"} <= set(names)
    for name in names:
        assert getattr(lib, name) is not None, name


def test_state_bytes_is_16_per_parameter(lib):
    lib.slidedp_state_bytes.restype = ctypes.c_size_t
    lib.slidedp_state_bytes.argtypes = [ctypes.c_int64]
    for n in (0, 1, 7, 1 << 20, 192_946_176, 2_642_493_440):
        assert lib.slidedp_state_bytes(n) == 16 * n
    assert lib.slidedp_state_bytes(-5) == 0


def declared_statuses():
    """{name: value} of the slidedp_status enum, read from the header."""
    text = open(os.path.join(ROOT, "include", "slidedp.h")).read()
    body = re.search(r"typedef enum \{(.*?)\} slidedp_status;", text, re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    return {k: int(v) for k, v in re.findall(r"(SLIDEDP_\w+)\s*=\s*(-?\d+)", body)}


def test_strerror_names_every_status(lib):
    lib.slidedp_strerror.restype = ctypes.c_char_p
    statuses = declared_statuses()
    assert statuses["SLIDEDP_OK"] == 0 and len(statuses) >= 9
    assert sorted(statuses.values()) == list(range(-(len(statuses) - 1), 1))     # dense, no gaps
    seen = {lib.slidedp_strerror(v).decode() for v in statuses.values()}
    assert len(seen) == len(statuses) and "unknown status" not in seen
    assert lib.slidedp_strerror(min(statuses.values()) - 1).decode() == "unknown status"
    assert lib.slidedp_strerror(-99).decode() == "unknown status"
    # the binding's constants are the header's
    import paper_2609_34162_b200.slidedp as sd
    for name, value in statuses.items():
        short = name.replace("SLIDEDP_", "")
        assert getattr(sd, short) == value, name


def test_argument_errors_need_no_gpu(lib):
    lib.slidedp_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_size_t]
    assert lib.slidedp_create(None, 0, 0) == -1
    assert lib.slidedp_destroy(None) == 0
    lib.slidedp_grad_norm.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                      ctypes.c_int64, ctypes.c_double, ctypes.c_int, ctypes.c_void_p]
    assert lib.slidedp_grad_norm(None, None, 2, 8, 0.5, 1, None) == -1
    if not torch.cuda.is_available():
        h = ctypes.c_void_p()
        assert lib.slidedp_create(ctypes.byref(h), 0, 0) == -5 and not h.value   # loud, no fallback


def test_binding_has_the_c_names_and_no_oracle_import():
    import paper_2609_34162_b200.slidedp as b
    for name in ("slidedp_grad_norm", "slidedp_grad_norm_finish", "slidedp_reduce_adamw_chunk",
                 "slidedp_stream_step", "slidedp_link_probe", "slidedp_destroy"):
        assert hasattr(b.Context, name)
    assert b.slidedp_state_bytes(3) == 48
    pkg = os.path.join(ROOT, "paper_2609_34162_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", text, re.M), fn
                assert "slidedp_oracle" not in text, fn
                assert not re.search(r"^\s*(import|from)\s+baseline\b", text, re.M), fn
                assert "cpu_route" not in text and "cpuroute" not in text, fn
    for fn in os.listdir(os.path.join(ROOT, "oracle")):
        if fn.endswith((".py", ".c", ".h")):
            text = open(os.path.join(ROOT, "oracle", fn)).read()
            assert "paper_2609_34162_b200" not in text and "slidedp.h" not in text, fn
            assert "cpu_route" not in text and "cpuroute" not in text, fn
    # the paper-route baseline stands alone as well: neither the library nor the oracle
    base = os.path.join(ROOT, "baseline", "cpu_route")
    for fn in os.listdir(base):
        if fn.endswith((".py", ".cpp", ".h")):
            text = open(os.path.join(base, fn)).read()
            assert not re.search(r"^\s*(import|from)\s+(oracle|paper_2609_34162_b200)\b", text, re.M), fn
            assert "slidedp.h" not in text and "slidedp_oracle" not in text and "internal.h" not in text, fn


def test_workload_sizes_and_determinism():
    from paper_2609_34162_b200 import workloads as W
    sizes = {k: w.numel for k, w in W.CONFIGS.items()}
    assert sizes == {"tiny": 1_048_576, "qwen3_8b_layer": 192_946_176,
                     "qwen3_14b_layer_host": 330_311_680, "qwen25_72b_layer_host": 877_660_160,
                     "qwen3_14b_8layers_host": 2_642_493_440}
    assert W.chunk_elems(64) == 16 * (1 << 20)
    w = W.scaled(W.CONFIGS["qwen25_72b_layer_host"], 4096)
    a = W.rank_gradient(w, rank=1, step=3)
    b = W.rank_gradient(w, rank=1, step=3)
    c = W.rank_gradient(w, rank=2, step=3)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16)) and not torch.equal(a, c)
    x = a.float()
    assert 0.5e-3 < x.std() < 3e-3 and x.abs().max() > 8e-3      # N(0,1e-3) body, heavy tail
    w2 = W.scaled(W.CONFIGS["qwen3_8b_layer"], 2048)
    mw = W.master_weights(w2)
    assert mw.dtype == torch.float32 and mw.numel() == w2.numel
    k = 2 * w2.tensors[-1][1]                       # the two RMSNorm vectors sit last
    assert torch.all(mw[-k:] == 1.0) and 0.015 < mw[:-k].std() < 0.025


def test_comparators():
    import parity
    y = np.array([1.0, 1e-3, 0.0, -2.0], np.float32)
    assert parity.fp32_violations(y.copy(), y)[0] == 0
    x = y.copy(); x[0] = np.float32(1.0 + 3e-6)
    assert parity.fp32_violations(x, y)[0] == 1
    x = y.copy(); x[2] = np.float32(5e-13)
    assert parity.fp32_violations(x, y)[0] == 0
    x[2] = np.float32(2e-12)
    assert parity.fp32_violations(x, y)[0] == 1
    a = np.array([0x3F80, 0x0000, 0x8001, 0x7F7F], np.uint16)
    b = np.array([0x3F81, 0x8000, 0x0000, 0x7F7F], np.uint16)
    assert parity.bf16_mismatch(a, a) == (0, 0.0)
    assert parity.bf16_mismatch(a, b) == (1, 0.5)      # +0 and -0 coincide on the line


def test_shard_bounds_are_tile_aligned_and_cover_the_space():
    import paper_2609_34162_b200.slidedp as b
    for n in (0, 1, 16383, 16384, 16385, 192_946_176, 2_642_493_440):
        for shards in (1, 2, 3, 4, 8, 16):
            bounds = b.shard_bounds(n, shards)
            assert len(bounds) == shards and bounds[0][0] == 0 and bounds[-1][1] == n
            assert all(x[1] == y[0] for x, y in zip(bounds, bounds[1:]))
            assert all((lo % b.NORM_TILE == 0 or lo == n) and lo <= hi for lo, hi in bounds)
            sizes = [hi - lo for lo, hi in bounds]
            assert max(sizes) - min(sizes) <= 2 * b.NORM_TILE     # balanced to a tile
