"""The C ABI driven from a plain C program (tests/c_abi_smoke.c): no Python between the caller and
libslidedp. The program is compiled on CPU machines too (so the header stays valid C), and run
where a GPU exists."""
import os
import subprocess

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def build_program(tmp_path):
    import oracle
    from paper_2609_34162_b200.build import build
    lib, olib = build(), oracle.build()
    exe = str(tmp_path / "c_abi_smoke")
    cmd = ["gcc", "-std=c99", "-O1", "-Wall", "-o", exe, os.path.join(ROOT, "tests", "c_abi_smoke.c"),
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(ROOT, "oracle"),
           "-I", os.path.join(CUDA, "include"), lib, olib, "-L", os.path.join(CUDA, "lib64"),
           "-lcudart", "-lm",
           f"-Wl,-rpath,{os.path.dirname(lib)}", f"-Wl,-rpath,{os.path.dirname(olib)}",
           f"-Wl,-rpath,{os.path.join(CUDA, 'lib64')}"]
    subprocess.run(cmd, check=True)
    return exe


def test_header_is_plain_c_and_the_program_links(tmp_path):
    assert os.path.exists(build_program(tmp_path))


@pytest.mark.gpu
def test_c_program_matches_the_oracle(tmp_path):
    assert torch.cuda.is_available()
    r = subprocess.run([build_program(tmp_path)], capture_output=True, text=True, timeout=300)
    print(r.stdout, r.stderr)
    assert r.returncode == 0 and r.stdout.startswith("PASS"), r.stdout + r.stderr
