"""A C++ program that uses the C ABI with nothing but the CUDA runtime (no Python, no tensor library) is built
against include/memstore.h and libmemstore.so and run on the GPU."""
import os
import subprocess
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu

ROOT = Path(__file__).resolve().parent.parent


def test_a_plain_cuda_runtime_client_of_the_c_abi(tmp_path):
    from paper_2607_27090_b200 import build

    lib = build.build()
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    exe = tmp_path / "abi_client"
    cmd = [nvcc, "-std=c++17", "-O1", "-I", str(ROOT / "include"), str(ROOT / "tests" / "abi_client.cpp"), str(lib),
           "-Xlinker", "-rpath", "-Xlinker", str(lib.parent), "-o", str(exe)]  # fmt: skip
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and "abi client ok" in r.stdout, r.stdout + r.stderr
