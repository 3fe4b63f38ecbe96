"""The library used from a plain CUDA-runtime program (no Python, no PyTorch in the process):
tests/c_abi/plain_caller.cu is compiled against include/awq_b200.h, linked with the in-tree
shared library and run; it checks every kernel family against a double-precision product and
exits 0 only if all are within tolerance."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "tests", "c_abi", "plain_caller.cu")


def _build(tmp_path):
    from paper_2306_00978_b200 import build
    lib = build.build()
    exe = str(tmp_path / "plain_caller")
    libdir = os.path.dirname(lib)
    cmd = ["nvcc", "-O2", "-std=c++17", "-I", os.path.join(ROOT, "include"), SRC, "-o", exe,
           "-L", libdir, "-l:" + os.path.basename(lib), "-Xlinker", "-rpath", "-Xlinker", libdir, "-lcudart"]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    return exe


def test_plain_caller_compiles_and_links(tmp_path):
    """No GPU needed: the header is usable from C++ host code and every symbol it uses resolves."""
    assert os.path.exists(_build(tmp_path))


@pytest.mark.gpu
def test_plain_caller_runs(tmp_path):
    exe = _build(tmp_path)
    out = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    sys.stdout.write(out.stdout)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.strip().endswith("OK")
