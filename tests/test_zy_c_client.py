"""The C ABI used from a plain C++ program (no Python, no PyTorch in the caller): built with nvcc against
include/w8a8_linear.h, linked to the shared library, run on the GPU; its expected values are worked out by hand."""
import os
import subprocess

import pytest

from paper_2606_14598_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "tests", "c_client", "client.cpp")
EXE = os.path.join(ROOT, "tests", "c_client", "client")


def build_client():
    libdir = os.path.dirname(binding.LIB_PATH)
    cmd = ["nvcc", "-std=c++17", "-O1", "-x", "cu", "-o", EXE, SRC, "-L" + libdir, "-lw8a8_linear",
           "-Xlinker", "-rpath," + libdir]
    subprocess.run(cmd, check=True, capture_output=True, text=True)


def test_c_client_builds_and_links():
    build_client()
    assert os.path.exists(EXE)


@pytest.mark.gpu
def test_c_client_runs_on_the_gpu():
    build_client()
    r = subprocess.run([EXE], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "c client ok" in r.stdout
