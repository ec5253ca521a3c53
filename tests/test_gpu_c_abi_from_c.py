"""The C ABI used from a plain C program (no Python binding, no torch): compiled with gcc against
include/a2sgd.h and the CUDA runtime, run on the GPU, checked against the hand-worked fixture e1."""
import os
import shutil
import subprocess

import pytest

from paper_2006_07405_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_c_program_through_the_c_abi(tmp_path):
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if not shutil.which("gcc") or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime.h")):
        pytest.skip("gcc or the CUDA runtime headers are not available")
    lib = build.build()
    exe = tmp_path / "c_abi_fixture_e1"
    subprocess.check_call([
        "gcc", "-std=c11", "-O1", "-Wall", os.path.join(ROOT, "tests", "c", "c_abi_fixture_e1.c"),
        "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
        "-o", str(exe), lib, "-L", os.path.join(cuda, "lib64"), "-lcudart",
        "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    out = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip().endswith("ok"), out.stdout + out.stderr
