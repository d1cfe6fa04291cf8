"""The library is usable from plain C: compile tests/c_abi/smoke.c with gcc against
include/maxdnn.h, libmaxdnn.so and the CUDA runtime, run it, expect "C ABI OK"."""
import os
import subprocess

import pytest

import paper_1501_06633_b200 as mx

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_plain_c_program_runs_forward_and_both_gradients(tmp_path):
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    lib_dir = os.path.dirname(mx.library_path())
    exe = str(tmp_path / "smoke")
    cmd = ["gcc", "-O1", "-std=c11", os.path.join(ROOT, "tests", "c_abi", "smoke.c"),
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
           "-L", lib_dir, "-l:libmaxdnn.so", "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm",
           "-Wl,-rpath," + lib_dir, "-Wl,-rpath," + os.path.join(cuda, "lib64"), "-o", exe]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "C ABI OK" in out.stdout
