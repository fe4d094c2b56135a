"""The library driven from a plain C program (no Python binding, no PyTorch): compiled with the host C compiler
against include/remoe.h, linked with libremoe.so and the CUDA runtime, run on the GPU.  The program carries its own
double-precision restatement of the step and compares every step with it."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def test_c_program_against_its_own_restatement(tmp_path):
    from paper_2605_27081_b200 import build
    lib = build.build_library()
    cc = shutil.which("gcc") or shutil.which("cc")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if cc is None or not os.path.isdir(os.path.join(cuda, "include")):
        pytest.skip("no C compiler or CUDA headers")
    exe = str(tmp_path / "abi_smoke")
    libdir = os.path.dirname(lib)
    subprocess.run([cc, "-std=c99", "-O1", "-Wall", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                    os.path.join(ROOT, "tests", "native", "abi_smoke.c"), "-o", exe,
                    "-L", libdir, "-lremoe", "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm",
                    "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(cuda, "lib64")], check=True)
    res = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip().endswith("ok"), res.stdout + res.stderr
