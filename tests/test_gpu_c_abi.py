"""The C boundary used from a plain C program (no Python, no C++): tests/c/abi_smoke.c is compiled with gcc against
include/gmlp.h, linked with libgmlp.so and the CUDA runtime, and run; it checks its results against loops of its own."""
import os
import shutil
import subprocess

import pytest

from paper_2606_26344_b200 import build as B

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_c_program_links_and_runs(tmp_path):
    B.build_libgmlp()
    libdir = os.path.join(ROOT, "paper_2606_26344_b200")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = tmp_path / "abi_smoke"
    assert shutil.which("gcc")
    r = subprocess.run(["gcc", "-std=c99", "-O1", os.path.join(ROOT, "tests", "c", "abi_smoke.c"),
                        "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                        "-L", libdir, "-lgmlp", "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm",
                        f"-Wl,-rpath,{libdir}", f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}", "-o", str(exe)],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    run = subprocess.run([str(exe)], capture_output=True, text=True, timeout=300)
    assert run.returncode == 0 and run.stdout.startswith("ok"), run.stdout + run.stderr
