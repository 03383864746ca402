"""The shared library used from a plain C program (gcc, CUDA runtime for the allocations): struct layouts,
enums and calling convention as the headers declare them, with no Python marshalling in between."""
import os
import subprocess

import pytest

from paper_2607_26444_b200 import binding as B

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_c_program_runs_the_worked_example(tmp_path):
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = str(tmp_path / "c_abi_demo")
    lib = B.LIB_PATH
    B.lib()                                          # fails loudly if the library is not built
    cmd = ["gcc", "-std=c11", "-Wall", "-Werror", os.path.join(ROOT, "tests", "c_abi_demo.c"),
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"), lib,
           "-L", os.path.join(cuda, "lib64"), "-lcudart", "-Wl,-rpath," + os.path.dirname(lib),
           "-Wl,-rpath," + os.path.join(cuda, "lib64"), "-o", exe]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    r = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.startswith("PASS"), r.stdout + r.stderr
