"""The boundary really is a C ABI: a plain C program (gcc, include/omc.h, no C++ and no Python
objects) links libomc.so, runs compress -> update -> decompress on the GPU and checks the result."""
import os
import subprocess

import pytest

import paper_2205_03494_b200 as omc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_plain_c_program_uses_the_library(tmp_path):
    omc.lib()
    exe = str(tmp_path / "use_from_c")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    libdir = os.path.dirname(omc.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c11", "-O1", "-o", exe, os.path.join(ROOT, "tests", "c_abi", "use_from_c.c"),
                           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                           "-L", libdir, "-l:libomc.so", "-L", os.path.join(cuda, "lib64"), "-lcudart",
                           "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    r = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.startswith("OK status=0"), r.stdout + r.stderr
