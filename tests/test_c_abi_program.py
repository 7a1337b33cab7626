"""The library used from a plain C program (no Python, no torch on the data path): it must compile
and link against include/wm.h and libwm.so anywhere, and run its round trip on a GPU."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


@pytest.fixture(scope="module")
def program(tmp_path_factory):
    from paper_2607_10389_b200 import build
    lib = build.build()
    exe = str(tmp_path_factory.mktemp("cabi") / "roundtrip")
    cmd = ["gcc", "-O1", "-std=c99", "-Wall", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"),
           os.path.join(ROOT, "tests", "c_abi", "roundtrip.c"), lib, "-L", os.path.join(CUDA, "lib64"), "-lcudart",
           "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.join(CUDA, "lib64"), "-o", exe]
    subprocess.check_call(cmd)
    return exe


def test_c_program_compiles_and_links(program):
    assert os.access(program, os.X_OK)


@pytest.mark.gpu
def test_c_program_round_trip(program):
    out = subprocess.run([program], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.count("ok") == 2
