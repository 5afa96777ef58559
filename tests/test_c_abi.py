"""The C ABI used from plain C: tests/c_abi/c_abi_check.c is compiled with gcc against
include/quantpipe.h and linked with the library.  Without a GPU only its host-side calls run;
the GPU test runs the whole path (sender call, unpack) from C."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


@pytest.fixture(scope="module")
def c_program(tmp_path_factory):
    from paper_2211_04515_b200 import build
    build.build()
    out = str(tmp_path_factory.mktemp("c_abi") / "c_abi_check")
    libdir = os.path.join(ROOT, "paper_2211_04515_b200")
    cmd = ["gcc", "-std=c99", "-Wall", "-Werror", "-I" + os.path.join(ROOT, "include"), "-I" + os.path.join(CUDA, "include"),
           os.path.join(ROOT, "tests", "c_abi", "c_abi_check.c"), "-L" + libdir, "-lquantpipe",
           "-L" + os.path.join(CUDA, "lib64"), "-lcudart", "-lm", "-Wl,-rpath," + libdir,
           "-Wl,-rpath," + os.path.join(CUDA, "lib64"), "-o", out]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    return out


def test_header_compiles_as_c_and_host_calls_work(c_program):
    res = subprocess.run([c_program], capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == "host ok", res.stderr


@pytest.mark.gpu
def test_whole_path_from_c(c_program):
    res = subprocess.run([c_program, "gpu"], capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == "gpu ok", res.stderr
