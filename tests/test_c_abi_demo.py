"""The C ABI used from plain C: the demo program under paper_2603_21331_b200/examples is compiled
with gcc against include/ak.h and libak.so (CPU check), and run on the GPU, where it verifies
its outputs against closed forms by itself."""
import os
import shutil
import subprocess

import pytest

import paper_2603_21331_b200 as ak

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "paper_2603_21331_b200", "examples", "c_abi_demo.c")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def _build(out_dir):
    exe = os.path.join(str(out_dir), "c_abi_demo")
    lib_dir = os.path.dirname(ak.LIB_PATH)
    cmd = ["gcc", SRC, "-I" + os.path.join(ROOT, "include"), "-I" + os.path.join(CUDA, "include"),
           "-L" + lib_dir, "-lak", "-L" + os.path.join(CUDA, "lib64"), "-lcudart", "-lm",
           "-Wl,-rpath," + lib_dir, "-Wall", "-Werror", "-o", exe]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    return exe


@pytest.mark.skipif(shutil.which("gcc") is None or not os.path.isdir(os.path.join(CUDA, "include")),
                    reason="needs gcc and the CUDA runtime headers")
def test_c_demo_compiles_against_the_header(tmp_path):
    ak.lib()                      # the library must exist (built on demand by conftest)
    assert os.path.exists(_build(tmp_path))


@pytest.mark.gpu
def test_c_demo_runs_and_checks_itself(tmp_path):
    exe = _build(tmp_path)
    p = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert p.returncode == 0, p.stdout + p.stderr
    assert "0 failures" in p.stdout
