"""A host program written in plain C (tests/c_host/step_host.c) drives the library without Python or torch."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "tests", "c_host", "step_host.c")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def test_c_host_compiles_against_the_header():
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-fsyntax-only", "-I", os.path.join(ROOT, "include"),
                    "-I", os.path.join(CUDA, "include"), SRC], check=True)


@pytest.mark.gpu
def test_c_host_runs_the_hot_path(tmp_path):
    from paper_2601_09093_b200 import build
    lib = build.build()
    libdir = os.path.dirname(lib)
    exe = str(tmp_path / "step_host")
    subprocess.run(["gcc", "-std=c99", "-O1", SRC, "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"),
                    "-L", libdir, "-lstep", "-Wl,-rpath," + libdir, "-L", os.path.join(CUDA, "lib64"), "-lcudart", "-lm",
                    "-o", exe], check=True)
    env = dict(os.environ, LD_LIBRARY_PATH=os.path.join(CUDA, "lib64") + ":" + os.environ.get("LD_LIBRARY_PATH", ""))
    r = subprocess.run([exe], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "C-HOST OK" in r.stdout
