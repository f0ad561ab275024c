"""The header is plain C and the library is usable from C alone."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def test_header_is_valid_c99():
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only",
                           "-x", "c", os.path.join(ROOT, "include", "ta.h")])


def _build(tmp_path):
    from paper_2609_40247_b200 import build
    if not os.path.exists(build.LIB):
        build.build()
    exe = str(tmp_path / "abi_example")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-O1", os.path.join(ROOT, "tests", "c", "abi_example.c"),
                           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"),
                           build.LIB, "-L", os.path.join(CUDA, "lib64"), "-lcudart",
                           "-Wl,-rpath," + os.path.dirname(build.LIB), "-Wl,-rpath," + os.path.join(CUDA, "lib64"),
                           "-o", exe])
    return exe


def test_c_example_builds(tmp_path):
    assert os.path.exists(_build(tmp_path))


@pytest.mark.gpu
def test_c_example_runs_without_python_or_allocator_callbacks(tmp_path):
    out = subprocess.run([_build(tmp_path)], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and "c abi ok" in out.stdout, out.stdout + out.stderr
