"""The C ABI from plain C: `include/gac.h` compiles as C99 with gcc, and a C
program (tests/c_abi_caller.c: no Python, C++ or torch in its process) pushes
the hand-derived worked examples through gac_init / gac_stats / gac_project."""
import os
import shutil
import subprocess

import pytest

from paper_2603_01501_b200 import binding as gb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def _compile(tmp_path, link: bool):
    exe = str(tmp_path / ("c_abi_caller" if link else "c_abi_caller.o"))
    cmd = ["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
           "-isystem", os.path.join(CUDA, "include"), os.path.join(ROOT, "tests", "c_abi_caller.c"), "-o", exe]
    if link:
        libdir = os.path.dirname(gb.LIB_PATH)
        cmd += ["-L", libdir, "-lgac_b200", "-L", os.path.join(CUDA, "lib64"), "-lcudart", "-lm",
                "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(CUDA, "lib64")]
    else:
        cmd.insert(1, "-c")
    out = subprocess.run(cmd, capture_output=True, text=True)
    assert out.returncode == 0, out.stderr
    return exe


@pytest.mark.skipif(shutil.which("gcc") is None, reason="needs gcc")
def test_header_and_caller_compile_as_c99(tmp_path):
    _compile(tmp_path, link=False)


@pytest.mark.gpu
@pytest.mark.skipif(shutil.which("gcc") is None, reason="needs gcc")
def test_plain_c_caller_reproduces_the_worked_examples(tmp_path):
    exe = _compile(tmp_path, link=True)
    out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.strip() == "ok"
