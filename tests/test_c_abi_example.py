"""The C ABI from plain C: the example program compiles against include/tutti.h on any
machine, and on a GPU machine it runs and checks its own result."""
import os
import subprocess

import pytest

from paper_2605_03375_b200 import _build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
EXE = os.path.join(ROOT, "tests", "c_abi_example.bin")


def _compile():
    _build.build_library()
    pkg = os.path.join(ROOT, "paper_2605_03375_b200")
    subprocess.check_call(["/usr/local/cuda/bin/nvcc", os.path.join(ROOT, "tests", "c_abi_example.c"),
                           "-I" + os.path.join(ROOT, "include"), "-L" + pkg, "-ltutti",
                           "-Xlinker", "-rpath", "-Xlinker", pkg, "-o", EXE])


def test_c_example_compiles_against_the_header():
    _compile()
    assert os.path.exists(EXE)


@pytest.mark.gpu
def test_c_example_runs():
    _compile()
    p = subprocess.run([EXE], capture_output=True, text=True, timeout=120)
    assert p.returncode == 0, p.stdout + p.stderr
    assert p.stdout.startswith("OK restored and saved 4325376 bytes")
