"""The kernels' index arithmetic at the largest admitted shapes, walked on the host (no GPU): grid-stride
loops end, ceilings do not wrap, the last work unit maps to the last elements.  See index_arithmetic_check.cpp."""
import os
import subprocess


def test_index_arithmetic_at_the_admitted_maxima(tmp_path):
    here = os.path.dirname(os.path.abspath(__file__))
    exe = tmp_path / "index_check"
    subprocess.run(["g++", "-O2", "-std=c++17", "-Wall", "-Wextra", "-Werror", os.path.join(here, "index_arithmetic_check.cpp"),
                    "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr
