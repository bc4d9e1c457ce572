"""Host-side check of the index arithmetic of the 2^16-state backward kernels: the kernels' own constexpr
functions (butterfly <-> thread/slot assignment and its step-to-step dependences, in-place slot function and its bank
spread) compiled for the host and run exhaustively.  Needs nvcc, no GPU."""
import shutil
import subprocess
import sys
from pathlib import Path

import pytest

HERE = Path(__file__).resolve().parent


@pytest.mark.skipif(shutil.which("nvcc") is None, reason="nvcc not available")
def test_backward_kernel_layouts(tmp_path):
    exe = tmp_path / "layout_check"
    build = subprocess.run(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", "-O1",
                            str(HERE / "layout_check.cu"), "-o", str(exe)], capture_output=True, text=True)
    assert build.returncode == 0, build.stdout + build.stderr
    run = subprocess.run([str(exe)], capture_output=True, text=True)
    sys.stdout.write(run.stdout)
    assert run.returncode == 0 and "layouts ok" in run.stdout, run.stdout + run.stderr
