"""Host-side logic of the CUDA sources that can run without a GPU: compiled as host code with
nvcc (the image has it; no device is touched) and executed."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


@pytest.mark.skipif(not os.path.exists(NVCC) and shutil.which("nvcc") is None, reason="nvcc not found")
def test_fastdiv_matches_integer_division(tmp_path):
    nvcc = NVCC if os.path.exists(NVCC) else shutil.which("nvcc")
    exe = str(tmp_path / "fastdiv_check")
    src = os.path.join(ROOT, "tests", "host_checks", "fastdiv_check.cu")
    subprocess.run([nvcc, "-std=c++17", "-O2", "-gencode", "arch=compute_100a,code=sm_100a", src, "-o", exe],
                   check=True, timeout=600)
    out = subprocess.run([exe], capture_output=True, text=True, timeout=600)
    sys.stdout.write(out.stdout)
    assert out.returncode == 0, out.stdout[-2000:]
    assert out.stdout.strip().startswith("OK")
