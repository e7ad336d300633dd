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


def test_paged_from_packed_keeps_every_row_where_the_table_says():
    """The page pool built from a packed batch holds, behind its block table, exactly the packed
    rows of every sequence; rows of a last page past the end of its sequence, and the spare
    pages, hold NaN."""
    import torch
    from paper_2410_16663_b200 import inputs as synth

    lens = (300, 1, 128, 517)
    total = sum(lens)
    k = torch.arange(total * 2 * 4, dtype=torch.float32).reshape(total, 2, 4).to(torch.float16)
    v = -k
    page = 128
    kp, vp, table = synth.paged_from_packed(k, v, lens, page, seed=3, spare_pages=2, poison=True)
    need = [(n + page - 1) // page for n in lens]
    assert kp.shape == (sum(need) + 2, page, 2, 4) and table.shape == (len(lens), max(need))
    used = [int(table[b, pg]) for b in range(len(lens)) for pg in range(need[b])]
    assert len(set(used)) == len(used) and min(used) >= 0 and max(used) < kp.shape[0]
    base = 0
    for b, n in enumerate(lens):
        for j in range(n):
            pg = int(table[b, j // page])
            assert torch.equal(kp[pg, j % page], k[base + j]) and torch.equal(vp[pg, j % page], v[base + j])
        assert (table[b, need[b]:] == -1).all()
        tail = n % page
        if tail:
            last = int(table[b, need[b] - 1])
            assert torch.isnan(kp[last, tail:].float()).all() and torch.isnan(vp[last, tail:].float()).all()
        base += n
    spare = sorted(set(range(kp.shape[0])) - set(used))
    assert len(spare) == 2 and torch.isnan(kp[spare].float()).all()
