"""The tile walk of the tensor-core kernels, replayed on the CPU: tests/host_tile_plan.cu compiles the
kernels' own host/device helpers (tile geometry, tile order, the per-CTA tile cursor, the carried-partials
slot arithmetic) for the host and checks that every tile is visited exactly once, in the order the carried
triples rely on, and that the merge pass is told exactly the slots that were written."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", shutil.which("nvcc")):
        if cand and os.path.exists(cand):
            return cand
    return None


def test_tile_walk_on_the_host(tmp_path):
    nvcc = _nvcc()
    if nvcc is None:
        pytest.skip("nvcc not found")
    exe = tmp_path / "host_tile_plan"
    src = os.path.join(ROOT, "tests", "host_tile_plan.cu")
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O1", "-std=c++17", "-I",
                    os.path.join(ROOT, "include"), "-I", os.path.join(ROOT, "paper_2605_15609_b200", "csrc"),
                    "-o", str(exe), src, "-lcudart"], check=True, capture_output=True, text=True)
    res = subprocess.run([str(exe)], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and res.stdout.strip().startswith("ok"), res.stdout[-3000:] + res.stderr[-1000:]
