"""The debug build of the library (the same sources compiled with PSD_DEBUG: bounds checks on every
partial-triple access, on the tile cursor's outputs and on the carried-triple table, and a check that each
stage of the shared-memory ring holds the K-slice the MMA issuer expects; a failed check reports
PSD_ERR_INTERNAL through the status word and skips the access, nothing traps) runs the shapes that reach
every path of the kernels — ragged rows and vocabularies, every tile order and band size, compacted rows,
the whole step, the give-up path — and must report nothing: the parity tests it runs demand status 0 and
the oracle's results.  It runs in a child process because the build is chosen when the package is
imported (PSD_B200_DEBUG=1)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SELECTION = ["tests/test_gpu_confidence.py::test_ragged_shapes",
             "tests/test_gpu_confidence.py::test_tile_orders_and_ragged_bands",
             "tests/test_gpu_confidence.py::test_many_rows_small_problem",
             "tests/test_gpu_confidence.py::test_single_request_config_all_rows",
             "tests/test_gpu_compact.py",
             "tests/test_gpu_timeout.py",
             "tests/test_gpu_step.py::test_step_stage_forced"]


def test_debug_build_reports_nothing_on_the_parity_cases():
    env = dict(os.environ, PSD_B200_DEBUG="1")
    probe = subprocess.run([sys.executable, "-c", "import paper_2605_15609_b200 as p; print(p.LIB_PATH)"],
                           capture_output=True, text=True, cwd=ROOT, env=env, timeout=600)
    assert probe.returncode == 0 and probe.stdout.strip().endswith("libpsd_b200_debug.so"), probe.stderr[-2000:]
    res = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", *SELECTION],
                         capture_output=True, text=True, cwd=ROOT, env=env, timeout=1500)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-1000:]
