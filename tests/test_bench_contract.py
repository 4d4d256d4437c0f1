"""bench.py prints ONE JSON line with the agreed keys: the library arm on a GPU (tiny workload, a few
steps), the reference arm (the CPU oracle) without one."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CONFIG_KEYS = {"workload", "B", "D", "M", "H", "V", "rows", "policy", "parallelism", "l2"}
COMMON = ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
          "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "cpu_baseline")


def _run(*args):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, res.stdout
    return json.loads(lines[0])


def test_reference_arm_line():
    d = _run("--impl", "reference", "--config", "tiny", "--steps", "2", "--warmup", "3")
    for k in COMMON:
        assert k in d, k
    assert d["impl"] == "reference" and d["gpu_launches"] == 0 and d["dtype"] == "f64"
    assert d["value"] > 0 and d["config"]["workload"] == "tiny" and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["sample"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["e2e"]["value"] == d["value"] == d["cpu_baseline"]["value"]
    assert set(d["config"]) == CONFIG_KEYS and d["config"]["rows"] == 128


def test_default_run_names_the_largest_workload_and_nests_the_small_one():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.DEFAULT_WORKLOADS == ("batched_serving", "single_request")
    big = bench.config_dict(bench.resolve_config("batched_serving"), 1)
    assert big["rows"] == 8192 and set(big) == CONFIG_KEYS


@pytest.mark.gpu
def test_library_arm_line():
    d = _run("--config", "tiny", "--steps", "50", "--warmup", "3")
    for k in COMMON + ("clocks", "roofline"):
        assert k in d, k
    assert "impl" not in d and d["n_gpus"] == 1 and d["steps"] == 50 and d["warmup"] == 3
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["data"] == "synthetic"
    assert d["gpu_launches"] == 2 * d["steps"]                      # two launches per step
    assert d["value"] > 0 and abs(d["value"] - 128 / (d["ms_per_step"] * 1e-3)) < 1e-6 * d["value"]
    r = d["roofline"]
    assert r["bound"] in ("hbm", "tensor") and r["unit"] in ("GB/s", "TFLOP/s")
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and "traffic" in r and r["kernel_ms"] > 0
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 128 * 256 * 2 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < d["value"]                                   # copies are inside its timed region
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["value"] > 0 and c["cores"] >= 1 and c["sample"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert set(d["config"]) == CONFIG_KEYS                           # the same keys as the reference arm's
    t = d["timing"]
    assert t["repeats"] >= 3 and t["steps_per_repeat"] == 50 and t["timed_seconds"] >= 1.0
    assert t["ms_per_step_min"] <= d["ms_per_step"] <= t["ms_per_step_max"]
    assert r["kernel"] == "confidence_tc_kernel" and "traffic_source" in r
