"""bench.py prints one JSON line with the agreed keys: the reference (oracle) arm on CPU,
the library arm on a GPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

COMMON = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
          "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"}


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True,
                         text=True, cwd=ROOT, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def test_reference_arm_line():
    j = _run("--impl", "reference", "--workload", "cfg2", "--steps", "1", "--warmup", "0")
    assert COMMON <= set(j) and j["impl"] == "reference" and j["unit"] == "GB/s"
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["value"] == j["value"] > 0
    assert j["e2e"]["h2d_bytes_per_step"] == 0 and j["config"]["workload"] == "cfg2"
    # the configuration is the library arm's, key for key; what the oracle was timed on is said beside it
    assert j["config"]["parallelism"] == "replicas x1" and j["config"]["n_clients_total"] == 10
    assert j["sample"]["d"] == 1 << 20 and 1 <= j["sample"]["n_clients"] <= 10


@pytest.mark.gpu
def test_library_arm_line():
    j = _run("--workload", "cfg2", "--steps", "3", "--warmup", "3")
    assert COMMON | {"roofline", "gpu_launches", "clocks", "kernels"} <= set(j)
    assert j["value"] > 0 and j["gpu_launches"] > 0 and j["dtype"] == "f32"
    r = j["roofline"]
    assert r["bound"] == "hbm" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert j["cpu_baseline"]["cores"] >= 1 and j["e2e"]["h2d_bytes_per_step"] > 10 * 2 ** 20 * 4
    assert j["status_word"] == 0 and 0 < j["nmse_vs_true_mean"] < 0.05
