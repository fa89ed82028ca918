"""bench.py's own arm on a reduced workload: the JSON line carries every key the contract names."""
import json
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parents[1]


def test_bench_line_on_the_reduced_workload():
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--layers", "0", "--steps", "4", "--warmup", "3",
                        "--cpu-seconds", "2"], cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["metric"] == "collage_adamw_step_params_per_sec" and j["unit"] == "params/s" and j["dtype"] == "bf16"
    assert j["n_gpus"] == 1 and j["steps"] == 4 and j["warmup"] == 3 and j["scaling"] == "weak" and j["data"] == "synthetic"
    assert j["gpu_launches"] == 8 and j["vs_baseline"] is None and "workload" in j["config"]
    r = j["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert 0.9 < r["traffic"] / r["algorithmic"] < 1.1
    assert abs(r["achieved"] - 22 * j["config"]["params_per_gpu"] / (r["kernel_ms"] * 1e-3) / 1e9) < 1e-6 * r["achieved"]
    assert set(j["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    e = j["e2e"]
    assert e["value"] > 0 and e["unit"] == "params/s" and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < j["value"]                      # host copies are inside its timed region
    c = j["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["value_one_thread"] > 0
