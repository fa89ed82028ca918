"""bench.py's own arm on a reduced workload: the JSON line carries every key the contract names."""
import json
import os
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
    assert j["gpu_launches"] == 4 and j["vs_baseline"] is None and "workload" in j["config"]      # one launch per step
    assert j["build_flavor"] == "product" and j["edq_fault"] == 0
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
    assert c["config0_whole"]["value"] > 0


def test_sharded_flow_with_two_emulated_ranks_through_the_benchmarks_own_code():
    # the flow the N-rank run times (one parameter set cut over the ranks, theta stored into every rank's full
    # copy by the step kernel, EDQ records combined), here with both ranks on this GPU one after the other
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--sharded-selfcheck", "--layers", "1", "--steps", "2"],
                       cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert p.returncode == 0, p.stderr[-2000:]
    j = json.loads([l for l in p.stdout.splitlines() if l.startswith("{")][-1])["sharded_selfcheck"]
    assert j["ok"] and j["theta_copies_bitwise_equal_to_unsharded"] and j["edq_max_relative_difference"] <= 1e-5
    assert j["theta_bytes_sent_per_rank_per_step"] == j["params_total"]          # 2 B x half of the parameters x 1 peer


def test_sharded_leg_as_two_processes_on_this_gpu():
    # what `bench.py --gpus N` runs for its "sharded" record, with the two ranks as separate processes on this
    # one GPU: CUDA IPC handles exchanged, each rank maps the other's theta copy and its step kernel stores
    # into it; the EDQ sums travel over gloo here (NCCL needs a GPU per rank).  The ranks' kernels never wait
    # on one another.  Afterwards both processes hold the same full theta.
    # launched the way rank 0 of an N-rank run launches it (child processes with their own rendezvous)
    import argparse
    sys.path.insert(0, str(ROOT))
    import bench
    args = argparse.Namespace(steps=3, warmup=2, layers=0, lib=None, sharded_backend="gloo", sharded_one_device=True)
    os.environ.setdefault("MASTER_PORT", "29526")
    j = bench.run_sharded_children(args, 2)
    assert "unavailable" not in j, j
    assert j["ranks"] == 2 and j["copies_agree"] and j["edq_fault"] == 0 and j["edq"] > 0
    assert j["params_total"] == 262_148_096 and abs(j["params_per_rank"] - j["params_total"] / 2) <= 8
    assert j["theta_bytes_sent_per_rank_per_step"] == 2 * j["params_per_rank"]


@pytest.mark.parametrize("config", [0, 1, 2])
def test_other_configurations_print_contract_lines(config):
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--config", str(config)], cwd=ROOT, capture_output=True,
                       text=True, timeout=900)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [json.loads(l) for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == {0: 3, 1: 1, 2: 2}[config]
    for j in lines:
        assert j["unit"] == "params/s" and j["value"] > 0 and j["gpu_launches_per_step"] == 1
        assert j["roofline"]["bound"] == "hbm" and 0 < j["roofline"]["frac"] < 1.3
