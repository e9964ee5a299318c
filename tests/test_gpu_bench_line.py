"""The benchmark's JSON line, on a small workload: every key of the contract is present and
consistent (own arm and reference arm)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *extra],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-3000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, "exactly one JSON line expected"
    return json.loads(lines[0])


def test_own_arm_line():
    j = _run("--workload", "lsq_4m", "--steps", "3", "--warmup", "3", "--cpu-elems", "131072")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config", "roofline",
                "cpu_baseline", "e2e", "gpu_launches", "clocks", "encode", "decode", "message"):
        assert key in j, key
    assert j["metric"] == "codec_step_throughput" and j["unit"] == "GB/s" and j["value"] > 0
    assert j["n_gpus"] == 1 and j["steps"] == 3 and j["warmup"] >= 3 and j["scaling"] == "weak"
    assert j["vs_baseline"] is None and j["dtype"] == "f32" and j["data"] == "synthetic"
    assert j["config"]["workload"] == "lsq_4m" and "model" not in j["config"]
    rf = j["roofline"]
    assert rf["bound"] == "hbm" and rf["unit"] == "GB/s" and rf["peak"] > 0
    assert abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9
    assert j["gpu_launches"] == 2 * 3                       # one batched encode + one decode per step
    cb = j["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] == 1 and cb["value"] > 0 and "sample" in cb
    e2e = j["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] == 8 * 4194304 * 4
    assert e2e["d2h_bytes_per_step"] == 4194304 * 4 and e2e["value"] < j["value"]
    assert set(j["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    m = j["message"]
    assert m["entropy_bound_bits_per_entry"] <= m["fixed_bits_per_entry"] + 1e-9
    # the receiver kernel: timed inside the step and by itself, against both of its roofs
    dec = j["decode"]
    assert dec["ms_per_launch"] > 0 and dec["alone"]["ms_per_launch"] > 0
    dr = j["decode_roofline"]
    assert dr["bound"] == "hbm" and abs(dr["frac"] - dr["achieved"] / dr["peak"]) < 1e-9
    if dr["issue"] is not None:
        assert dr["issue"]["bound"] == "alu" and 0 < dr["issue"]["frac"] < 1.5
        assert dr["issue"]["issue_slots_per_code"] == pytest.approx(1 + 1 / 7 + 2)    # r = 3
    if (os.cpu_count() or 1) > 1:
        ca = j["cpu_baseline_all_cores"]
        assert ca["kind"] == "oracle" and ca["cores"] == min(8, os.cpu_count()) and ca["value"] > 0
    assert "sweep" not in j                                 # only the default workload carries it
    assert dec["length_ladder"] is None                     # shorter than two rounds of long-vector tiles
    gr = j["graph_replay"]                                  # an L2-resident workload: also as one CUDA graph
    assert gr["steps_per_graph"] == 3 and 0 < gr["ms_per_step"] <= j["ms_per_step"] * 1.5 and gr["GB/s"] > 0


def test_receiver_length_ladder_on_a_mid_size_workload():
    j = _run("--workload", "resnet50", "--steps", "3", "--warmup", "3", "--no-e2e", "--no-cpu",
             "--no-message")
    lad = j["decode"]["length_ladder"]
    assert lad["rounds"] == [1, 2, 3, 4] and lad["entries_per_round"] % 30720 == 0
    assert "graph_replay" not in j                          # larger than L2: the plain loop is the measure
    for name in ("ring", "warp"):
        k = lad[name]
        assert len(k["us"]) == 4 and all(u > 0 for u in k["us"])
        assert k["us"][-1] > k["us"][0] and k["us_per_round"] > 0 and k["per_round_GB/s"] > 0
    j = _run("--workload", "resnet50", "--steps", "3", "--no-e2e", "--no-cpu", "--no-message", "--no-ladder")
    assert j["decode"]["length_ladder"] is None
