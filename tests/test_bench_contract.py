"""bench.py prints one JSON line with the keys its callers rely on: checked on the small
configuration (the reference arm needs no GPU; the product arm is a GPU test)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, timeout=600):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, capture_output=True,
                       text=True, timeout=timeout)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, lines
    return json.loads(lines[0])


def test_reference_arm_line_on_the_small_config():
    j = _run(["--impl", "reference", "--workload", "cfg1", "--steps", "2", "--warmup", "1"])
    assert j["impl"] == "reference" and j["unit"] == "GB/s" and j["higher_is_better"] is True
    assert j["steps"] == 2 and j["warmup"] == 1 and j["value"] > 0 and j["ms_per_step"] > 0
    assert j["dtype"] == "f64" and j["data"] == "synthetic" and j["vs_baseline"] is None
    assert "cfg1" in j["config"]["workload"]
    cb = j["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == pytest.approx(j["value"]) and cb["sample"]
    assert j["e2e"] == {"value": j["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


@pytest.mark.gpu
def test_product_arm_line_on_the_small_config():
    j = _run(["--workload", "cfg1", "--steps", "4", "--warmup", "3", "--ref-positions", "4096",
              "--configs", "cfg2,sweep_N4_c16_d2^26"])
    with open(os.path.join(ROOT, "BASELINE.json")) as f:
        assert j["metric"] == json.load(f)["metric"]
    assert j["unit"] == "GB/s" and j["n_gpus"] == 1 and j["steps"] == 4 and j["warmup"] == 3
    assert j["higher_is_better"] is True and j["scaling"] == "weak" and j["vs_baseline"] is None
    assert j["dtype"] == "f32" and j["data"] == "synthetic" and "cfg1" in j["config"]["workload"]
    N, c = 4, 8
    assert j["gpu_launches"] == 4 * (c + N - 2 + 2)                       # K x (encode + L rounds + decode)
    assert j["value"] > 0 and j["ms_per_step"] > 0
    rf = j["roofline"]
    assert rf["bound"] == "hbm" and rf["unit"] == "GB/s" and rf["peak"] > 1000
    assert rf["frac"] == pytest.approx(rf["achieved"] / rf["peak"])
    assert "traffic" in rf and set(rf["per_kernel"]) == {"encode", "round_kernel", "decode"}
    cb = j["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] > 0 and cb["unit"] == "GB/s" and cb["sample"]
    e = j["e2e"]
    d = 65536
    assert e["h2d_bytes_per_step"] == N * d * 4 and e["d2h_bytes_per_step"] == N * d * 4 and e["value"] > 0
    assert e["value"] != j["value"]
    ck = j["clocks"]
    assert ck is None or {"sm_mhz", "sm_max_mhz", "reasons"} <= set(ck)
    assert j["one_call"]["ms_per_step"] > 0
    # DRAM-based fraction next to the algorithmic one
    assert rf["dram_frac"] == pytest.approx(rf["traffic"] / (rf["avg_launch_ms"] * 1e-3) / 1e9 / rf["peak"])
    # parity next to the number: GPU against the oracle on sampled positions, outside the timed region
    par = j["parity"]
    assert par["sampled_positions"] == 4096 and par["rel_l2_Y"] < 2e-6
    assert par["kappa_times_2^-24"] == pytest.approx(par["kappa_M"] * 2.0 ** -24)
    assert par["rel_l2_out"] < 4 * par["kappa_times_2^-24"]
    assert par["end_to_end_residual_over_bound"] <= 1.0 and par["decode_residual_over_bound"] <= 1.0
    # the other configurations, timed the same way
    cf = j["configs"]
    assert set(cf) == {"cfg2", "sweep_N4_c16_d2^26"}
    for key, N2, c2 in (("cfg2", 4, 16), ("sweep_N4_c16_d2^26", 4, 16)):
        e2 = cf[key]
        assert "error" not in e2 and "skipped" not in e2, e2
        assert e2["gpu_launches"] == e2["steps"] * (c2 + N2 - 2 + 2)
        assert e2["ms_per_step"] > 0 and e2["frac"] == pytest.approx(e2["value"] / rf["peak"])
        assert set(e2["per_kernel_GBps"]) == {"encode", "round_kernel", "decode"}
