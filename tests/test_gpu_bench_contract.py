"""bench.py on one GPU, a short run: the JSON line carries every key of the measurement contract and the numbers
are consistent with one another."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*flags):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], cwd=ROOT, capture_output=True,
                         text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def launches_fit_the_step(r, ms_per_step):
    """One launch of every timed row count (draft pass, verification pass) cannot take longer than the step
    that contains them."""
    per = r["per_row_count"]
    assert len(per) >= 1 and all(x["launches"] >= 1 for x in per)
    assert sum(x["avg_launch_us"] for x in per) * 1e-3 <= ms_per_step * 1.0005


def test_default_workload_line():
    d = run_bench("--steps", "24", "--warmup", "3", "--cpu-rows", "4")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 24 and d["warmup"] == 3 and d["higher_is_better"] is True
    assert d["vs_baseline"] is None and d["dtype"] == "bf16" and d["data"] == "synthetic" and d["scaling"] == "weak"
    cfg = d["config"]
    assert cfg["workload"] == "cfg1a" and cfg["draft_rows"] == 32 and "model" not in cfg
    # value = draft rows per second of the whole step
    assert d["value"] == pytest.approx(cfg["draft_rows"] / (d["ms_per_step"] * 1e-3), rel=1e-6)
    assert d["gpu_launches"] == 4 * d["steps"]                      # projection + draft kernel, projection + verify kernel
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["kernel"] == "pvf_score_stream_kernel"
    assert r["frac"] == pytest.approx(r["achieved"] / r["peak"], rel=1e-9)
    assert r["achieved"] == pytest.approx(r["algorithmic_bytes_per_launch"] / (r["avg_launch_us"] * 1e-6) / 1e9, rel=1e-6)
    assert 0.5 < r["frac"] < 1.1 and r["traffic"] is not None and r["traffic"] >= r["algorithmic_bytes_per_launch"]
    # two projection launches per step cannot take longer than the step that contains them
    assert 2 * r["avg_launch_us"] * 1e-3 < d["ms_per_step"]
    launches_fit_the_step(r, d["ms_per_step"])
    # the step as a whole (decision kernels and gaps included) against the same peak
    assert r["step"]["unit"] == "GB/s" and 0.5 < r["step"]["frac"] <= r["frac"] * 1.0005
    assert r["timed_every_nth_step"] == 8 and d["repeats"] >= 20      # 24 steps of a third of a millisecond: many blocks
    assert d["clocks"]["samples"] >= 10 and d["clocks"]["sm_mhz"] > 0
    assert r["sm_cycles_per_launch"] == pytest.approx(r["avg_launch_us"] * d["clocks"]["sm_mhz"], rel=1e-9)
    for item in r["per_row_count"]:                               # the kernels' own clock: every launch of the region counted
        assert item["device_launches"] == d["steps"] * d["repeats"] and 500 < item["device_sm_mhz"] <= d["clocks"]["sm_max_mhz"] + 1
        assert item["device_sm_cycles"] == pytest.approx(item["device_kernel_us"] * item["device_sm_mhz"], rel=1e-6)
        # block 0's span starts when its wait returns: its first weight tiles were fetched before that
        assert 0.75 * item["avg_launch_us"] < item["device_kernel_us"] <= 1.02 * item["avg_launch_us"]
    e = d["e2e"]
    assert e["unit"] == d["unit"] and e["h2d_bytes_per_step"] > 2 * 30 * 4096 * 2 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < d["value"]                                   # host copies inside the timed region
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["unit"] == d["unit"]
    assert isinstance(d["clocks"]["reasons"], list)
    p = d["parity"]
    assert p["max_conf_err"] <= 1e-3 and p["max_ent_err"] <= 1e-3 and p["token_mismatches_outside_near_ties"] == 0
    # the tensor-bound regime (config 3) and the decode loop (config 4) ride on the same line
    t = d["tensor_regime"]
    assert t["workload"] == "cfg3" and t["draft_rows"] == 32768 and t["verify_rows"] > 65536 and t["status"] == 0
    tr = t["roofline"]
    assert tr["bound"] == "tensor" and tr["unit"] == "TFLOP/s" and tr["timed_every_nth_step"] == 1
    assert tr["frac"] == pytest.approx(tr["achieved"] / tr["peak"], rel=1e-9) and tr["frac"] >= 0.6
    assert tr["frac_sustained"] == pytest.approx(tr["achieved"] / tr["peak_sustained"], rel=1e-9)
    assert [x["rows"] for x in tr["per_row_count"]] == [t["draft_rows"], t["verify_rows"]]
    launches_fit_the_step(tr, t["ms_per_step"])
    assert t["value"] == pytest.approx(t["draft_rows"] / (t["ms_per_step"] * 1e-3), rel=1e-6)
    assert t["clocks"]["samples"] >= 10
    tp = t["parity"]
    assert tp["max_conf_err"] <= 1e-3 and tp["max_ent_err"] <= 1e-3 and tp["max_conf_err_verify"] <= 1e-3
    assert tp["token_mismatches_outside_near_ties"] == 0 and tp["token_mismatches_outside_near_ties_verify"] == 0
    loop = d["decode_loop"]
    for arm in ("pvf", "threshold_only"):
        a = loop[arm]
        assert a["status"] == 0 and a["all_committed"] and a["steps"] >= 8 and a["kernel_ms_per_step"] > 0
        assert 1.0 <= a["tokens_per_forward"] <= 32.0
    assert loop["pvf"]["steps"] <= loop["threshold_only"]["steps"]
    assert loop["pvf"]["scored_rows"] > loop["threshold_only"]["scored_rows"]     # the verification branches


def test_tensor_regime_launch_times_fit_their_step():
    # 8 of config 3's 64 sequences: same kernels and geometry rule, every projection launch timed
    d = run_bench("--workload", "cfg3s", "--steps", "4", "--warmup", "3", "--min-seconds", "1", "--no-cpu-baseline", "--no-graph")
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["timed_every_nth_step"] == 1 and d["config"]["draft_rows"] == 4096
    assert r["launches"] == 2 * d["steps"] and d["repeats"] >= 3      # the median block's own launches
    launches_fit_the_step(r, d["ms_per_step"])
    assert d["gpu_launches"] == 4 * d["steps"]


def test_ridge_workload_reports_the_kernel_mix():
    d = run_bench("--workload", "cfg2", "--steps", "12", "--warmup", "3", "--min-seconds", "0.5", "--no-cpu-baseline")
    r = d["roofline"]
    assert set(r["kernel"].split("+")) == {"pvf_score_gemm_pair_kernel", "pvf_score_swap_pair_kernel"}
    assert d["config"]["draft_rows"] == 232 and d["config"]["verify_rows"] == 181
    assert r["traffic"] is not None and d["gpu_launches"] == 4 * d["steps"]
