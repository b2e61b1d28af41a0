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


def test_default_workload_line():
    d = run_bench("--steps", "24", "--warmup", "3", "--cpu-rows", "4")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 24 and d["warmup"] == 3 and d["higher_is_better"] is True
    assert d["vs_baseline"] is None and d["dtype"] == "bf16" and d["data"] == "synthetic" and d["scaling"] == "weak"
    cfg = d["config"]
    assert cfg["workload"].startswith("cfg1a") and cfg["draft_rows"] == 32 and "model" not in cfg
    # value = draft rows per second of the whole step
    assert d["value"] == pytest.approx(cfg["draft_rows"] / (d["ms_per_step"] * 1e-3), rel=1e-6)
    assert d["gpu_launches"] == 7 * d["steps"]                      # 2 x (projection + merge) + commit + select + verify
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["kernel"] == "pvf_score_stream_kernel"
    assert r["frac"] == pytest.approx(r["achieved"] / r["peak"], rel=1e-9)
    assert r["achieved"] == pytest.approx(r["algorithmic_bytes_per_launch"] / (r["avg_launch_us"] * 1e-6) / 1e9, rel=1e-6)
    assert 0.5 < r["frac"] < 1.1 and r["traffic"] is not None and r["traffic"] >= r["algorithmic_bytes_per_launch"]
    # two projection launches per step cannot take longer than the step that contains them
    assert 2 * r["avg_launch_us"] * 1e-3 < d["ms_per_step"]
    e = d["e2e"]
    assert e["unit"] == d["unit"] and e["h2d_bytes_per_step"] > 2 * 30 * 4096 * 2 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < d["value"]                                   # host copies inside the timed region
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["unit"] == d["unit"]
    assert isinstance(d["clocks"]["reasons"], list)
    p = d["parity"]
    assert p["max_conf_err"] <= 1e-3 and p["max_ent_err"] <= 1e-3 and p["token_mismatches_outside_near_ties"] == 0


def test_ridge_workload_reports_the_kernel_mix():
    d = run_bench("--workload", "cfg2", "--steps", "12", "--warmup", "3", "--no-cpu-baseline")
    r = d["roofline"]
    assert set(r["kernel"].split("+")) == {"pvf_score_gemm_pair_kernel", "pvf_score_swap_pair_kernel"}
    assert d["config"]["draft_rows"] == 232 and d["config"]["verify_rows"] == 181
    assert r["traffic"] is not None and d["gpu_launches"] == 7 * d["steps"]
