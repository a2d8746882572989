"""bench.py on a small case: the one JSON line carries every key its readers rely on, with sane values."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_logits_in_line_small_case():
    d = run_bench("--workload", "C2s", "--steps", "5", "--warmup", "3")
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert k in d, k
    assert d["metric"] == "policy_loss_fwd_bwd_tokens_per_s" and d["unit"] == "tokens/s" and d["n_gpus"] == 1
    assert d["steps"] == 5 and d["warmup"] >= 3 and d["higher_is_better"] is True and d["scaling"] == "weak"
    assert d["vs_baseline"] is None and d["data"] == "synthetic" and "workload" in d["config"]
    assert d["gpu_launches"] > 0 and d["value"] > 0
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and 0.3 < r["frac"] < 1.2
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["traffic"] is None or r["traffic"] >= r["algorithmic_bytes_per_launch"]
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and e["value"] < d["value"]
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["sample"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert d["skip_zero_rows"]["streamed_rows"] <= d["skip_zero_rows"]["rows"]
    assert 0.5 < d["token_logprobs"]["roofline"]["frac"] < 1.2


def test_lmhead_line_small_case():
    d = run_bench("--workload", "C5s", "--steps", "2", "--warmup", "3", "--no-cpu-baseline")
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and 0.2 < r["frac"] < 1.2
    assert d["dtype"] == "bf16" and d["gpu_launches"] > 0 and d["e2e"]["value"] > 0
    assert d["config"]["rows_worked_on"]["backward"] <= d["config"]["rows"]


def test_single_thread_oracle_figure_and_nominal_fractions_are_reported():
    d = run_bench("--workload", "C2s", "--steps", "3", "--warmup", "3", "--no-e2e")
    c = d["cpu_baseline"]
    assert c["single_thread"]["cores"] == 1 and c["single_thread"]["value"] > 0
    r = d["roofline"]
    assert r["kernel"].startswith("row_stream_kernel") and 0 < r["frac_nominal"] < r["frac"]


@pytest.mark.parametrize("workload,rows", [("C3", 4200), ("C4", 3000)])
def test_slab_legs_of_the_pool_and_gate_shapes(workload, rows):
    """One slab of the PRP-pool shape (config 3) and of the XGRPO + SGT shape (config 4), cut small."""
    d = run_bench("--workload", workload, "--steps", "3", "--warmup", "3", "--slab-rows", str(rows))
    cfg, r = d["config"], d["roofline"]
    assert cfg["rows"] <= rows and cfg["rows"] >= 1024 and cfg["step_rows"] > 500_000
    assert r["bound"] == "hbm" and 0 < r["frac"] < 1.2 and r["rows_read"] <= cfg["rows"]
    assert d["e2e"] is None and d["cpu_baseline"] is None       # the legs beside the headline carry neither
    if workload == "C4":
        assert cfg["nll_rows_in_slab"] >= 0 and cfg["selected_peer_rollouts_in_step"] > 0
