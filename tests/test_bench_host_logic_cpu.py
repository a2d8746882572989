"""Host-side arithmetic of bench.py that needs no GPU: the per-product time x clock table and the roofline lookups."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


class FakeClocks:
    """Samples every millisecond: 1,000 MHz / 900 W during the first 10 ms, 1,500 MHz / 1,000 W afterwards."""

    def __init__(self):
        self.timed = [(100.0 + i * 1e-3, 1000 if i < 10 else 1500, 900.0 if i < 10 else 1000.0) for i in range(40)]

    median_between = bench.ClockSampler.median_between


def test_per_product_table_attributes_clock_samples_to_the_launches_that_ran_under_them():
    kinds = ["forward", "dZ", "dZ"]
    flops = {"forward": 2.0e12, "dZ": 1.0e12}
    offsets_ms = [0.0, 12.0, 20.0]          # after t_start = 100.0 s
    durations_ms = [8.0, 4.0, 6.0]
    t = bench.per_product_table(kinds, flops, offsets_ms, durations_ms, 100.0, FakeClocks(), sms=100)
    f, d = t["forward"], t["dZ"]
    assert f["launches"] == 1 and d["launches"] == 2
    assert abs(f["ms"] - 8.0) < 1e-12 and abs(d["ms"] - 5.0) < 1e-12
    assert f["sm_mhz"] == 1000 and d["sm_mhz"] == 1500 and f["watts"] == 900.0 and d["watts"] == 1000.0
    assert abs(f["tflops"] - 250.0) < 1e-9 and abs(d["tflops"] - 200.0) < 1e-9
    # flops / (seconds x Hz x SMs)
    assert abs(f["flop_per_clk_per_sm"] - 2.0e12 / (8e-3 * 1000e6 * 100)) < 1e-9
    assert abs(d["flop_per_clk_per_sm"] - 1.0e12 / (5e-3 * 1500e6 * 100)) < 1e-9


def test_per_product_table_without_samples_reports_no_clock():
    empty = FakeClocks()
    empty.timed = []
    t = bench.per_product_table(["dW"], {"dW": 1.0e12}, [0.0], [1.0], 0.0, empty, sms=148)
    assert t["dW"]["sm_mhz"] is None and t["dW"]["flop_per_clk_per_sm"] is None and t["dW"]["tflops"] == 1000.0


def test_traffic_figures_are_keyed_by_kernel_vocabulary_and_batch_kind():
    keys = set(bench.DRAM_BYTES_PER_TOKEN)
    assert ("row_stream_kernel", 151936, "half-live") in keys and ("row_stream_kernel", 151936, "all-live") in keys
    for k, v in bench.DRAM_BYTES_PER_TOKEN.items():
        alg = 2 * k[1] * 2
        assert v is None or alg <= v < 1.3 * alg, k         # measured traffic is at least the algorithmic bytes
    assert bench.DRAM_BYTES_PER_TOKEN.get(("row_general_kernel", 151936, "half-live")) is None


def test_measured_peaks_fall_back_to_the_stated_figures(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    p = bench.measured_peaks()
    assert p["source"] == "fallback" and p["hbm_gbs"] == 6650.0 and p["bf16_tflops"] == 1590.0
    (tmp_path / "MEASURED_PEAKS.json").write_text('{"hbm_gbs": 6000, "bf16_tflops": 1500, "bf16_tflops_sustained": 1300}')
    p = bench.measured_peaks()
    assert p["source"] == "measured" and p["hbm_gbs"] == 6000.0 and p["bf16_tflops_sustained"] == 1300.0
