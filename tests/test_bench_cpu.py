"""Host logic of bench.py that needs no GPU: repeat sizing, the spread record, the clock sampler's windows, the
byte model of a sweep-kernel launch, the JSON line of the reference arm."""
import importlib.util
import json
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest

from paper_2608_15473_b200 import workloads as wl

ROOT = Path(__file__).resolve().parents[1]
spec = importlib.util.spec_from_file_location("qf_bench", ROOT / "bench.py")
bench = importlib.util.module_from_spec(spec)
spec.loader.exec_module(bench)


def test_repeats_cover_the_target_load_and_stay_in_bounds():
    assert bench.n_repeats(0.3, 20) == int(np.ceil(bench.TARGET_LOAD_MS / 6.0))
    assert bench.n_repeats(50.0, 20) == bench.MIN_REPEATS           # long steps: the minimum
    assert bench.n_repeats(0.001, 1) == bench.MAX_REPEATS           # tiny steps: capped
    for est, k in ((0.3, 20), (0.6, 20), (1.2, 20), (0.19, 5)):
        r = bench.n_repeats(est, k)
        assert bench.MIN_REPEATS <= r <= bench.MAX_REPEATS and r * est * k >= min(bench.TARGET_LOAD_MS, r * est * k)


def test_spread_reports_median_extremes_and_separates_clock_from_kernel():
    # time inversely proportional to the clock: time x clock is flat, correlation -1
    mhz = [1965.0, 1900.0, 1850.0, 1800.0, 1965.0, 1930.0, 1870.0]
    ms = [590.0 / c for c in mhz]
    rec = bench.spread(ms, mhz)
    assert rec["repeats"] == 7 and rec["median_ms"] == pytest.approx(float(np.median(ms)))
    assert rec["min_ms"] == pytest.approx(min(ms)) and rec["max_ms"] == pytest.approx(max(ms))
    assert rec["ms_x_mhz_rel_spread"] < 1e-9 and rec["corr_ms_vs_mhz"] < -0.99
    assert rec["fastest_repeat_sm_mhz"] == 1965.0 and rec["slowest_repeat_sm_mhz"] == 1800.0
    # a kernel-side spread at a steady clock: the product varies as much as the time does
    rec = bench.spread([0.30, 0.31, 0.32, 0.30, 0.33, 0.31, 0.30], [1965.0] * 7)
    assert rec["ms_x_mhz_rel_spread"] == pytest.approx(0.03 / 0.31, rel=1e-6) and "corr_ms_vs_mhz" not in rec
    # no clock samples at all
    rec = bench.spread([1.0, 2.0, 3.0], [None, None, None])
    assert rec["median_ms"] == 2.0 and rec["per_repeat_sm_mhz"] == [None, None, None]


def test_clock_sampler_windows():
    s = bench.ClockSampler.__new__(bench.ClockSampler)
    s.samples = [(0.0, 1000.0), (1.0, 1100.0), (2.0, 1200.0), (3.0, 1300.0), (10.0, 1900.0)]
    s.reasons, s.max_mhz, s.power_w, s._nvml = {"sw_power_cap"}, 1965.0, [500.0, 610.0], None
    assert s.window(0.5, 2.5) == 1150.0                  # median of the samples inside
    assert s.window(4.0, 5.0) == 1300.0                  # none inside: the nearest
    summ = s.summary([(0.0, 1.0), (9.0, 11.0)])
    assert summ["sm_mhz"] == 1100.0 and summ["samples"] == 3 and summ["reasons"] == ["sw_power_cap"]
    assert summ["sm_max_mhz"] == 1965.0 and summ["power_w_max"] == 610.0


def test_sweep_kernel_bytes_follow_the_byte_model():
    w = wl.config3(seed=2, batch=4, hi=5000)
    tok = w.swept_tokens()
    n_sh = int(w.shard_counts.sum())
    want = tok * 4096 + 4 * ((tok + 15) // 16) + 4 * 32 * 128 * 2 + n_sh * 32 * 130 * 4
    assert bench.sweep_kernel_bytes(w) == want
    # the whole pass adds what the merge reads and writes
    assert w.algorithmic_bytes() == want + n_sh * 32 * 129 * 4 + 4 * 32 * 129 * 4


def test_reference_arm_prints_one_line_with_the_cuda_arms_config():
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--workload", "1",
                          "--steps", "1", "--warmup", "3"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == "GB/s" and d["higher_is_better"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["sample"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]

    class A:
        workload, seed, kv_layout = 1, 0, "hnd"
    assert d["config"] == bench.config_record(A, wl.config1(seed=0), 1)
