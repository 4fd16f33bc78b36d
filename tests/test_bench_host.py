"""Host-side pieces of bench.py that need no GPU: the traffic figure stays tied to the kernel source it was measured
with, the clock/power sampler parses what nvidia-smi prints (and says so when there is none), and the peaks come
from the measured file when it is there and from the stated fallback otherwise."""
import json
import os
import time

import bench


def test_traffic_figure_belongs_to_the_committed_kernel_source():
    # bench.py reports DRAM traffic from an ncu capture; the figure is only valid for the source it was taken with.
    # A kernel change without a new capture must show up here, not as a stale number in the bench line.
    assert bench.kernel_traffic() == bench.NCU_TRAFFIC["bytes_per_launch"]
    assert 1e9 < bench.NCU_TRAFFIC["bytes_per_launch"] < 1e11


def test_sampler_parses_rows_and_windows_them(monkeypatch):
    monkeypatch.setattr(bench, "_POWER_FIELD", "power.draw")
    s = bench.ClockSampler(0)

    class Done:
        def terminate(self): pass
        def wait(self, timeout=None): return 0
        def kill(self): pass
    s.proc = Done()
    t = time.time()
    s.rows = [(t - 10.0, "1965, 1965, 300.0, Not Active, Not Active, Not Active, Not Active"),      # before the window
              (t + 0.1, "1400, 1965, 990.5, Not Active, Not Active, Not Active, Active"),
              (t + 0.2, "1300, 1965, 1001.0, Not Active, Not Active, Not Active, Active"),
              (t + 0.3, "1350, 1965, [N/A], Not Active, Not Active, Not Active, Active"),             # unparsable power: row skipped
              (t + 0.4, "garbage")]
    out = s.stop(t, t + 1.0)
    assert out["sm_mhz"] == 1350.0 and out["sm_max_mhz"] == 1965.0 and out["samples"] == 2      # median of 1400 and 1300
    assert out["power_w_max"] == 1001.0 and abs(out["power_w_median"] - 995.75) < 1e-9
    assert out["reasons"] == ["sw_power_cap"]


def test_sampler_without_nvidia_smi_reports_it(monkeypatch):
    monkeypatch.setattr(bench, "_POWER_FIELD", "power.draw")
    s = bench.ClockSampler(0)
    out = s.stop()
    assert out["sm_mhz"] is None and out["reasons"] == ["nvidia-smi unavailable"]


def test_peaks_come_from_the_measured_file_or_the_fallback(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    peaks, src = bench.load_peaks()
    assert src == "fallback" and peaks == bench.FALLBACK_PEAKS
    d = {k: 1.0 + i for i, k in enumerate(bench.FALLBACK_PEAKS)}
    (tmp_path / "MEASURED_PEAKS.json").write_text(json.dumps(d))
    peaks, src = bench.load_peaks()
    assert src == "measured" and peaks == d
