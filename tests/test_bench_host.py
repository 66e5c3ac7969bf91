"""Host-side logic of bench.py and bench_configs.py that needs no GPU: the reported block is the
median, the ncu traffic figure is dropped when the kernel sources have changed since it was taken,
and the clock sampler's windows select by timestamp."""
import json

import bench
import bench_configs


def test_median_block_is_reported():
    assert bench.median_block([3.0, 1.0, 2.0, 10.0, 2.5]) == 2.5


def test_traffic_is_null_when_the_sources_changed(tmp_path, monkeypatch):
    f = tmp_path / "traffic.json"
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(f))
    assert bench.ncu_traffic() is None                                   # no capture on record
    f.write_text(json.dumps({"csrc_hash": "stale", "dram_bytes_read": 1, "dram_bytes_write": 2}))
    assert bench.ncu_traffic() is None                                   # taken from other sources
    f.write_text(json.dumps({"csrc_hash": bench.csrc_hash(), "dram_bytes_read": 100, "dram_bytes_write": 23}))
    assert bench.ncu_traffic() == 123


def test_clock_windows_select_by_timestamp():
    s = bench_configs.ClockSampler(0)
    s.samples = [(10.0, 1500.0, 1965.0, 700.0, []), (10.5, 1800.0, 1965.0, 900.0, ["sw_power_cap"]),
                 (11.0, 1900.0, 1965.0, 950.0, [])]
    w = s.window(10.4, 11.1)
    assert w["sm_mhz"] == 1850.0 and w["samples"] == 2 and w["reasons"] == ["sw_power_cap"]
    w = s.window(10.6, 10.7)                                             # shorter than the sampling period
    assert w["samples"] == 1 and w["sm_mhz"] == 1800.0


def test_records_carry_fraction_of_peak():
    r = bench_configs.record("x", tokens=1000, nbytes=2e9, launches=1, times_ms=[2.0, 1.0, 3.0], n=2, window=(0.0, 1.0))
    peak, _ = bench_configs.measured_peak()
    assert r["ms"] == 1.0 and r["ms_min"] == 0.5 and r["ms_max"] == 1.5
    assert abs(r["algorithmic_GBps"] - 2000.0) < 1e-9 and abs(r["frac"] - 2000.0 / peak) < 1e-12
