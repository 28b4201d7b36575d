"""Host-side logic of bench.py that needs no GPU: the algorithmic-byte tables, the lookup of the
recorded profiler traffic, the clock record's time windows, and the oracle arm on a tiny sample."""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_algorithmic_bytes_per_element():
    # block 32: 1/32 scale byte per element beside the codes
    assert bench.b_quantize(2, "int8") == 3.03125 and bench.b_quantize(4, "e4m3") == 5.03125
    assert bench.b_slice_scale("int6") == 1.8125 and bench.b_slice_scale("e2m1") == 1.5625
    assert bench.b_dequantize("int4", 2) == 2.53125 and bench.b_dequantize("e2m1", 4) == 4.53125
    assert bench.STEP_BYTES_PER_ELEM == 25.875 and len(bench.STEP_OPS) == 10
    assert bench.W2_STEP_BYTES_PER_ELEM == 29.78125 and len(bench.W2_OPS) == 12
    shapes = bench.inputs.llama8b_shapes()
    assert int(bench.STEP_BYTES_PER_ELEM * sum(r * c for *_, r, c in shapes)) == 180589953024


def test_recorded_traffic_is_used_only_for_the_sources_it_was_taken_from(tmp_path, monkeypatch):
    rec = {"kernel_sources": "0123456789abcdef",
           "kernels": {"fake_quant_bwd_bf16": {"dram_bytes_per_element": 3.9, "dram_pct_of_peak": 84.0}}}
    os.makedirs(tmp_path / "profiles")
    json.dump(rec, open(tmp_path / "profiles" / "ncu_traffic.json", "w"))
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    monkeypatch.setattr(bench, "kernel_sources_digest", lambda: "0123456789abcdef")
    assert bench.ncu_traffic("fake_quant_bwd_bf16", 1000) == (3900, 84.0)
    assert bench.ncu_traffic("no_such_kernel", 1000) == (None, None)
    monkeypatch.setattr(bench, "kernel_sources_digest", lambda: "fedcba9876543210")
    assert bench.ncu_traffic("fake_quant_bwd_bf16", 1000) == (None, None)       # the kernels have changed since


def test_kernel_sources_digest_covers_the_library_sources_only():
    d = bench.kernel_sources_digest()
    assert len(d) == 16 and d == bench.kernel_sources_digest()


def test_clock_windows():
    s = bench.ClockSampler(0)
    s.max_mhz = 1965.0
    s.how = "test"
    s.samples = [(10.0, 1900.0, 0), (10.1, 1800.0, 0x4), (10.2, 1700.0, 0x4), (11.0, 1965.0, 0)]
    assert s.window(10.05, 10.25) == 1750.0
    assert s.window(10.3, 10.4) == 1700.0                  # no sample inside: the nearest one
    rec = s.summary(10.0, 10.2)
    assert rec["sm_mhz"] == 1800.0 and rec["sm_min_mhz"] == 1700.0 and rec["samples"] == 3
    assert rec["reasons"] == ["sw_power_cap"] and rec["sm_max_mhz"] == 1965.0
    assert bench.ClockSampler(0).summary(0, 1)["samples"] == 0


def test_reps_for():
    assert bench.reps_for(3.0) == 50 and bench.reps_for(1000.0) == 2 and bench.reps_for(100.0) == 15


def test_oracle_step_and_core_split_on_a_tiny_sample(tmp_path):
    import multiprocessing as mp
    x = bench.inputs.weight_bf16_normal(8, 256, seed=3)
    assert bench.oracle_step(x) == x.size
    path = str(tmp_path / "s.npy")
    np.save(path, x)
    with mp.get_context("fork").Pool(3) as pool:
        assert bench.oracle_all_cores(x, pool, 3, path) > 0
