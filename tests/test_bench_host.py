"""Host-side logic of bench.py: the algorithmic work of a call, the roofline object and the clock windows."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2603_06588_b200 import inputs  # noqa: E402


def test_algorithmic_work_counts_every_kv_element_once_and_only_visible_pairs():
    case = inputs.config1_tiny_prefill()          # 1 x 256 tokens, Hq = Hkv = 8, D = 64, two spans, all 8 heads probed
    nbytes, flops = bench.algorithmic_work(case)
    pairs = 256 * 257 // 2                        # causal: row i sees i + 1 keys
    assert flops == 4.0 * 64 * pairs * 8
    kv = 256 * 8 * 64 * 2 * 2                     # K and V, bf16, once per KV head
    qo = 2 * 256 * 8 * 64 * 2
    mass = 256 * 8 * 2 * 4
    assert nbytes == kv + qo + mass + (256 // 16) * 4 + 1 * 8
    dec = inputs.config2_decode(num_seqs=5, lo=100, hi=300)
    nbytes, flops = bench.algorithmic_work(dec)
    keys = int(dec.seq_lens.sum())
    assert flops == 4.0 * 128 * keys * 32         # one row per sequence sees all its keys
    assert nbytes >= keys * 8 * 128 * 2 * 2


def test_roofline_object_takes_the_peak_that_fits_the_timed_region():
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "source": "measured"}
    r = bench.roofline("hbm", 650e6, 1e-4, peaks, "k", 0.0, traffic=651e6)
    assert r["unit"] == "GB/s" and r["achieved"] == pytest.approx(6500.0) and r["frac"] == pytest.approx(1.0)
    assert r["traffic"] == 651e6 and "measured" in r["peak_source"]
    short = bench.roofline("tensor", 1.4e12, 1e-3, peaks, "k", 0.5)
    long_ = bench.roofline("tensor", 1.4e12, 1e-3, peaks, "k", 3.0)
    assert short["peak"] == 1600.0 and long_["peak"] == 1400.0
    assert short["achieved"] == pytest.approx(1400.0) and long_["frac"] == pytest.approx(1.0)
    assert short["frac_of_sustained"] == pytest.approx(1.0) and short["traffic"] is None


def test_clock_windows_pick_the_samples_between_two_instants():
    import datetime
    s = bench.ClockSampler(0)
    t0 = datetime.datetime(2026, 1, 1, 12, 0, 0).timestamp()
    s.rows = [(t0 + 0.1 * i, 1900.0 - 100.0 * (i >= 5), 1965.0, 900.0 + i, ["sw_power_cap"] if i >= 5 else []) for i in range(10)]
    early, late = s.window(t0, t0 + 0.4), s.window(t0 + 0.5, t0 + 0.9)
    assert early["samples"] == 5 and early["sm_mhz"] == 1900.0 and early["reasons"] == []
    assert late["samples"] == 5 and late["sm_mhz"] == 1800.0 and late["reasons"] == ["sw_power_cap"] and late["sm_max_mhz"] == 1965.0
    assert s.window(t0 + 5.0, t0 + 6.0)["samples"] == 0 and s.window(t0 + 5.0, t0 + 6.0)["sm_mhz"] is None


def test_every_table_entry_is_a_named_workload_and_the_traffic_keys_exist():
    assert bench.HEADLINE in bench.WORKLOADS
    for name in bench.TABLE:
        assert name in bench.WORKLOADS, name
    for name in bench.DRAM_TRAFFIC:
        assert name in bench.WORKLOADS, name
