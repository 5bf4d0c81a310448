"""Host-side logic of bench.py that decides what the JSON line claims: which measured peak a run is compared with,
which (segment, head) pairs the CPU legs time, and where the recorded DRAM traffic comes from.  No GPU."""
import json
import os

import numpy as np

import bench
from paper_2607_03229_b200 import workloads as W

PEAKS = {"bf16_tflops": 1650.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6500.0}


def test_peak_follows_the_sampled_clock():
    burst, why_b = bench.pick_peak({"sm_mhz": 1950.0, "sm_max_mhz": 1965.0}, PEAKS)
    sust, why_s = bench.pick_peak({"sm_mhz": 1665.0, "sm_max_mhz": 1965.0}, PEAKS)
    assert burst == 1650.0 and "burst" in why_b
    assert sust == 1400.0 and "sustained" in why_s
    # exactly at the 5 % line the burst figure applies; with no clock sample the lower (stricter-to-meet) one
    assert bench.pick_peak({"sm_mhz": 0.95 * 1965.0, "sm_max_mhz": 1965.0}, PEAKS)[0] == 1650.0
    assert bench.pick_peak({"sm_mhz": None, "sm_max_mhz": None}, PEAKS)[0] == 1400.0


def test_oracle_sample_is_a_prefix_of_the_segment_major_order():
    w = W.vit_l()
    counts = [int(n) for n in w.patch_counts]
    segs = [i for i, n in enumerate(counts) if n > 0]
    target = 3e11
    pairs, flops = bench.oracle_sample(w, target)
    order = [(s, h) for h in range(w.n_heads) for s in segs]
    assert pairs == order[:len(pairs)]
    per = [14.0 * w.head_dim * counts[s] ** 2 for s, _ in pairs]
    assert abs(flops - sum(per)) <= 1e-6 * flops
    assert flops >= target > flops - per[-1]                 # stops at the first pair that reaches the target
    everything, total = bench.oracle_sample(w, float("inf"))  # the whole workload when the target is out of reach
    assert len(everything) == len(order)
    assert abs(total - w.flops(True, True)) <= 1e-9 * total
    text = bench.sample_text(w, pairs, flops)
    assert f"{len(pairs)} of {len(order)}" in text


def test_oracle_sample_skips_empty_segments_and_never_returns_nothing():
    w = W.Workload("holes", 1, [0, 130, 0, 64], 2, 64, True)
    pairs, flops = bench.oracle_sample(w, 0.0)
    assert pairs == [(1, 0)] and flops == 14.0 * 64 * 130 * 130
    assert all(s in (1, 3) for s, _ in bench.oracle_sample(w, float("inf"))[0])


def test_recorded_traffic_reads_the_tracked_table():
    path = os.path.join(os.path.dirname(os.path.abspath(bench.__file__)), "profiles", "dram_traffic.json")
    with open(path) as f:
        table = json.load(f)
    key = next(k for k in table if "@" in k)
    kernel, workload = key.split("@")
    assert bench.recorded_traffic(kernel, workload) == table[key]
    assert bench.recorded_traffic("no_such_kernel", "vit_l") is None


def test_rates_fractions_are_consistent():
    w = W.vit_l()
    kern = {"fwd": 0.6, "bwd_main": 1.3, "merge": 0.04}
    out = bench.rates(w, 2.1, kern, {"sm_mhz": 1665.0, "reasons": ["sw_power_cap"], "samples": 7}, PEAKS)
    tf = w.flops(True, True) / 2.1e-3 / 1e12
    assert np.isclose(out["step_tflops"], tf)
    assert np.isclose(out["step_frac"]["of_measured_burst"], tf / 1650.0)
    assert np.isclose(out["step_frac"]["of_measured_sustained"], tf / 1400.0)
    cyc = 1665.0e6 * 148 * 8192 / 1e12
    assert np.isclose(out["step_frac"]["of_cycle_peak_at_sampled_clock"], tf / cyc)
    assert np.isclose(out["fwd_tflops"], w.flops(True, False) / 0.6e-3 / 1e12)
    assert np.isclose(out["bwd_main_tflops"], w.flops(False, True) / 1.3e-3 / 1e12)


def test_repeat_count_covers_the_minimum_time_within_its_bounds():
    assert bench.repeat_count(2.0, 200, 2.0) == 5           # 0.4 s per region -> five regions
    assert bench.repeat_count(2.0, 200, 2.1) == 6
    assert bench.repeat_count(50.0, 200, 2.0) == 1          # one region is already longer
    assert bench.repeat_count(0.01, 3, 2.0) == 40           # capped
    assert bench.repeat_count(0.0, 3, 2.0) == 40            # a zero time does not divide by zero
