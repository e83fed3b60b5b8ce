"""CPU checks of bench.py's host logic: which clock samples belong to a timed region, which measured peak a roofline
fraction is taken against, and the reference arm's JSON line on the smallest workload."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def sampler(samples):
    s = bench.ClockSampler(0)
    s.samples = samples
    return s


def test_clock_window_takes_the_samples_of_its_own_region():
    # (time, sm MHz, max MHz, W, reasons)
    smp = [(100.00, 1965.0, 1965.0, 250.0, []), (100.02, 1500.0, 1965.0, 900.0, ["sw_power_cap"]),
           (100.04, 1200.0, 1965.0, 990.0, ["sw_power_cap"]), (100.06, 1100.0, 1965.0, 995.0, ["sw_power_cap"]),
           (100.50, 1965.0, 1965.0, 260.0, [])]
    w = sampler(smp).window(100.01, 100.07)
    assert w["samples"] == 3 and w["sm_mhz"] == 1200.0 and w["sm_min_mhz"] == 1100.0 and w["reasons"] == ["sw_power_cap"]
    assert w["power_w_max"] == 995.0 and w["sm_max_mhz"] == 1965.0
    # a region shorter than the sampling period: the nearest sample, and the record says so
    w = sampler(smp).window(100.47, 100.48)
    assert w["samples"] == 1 and w["sm_mhz"] == 1965.0 and "nearest" in w["note"]
    assert sampler([]).window(0, 1)["sm_mhz"] is None
    assert sampler(None).window(0, 1)["sm_mhz"] is None


def test_roofline_fraction_is_taken_against_the_peak_that_fits_the_run():
    pk = {"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6400.0, "source": "measured"}
    short_full_clock = bench.roofline_fracs(800.0, pk, False, 0.05, {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0})
    assert short_full_clock["peak"] == 1600.0 and abs(short_full_clock["frac"] - 0.5) < 1e-12
    long_run = bench.roofline_fracs(800.0, pk, False, 3.0, {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0})
    assert long_run["peak"] == 1400.0
    capped = bench.roofline_fracs(800.0, pk, False, 0.05, {"sm_mhz": 1200.0, "sm_max_mhz": 1965.0})
    assert capped["peak"] == 1400.0 and abs(capped["frac_of_burst"] - 0.5) < 1e-12
    assert abs(capped["frac_of_sustained"] - 800.0 / 1400.0) < 1e-12
    mx = bench.roofline_fracs(800.0, pk, True, 0.05, {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0})
    assert mx["peak"] == 3200.0                                  # fp8 peak = bf16 peak x the nominal 2 : 1 ratio


def test_reference_arm_prints_the_contract_line_on_the_smallest_workload():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, check=True).stdout
    line = json.loads(out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["config"]["workload"] == "tiny" and line["value"] > 0 and line["higher_is_better"] is True
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]


def test_expert_parallel_shard_of_the_inputs_equals_the_rows_of_the_full_tensors():
    """make_inputs(expert_range=...) is what an expert-parallel rank generates: the same values as its rows of the
    full expert tensors."""
    import numpy as np
    from paper_2609_36070_b200 import inputs
    cfg = inputs.CONFIGS["tiny"]
    full = inputs.make_inputs(cfg)
    lo, hi = cfg.E // 2, cfg.E
    part = inputs.make_inputs(cfg, expert_range=(lo, hi))
    assert np.array_equal(part["W_gate_up"], full["W_gate_up"][lo:hi])
    assert np.array_equal(part["W_down"], full["W_down"][lo:hi])
    assert np.array_equal(part["x"], full["x"]) and np.array_equal(part["W_r"], full["W_r"])
