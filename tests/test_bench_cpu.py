"""Host logic of bench.py that needs no GPU: the regime rule behind the roofline denominator and the flop count."""
import importlib.util
import os

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
spec = importlib.util.spec_from_file_location("bench", os.path.join(ROOT, "bench.py"))
bench = importlib.util.module_from_spec(spec)
spec.loader.exec_module(bench)


def test_regime_follows_the_sampled_clock_and_falls_back_to_the_duration():
    at_max = {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "samples": 20}
    capped = {"sm_mhz": 1567.0, "sm_max_mhz": 1965.0, "samples": 257, "reasons": ["sw_power_cap"]}
    assert bench.run_was_burst(at_max, 0.05) and bench.run_was_burst(at_max, 5.0)
    assert not bench.run_was_burst(capped, 0.54) and not bench.run_was_burst(capped, 5.0)
    # too few samples to trust: the length of the timed region decides
    assert bench.run_was_burst({"sm_mhz": 1200.0, "sm_max_mhz": 1965.0, "samples": 1}, 0.007)
    assert not bench.run_was_burst(None, 2.0) and bench.run_was_burst(None, 0.5)


def test_algorithmic_flops_of_the_named_configs():
    from paper_2604_17397_b200 import synth
    # 4 T Lk D H: the 14B step of the metric (3.140 TFLOP) and the drafter shape (0.404 TFLOP)
    assert bench.attn_flops(synth.WAN_14B, 7 * 4680) == pytest.approx(3.140e12, rel=1e-3)
    assert bench.attn_flops(synth.WAN_1_3B, 3 * 4680) == pytest.approx(0.404e12, rel=2e-3)


def test_peaks_come_from_the_measured_file_when_present():
    pk = bench.peaks()
    assert pk["source"] in ("measured", "fallback")
    assert pk["bf16_tflops"] >= pk["bf16_tflops_sustained"] > 0 and pk["hbm_gbs"] > 0
