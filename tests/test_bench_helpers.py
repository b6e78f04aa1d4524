"""Host logic of bench.py: which measured peak a fraction is taken of, and the pattern split of the scaling modes."""
import importlib.util
import os

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
_spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
bench = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(bench)

PEAKS = {"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 2000.0,
         "clocks_under_load": {"sm_mhz_median": 1400.0}, "_source": "measured"}


def test_tensor_peaks_halve_the_bf16_rates_for_tf32_only():
    tf = bench.tensor_peaks(PEAKS, half=False)
    bf = bench.tensor_peaks(PEAKS, half=True)
    assert (tf["burst"], tf["sustained"]) == (800.0, 700.0) and (bf["burst"], bf["sustained"]) == (1600.0, 1400.0)
    assert tf["burst_clock_mhz"] == 2000.0 and tf["sustained_clock_mhz"] == 1400.0
    assert "x 0.5" in tf["source"] and "x 0.5" not in bf["source"]


def test_short_regions_are_held_to_the_burst_peak_and_long_ones_to_the_sustained_peak():
    tp = bench.tensor_peaks(PEAKS, half=False)
    short = bench.fractions(600.0, tp, timed_region_ms=330.0, sm_mhz=1900.0)
    assert short["peak_kind"] == "burst" and short["frac"] == pytest.approx(0.75) and short["frac_of_sustained"] == pytest.approx(600 / 700)
    # the clock-normalised fraction scales the peak to the clock of the run
    assert short["frac_clock_normalised"] == pytest.approx(600.0 / (800.0 * 1900.0 / 2000.0))
    long = bench.fractions(600.0, tp, timed_region_ms=1500.0, sm_mhz=1400.0)
    assert long["peak_kind"] == "sustained" and long["frac"] == pytest.approx(600 / 700) and long["frac_of_burst"] == pytest.approx(0.75)
    assert long["frac_clock_normalised"] == pytest.approx(600 / 700)
    # no clock sample: no clock-normalised figure, everything else still there
    assert "frac_clock_normalised" not in bench.fractions(600.0, tp, 10.0, None)


def test_scaling_workloads_of_the_processor_scaling_experiment():
    assert bench.WORKLOADS["scale_small"][:2] == ([400, 80, 200], 40960)
    assert bench.WORKLOADS["scale_jocr"][:2] == ([400, 480, 3203], 163480)
    assert bench.WORKLOADS["scale_worker"][:2] == ([400, 480, 3203], 32000)
    assert bench.DEFAULT_SCALING == {"scale_small": "strong", "scale_jocr": "strong"}
    # every shape of the SGEMM sweep with 3203 columns is there as the configuration states it (not a stand-in)
    assert ("N", "N", 65536, 3203, 480) in bench.SGEMM_SWEEP and ("T", "N", 480, 3203, 65536) in bench.SGEMM_SWEEP
    assert not any(n == 3204 for _, _, _, n, _ in bench.SGEMM_SWEEP)
