"""Seeded input generator and the paper's flop accounting (host logic)."""
import json
import os

import numpy as np
import pytest

import synth_inputs as si
from paper_1911_05181_b200 import flops

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_generator_is_sliceable_and_deterministic():
    a = si.uniform01(5, si.TID_X, 1000)
    b = np.concatenate([si.uniform01(5, si.TID_X, 400), si.uniform01(5, si.TID_X, 600, offset=400)])
    assert np.array_equal(a, b)
    assert not np.array_equal(a, si.uniform01(6, si.TID_X, 1000))
    assert not np.array_equal(a, si.uniform01(5, si.TID_X + 1, 1000))
    X, y = si.mlp_batch(2, [400, 480, 3203], 10)
    X2, y2 = si.mlp_batch(2, [400, 480, 3203], 4, offset=6)
    assert np.array_equal(X[6:], X2) and np.array_equal(y[6:], y2)


def test_generator_ranges_and_moments():
    u = si.uniform01(1, 3, 200000)
    assert u.dtype == np.float32 and u.min() >= 0 and u.max() < 1
    assert abs(u.mean() - 0.5) < 5e-3 and abs(u.var() - 1 / 12) < 2e-3
    assert np.array_equal(u * 2 ** 24, np.floor(u * 2 ** 24))      # 24-bit grid: exact in fp32
    s = si.uniform_pm1(1, 4, 200000)
    assert s.min() >= -1 and s.max() < 1 and abs(s.mean()) < 1e-2
    lab = si.labels(1, 5, 200000, 3203)
    assert lab.dtype == np.int32 and lab.min() >= 0 and lab.max() < 3203
    assert np.bincount(lab, minlength=3203).max() < 130           # ~62 expected per class
    g = si.normal(1, 6, 200000, 0.05)
    assert abs(g.mean()) < 1e-3 and abs(g.std() - 0.05) < 1e-3
    Ws, bs = si.mlp_params(2, [400, 480, 3203])
    assert Ws[0].shape == (480, 400) and Ws[1].shape == (3203, 480)
    assert abs(Ws[1].std() - 480 ** -0.5) < 1e-3 and all((b == 0).all() for b in bs)


def test_paper_flop_and_parameter_counts():
    g = json.load(open(os.path.join(GOLD, "paper_counts.json")))
    sizes, n_p = g["sizes"], g["n_patterns"]
    assert flops.n_params(sizes) == g["n_params"]
    assert flops.n_params(sizes) * 4 / 2 ** 20 == pytest.approx(g["param_mbytes"], abs=0.05)
    assert flops.forward_flops(sizes, n_p) == 2 * n_p * (400 + 3203) * 480
    assert flops.gradient_flops(sizes, n_p) == n_p * (4 * 400 * 480 + 6 * 480 * 3203)
    assert round(flops.forward_flops(sizes, n_p) / 1e12) == g["error_tflop"]
    # the paper prints 92; the formula gives 92.57, i.e. the paper truncated
    assert int(flops.gradient_flops(sizes, n_p) / 1e12) == g["gradient_tflop"]
    assert round(0.8 * flops.forward_flops(sizes, n_p) / 1e12) == g["error_tflop_80pct"]
    assert round(0.8 * flops.gradient_flops(sizes, n_p) / 1e12) == g["gradient_tflop_80pct"]
    per = 0.8 * flops.gradient_flops(sizes, n_p) / g["n_procs"] / 1e9
    assert per == pytest.approx(g["gradient_gflop_per_proc_80pct"], rel=0.01)
    per_e = 0.8 * flops.forward_flops(sizes, n_p) / g["n_procs"] / 1e9
    assert per_e == pytest.approx(g["error_gflop_per_proc_80pct"], rel=0.02)
    assert flops.sgemm_flops(3, 5, 7) == 210
    assert flops.gradient_flops_per_pattern([400, 480, 3203]) == 9992640
    assert flops.gradient_flops_per_pattern([1024, 4096, 4096, 3203]) == 196157440
    assert flops.gradient_flops_per_pattern([256, 128, 64]) == 180224
