"""Error / gradient evaluation (Sections 4.1-4.3) of the CUDA path against the CPU checker, through the C-ABI."""
import math

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_1911_05181_b200 import binding as ul
from helpers import TOL, GpuNet, dev

pytestmark = pytest.mark.gpu

MATHS = [ul.MATH_FP32_SIMT, ul.MATH_3XTF32, ul.MATH_TF32, ul.MATH_BF16]


def _net(seed, sizes, bias_scale=0.2):
    Ws, bs = si.mlp_params(seed, sizes)
    if bias_scale:
        bs = [si.uniform_pm1(seed, 900 + l, b.size) * np.float32(bias_scale) for l, b in enumerate(bs)]
    return Ws, bs


def _compare(got, want, tol):
    gl, gW, gb = got; wl, wW, wb = want
    assert abs(gl - wl) <= tol * abs(wl), (gl, wl)
    for l, (a, b) in enumerate(zip(gW, wW)):
        e = oracle.rel_l2(a, b); assert e <= tol, ("dW", l, e)
    for l, (a, b) in enumerate(zip(gb, wb)):
        e = oracle.rel_l2(a, b); assert e <= tol, ("db", l, e)


@pytest.mark.parametrize("math_mode", MATHS)
def test_config1_tiny_mlp(math_mode):
    # 256-128-64, 4096 patterns, seed 0, biases zero: one full summed gradient + loss
    sizes = [256, 128, 64]
    Ws, bs = si.mlp_params(0, sizes)
    X, y = si.mlp_batch(0, sizes, 4096)
    g = GpuNet(sizes, math_mode, 4096); g.set_params(Ws, bs)
    got = g.gradient(X, y)
    _compare(got, oracle.mlp_gradient(Ws, bs, X, y), TOL[math_mode])
    assert abs(g.forward_loss(X, y) - got[0]) <= 1e-9 * abs(got[0])


@pytest.mark.parametrize("math_mode", MATHS)
@pytest.mark.parametrize("sizes,n", [([37, 29, 11], 300), ([130, 260, 131, 67], 517), ([20, 9], 150), ([400, 480, 3203], 700)])
def test_ragged_shapes_and_depths(math_mode, sizes, n):
    # nothing is a multiple of a tile; one, two and three weight matrices; non-zero biases
    Ws, bs = _net(21, sizes)
    X, y = si.mlp_batch(21, sizes, n)
    g = GpuNet(sizes, math_mode, n + 5); g.set_params(Ws, bs)
    _compare(g.gradient(X, y), oracle.mlp_gradient(Ws, bs, X, y), TOL[math_mode])
    wl = oracle.mlp_forward_loss(Ws, bs, X, y)
    assert abs(g.forward_loss(X, y) - wl) <= TOL[math_mode] * abs(wl)


@pytest.mark.parametrize("math_mode", MATHS)
def test_zero_weights_closed_form(math_mode):
    sizes = [64, 48, 40]; n = 1000
    Ws = [np.zeros((sizes[l + 1], sizes[l]), np.float32) for l in range(2)]
    bs = [np.zeros(sizes[l + 1], np.float32) for l in range(2)]
    X, y = si.mlp_batch(22, sizes, n)
    g = GpuNet(sizes, math_mode, n); g.set_params(Ws, bs)
    loss, dW, db = g.gradient(X, y)
    assert abs(loss - n * math.log(40)) <= 1e-6 * loss
    assert all(np.all(w == 0) for w in dW) and np.all(db[0] == 0)
    # each entry is a sum of n probabilities of 1/40 minus a count: the tolerance scales with that sum
    assert np.allclose(db[1], n / 40 - np.bincount(y, minlength=40), atol=max(1e-3, TOL[math_mode] * n / 40))


@pytest.mark.parametrize("math_mode", MATHS)
def test_chunk_accumulation_matches_one_batch_and_oracle(math_mode):
    # Section 4.3: additive over disjoint subsets; ragged chunks 300 + 300 + 177, in a fixed order
    sizes = [50, 70, 33]; n = 777
    Ws, bs = _net(23, sizes)
    X, y = si.mlp_batch(23, sizes, n)
    want = oracle.mlp_gradient(Ws, bs, X, y)
    g = GpuNet(sizes, math_mode, 300); g.set_params(Ws, bs)
    for i, lo in enumerate(range(0, n, 300)):
        got = g.gradient(X[lo:lo + 300], y[lo:lo + 300], accumulate=(i > 0))
    _compare(got, want, TOL[math_mode])
    # an empty block changes nothing when accumulating, and zeroes everything when not
    again = g.gradient(X[:0], y[:0], accumulate=True)
    assert again[0] == got[0] and all(np.array_equal(a, b) for a, b in zip(again[1] + again[2], got[1] + got[2]))
    zero = g.gradient(X[:0], y[:0], accumulate=False)
    assert zero[0] == 0.0 and all(np.all(a == 0) for a in zero[1] + zero[2])


@pytest.mark.parametrize("math_mode", MATHS)
def test_bitwise_repeatable(math_mode):
    sizes = [400, 480, 3203]; n = 3000
    Ws, bs = _net(24, sizes)
    X, y = si.mlp_batch(24, sizes, n)
    g = GpuNet(sizes, math_mode, n); g.set_params(Ws, bs)
    a = g.gradient(X, y)
    for t in g.dW + g.db: t.fill_(float("nan"))
    b = g.gradient(X, y)
    assert a[0] == b[0]
    assert all(np.array_equal(p, q) for p, q in zip(a[1] + a[2], b[1] + b[2]))


def test_leading_dimension_of_x():
    sizes = [30, 20, 10]; n = 200
    Ws, bs = _net(25, sizes)
    X, y = si.mlp_batch(25, sizes, n)
    big = np.full((n, 36), 9.0, np.float32); big[:, :30] = X
    g = GpuNet(sizes, ul.MATH_FP32_SIMT, n); g.set_params(Ws, bs)
    a = g.gradient(X, y)
    b = g.gradient(dev(big), y, ldx=36)
    _compare(b, oracle.mlp_gradient(Ws, bs, X, y), 1e-5)
    assert a[0] == b[0]


def test_sgd_step_matches_checker_within_an_ulp():
    sizes = [40, 30, 20]
    Ws, bs = _net(26, sizes)
    X, y = si.mlp_batch(26, sizes, 256)
    g = GpuNet(sizes, ul.MATH_FP32_SIMT, 256); g.set_params(Ws, bs)
    _, dW, db = g.gradient(X, y)
    g.net.sgd_step(g.W, g.b, g.dW, g.db, 1e-3)
    torch.cuda.synchronize()
    for w_new, w_old, gr in zip(g.W + g.b, Ws + bs, dW + db):
        want = oracle.sgd_step(w_old.ravel(), gr.ravel(), float(np.float32(1e-3)))
        got = w_new.cpu().numpy().ravel()
        ulp = np.spacing(np.abs(want))
        assert np.all(np.abs(got - want) <= ulp)


def test_device_fill_matches_host_generator_bitwise():
    n = 100003
    t = torch.empty(n, device="cuda"); ul.fill_uniform(t, n, 3, si.TID_X, 17, 0)
    assert np.array_equal(t.cpu().numpy(), si.uniform01(3, si.TID_X, n, 17))
    ul.fill_uniform(t, n, 1, si.TID_GEMM_A, 0, 1)
    assert np.array_equal(t.cpu().numpy(), si.uniform_pm1(1, si.TID_GEMM_A, n))
    lab = torch.empty(n, dtype=torch.int32, device="cuda"); ul.fill_labels(lab, n, 3, si.TID_LABELS, 5, 3203)
    assert np.array_equal(lab.cpu().numpy(), si.labels(3, si.TID_LABELS, n, 3203, 5))


def test_device_status_is_clean_after_all_this():
    g = GpuNet([8, 4, 2], ul.MATH_3XTF32, 8)
    assert g.net.last_device_status() == ul.OK


@pytest.mark.parametrize("math_mode", MATHS)
def test_config3_paper_scale_full_batch(math_mode):
    """400-480-3203, 65536 patterns, seed 2 (the launch configuration the bench times), against the full checker.
    The checker needs about a minute on 8 cores; its result is shared by the three math modes."""
    sizes = [400, 480, 3203]; n = 65536
    Ws, bs = si.mlp_params(2, sizes)
    X, y = si.mlp_batch(2, sizes, n)
    if not hasattr(test_config3_paper_scale_full_batch, "want"):
        test_config3_paper_scale_full_batch.want = oracle.mlp_gradient(Ws, bs, X, y)
    g = GpuNet(sizes, math_mode, n); g.set_params(Ws, bs)
    got = g.gradient(X, y)
    _compare(got, test_config3_paper_scale_full_batch.want, TOL[math_mode])
    assert got[0] > n * math.log(3203)
