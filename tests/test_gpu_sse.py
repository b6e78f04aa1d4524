"""The paper's own output layer (tanh units, summed squared error, Eqs. 1 and 3) on the CUDA path against the CPU
checker, through the C-ABI."""
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
    bs = [si.uniform_pm1(seed, 900 + l, b.size) * np.float32(bias_scale) for l, b in enumerate(bs)]
    return Ws, bs


def _grad(g, X, T, accumulate=False):
    dX, dT = dev(X), dev(T)
    n = dX.shape[0]
    g.net.gradient_sse(g.W, g.b, dX, X.shape[1], dT, T.shape[1], n, accumulate, g.dW, g.db, g.loss)
    torch.cuda.synchronize()
    return float(g.loss.item()), [t.cpu().numpy() for t in g.dW], [t.cpu().numpy() for t in g.db]


def _compare(got, want, tol):
    assert abs(got[0] - want[0]) <= tol * abs(want[0]), (got[0], want[0])
    for name, gs, ws in (("dW", got[1], want[1]), ("db", got[2], want[2])):
        for l, (a, b) in enumerate(zip(gs, ws)):
            e = oracle.rel_l2(a, b); assert e <= tol, (name, l, e)


@pytest.mark.parametrize("math_mode", MATHS)
@pytest.mark.parametrize("sizes,n", [([37, 29, 11], 300), ([132, 260, 128, 68], 517), ([20, 12], 150), ([400, 480, 3203], 700)])
def test_ragged_shapes_and_depths(math_mode, sizes, n):
    Ws, bs = _net(41, sizes)
    X, _ = si.mlp_batch(41, sizes, n)
    T = si.mlp_targets(41, sizes, n)
    g = GpuNet(sizes, math_mode, n + 3); g.set_params(Ws, bs)
    got = _grad(g, X, T)
    _compare(got, oracle.mlp_sse_gradient(Ws, bs, X, T), TOL[math_mode])
    # the error alone
    g.net.forward_sse(g.W, g.b, dev(X), X.shape[1], dev(T), T.shape[1], n, g.loss)
    torch.cuda.synchronize()
    assert abs(float(g.loss.item()) - got[0]) <= 1e-9 * abs(got[0])


@pytest.mark.parametrize("math_mode", MATHS)
def test_coded_targets_chunks_and_repeat(math_mode):
    # +1 / -1 class codes; 300 + 300 + 177 patterns accumulated equal the whole batch; a second run repeats bitwise
    sizes = [50, 70, 33]; n = 777
    Ws, bs = _net(42, sizes)
    X, _ = si.mlp_batch(42, sizes, n)
    T = si.mlp_targets(42, sizes, n, coded=True)
    want = oracle.mlp_sse_gradient(Ws, bs, X, T)
    g = GpuNet(sizes, math_mode, 300); g.set_params(Ws, bs)
    for i, lo in enumerate(range(0, n, 300)):
        got = _grad(g, X[lo:lo + 300], T[lo:lo + 300], accumulate=(i > 0))
    _compare(got, want, TOL[math_mode])
    for i, lo in enumerate(range(0, n, 300)):
        again = _grad(g, X[lo:lo + 300], T[lo:lo + 300], accumulate=(i > 0))
    assert again[0] == got[0] and all(np.array_equal(a, b) for a, b in zip(again[1] + again[2], got[1] + got[2]))
    empty = _grad(g, X[:0], T[:0], accumulate=True)
    assert empty[0] == got[0] and all(np.array_equal(a, b) for a, b in zip(empty[1] + empty[2], got[1] + got[2]))


@pytest.mark.parametrize("math_mode", [ul.MATH_3XTF32, ul.MATH_TF32, ul.MATH_BF16])
def test_paper_network_8192_patterns(math_mode):
    # 400-480-3203 with +1 / -1 codes: several 256-row tiles on every product, in the launch shapes of the benchmark
    sizes = [400, 480, 3203]; n = 8192
    Ws, bs = si.mlp_params(2, sizes)
    X, _ = si.mlp_batch(2, sizes, n)
    T = si.mlp_targets(2, sizes, n, coded=True)
    if not hasattr(test_paper_network_8192_patterns, "want"):
        test_paper_network_8192_patterns.want = oracle.mlp_sse_gradient(Ws, bs, X, T)
    g = GpuNet(sizes, math_mode, n); g.set_params(Ws, bs)
    _compare(_grad(g, X, T), test_paper_network_8192_patterns.want, TOL[math_mode])


def test_bad_arguments():
    sizes = [8, 4, 3]
    g = GpuNet(sizes, ul.MATH_FP32_SIMT, 16); g.set_params(*_net(43, sizes))
    X = dev(np.zeros((4, 8), np.float32)); T = dev(np.zeros((4, 3), np.float32))
    assert g.net.gradient_sse(g.W, g.b, X, 8, T, 2, 4, False, g.dW, g.db, g.loss, check=False) == ul.ERR_INVALID_ARG   # ldt < n_L
    assert g.net.gradient_sse(g.W, g.b, X, 8, None, 3, 4, False, g.dW, g.db, g.loss, check=False) == ul.ERR_INVALID_ARG
    assert g.net.forward_sse(g.W, g.b, X, 8, T, 3, 17, g.loss, check=False) == ul.ERR_INVALID_ARG                     # n > max

