"""The conjugate-gradient iteration of Section 4.2 on the device (paper_1911_05181_b200.cg) against the CPU checker
(oracle.cg) on the same seeded problems: same brackets, same steps, same errors, same parameters."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from oracle import cg as ocg
from paper_1911_05181_b200 import binding as ul, cg
from helpers import dev

pytestmark = pytest.mark.gpu


def _checker_run(sizes, Ws, bs, X, y, n_bracket, iters, a0):
    shapes = [w.shape for w in Ws] + [b.shape for b in bs]
    L = len(Ws)

    def unpack(v):
        out, o = [], 0
        for s in shapes:
            k = int(np.prod(s)); out.append(v[o:o + k].reshape(s).astype(np.float32)); o += k
        return out[:L], out[L:]

    def full(v):
        W, b = unpack(v); l, dW, db = oracle.mlp_gradient(W, b, X, y)
        return l, np.concatenate([t.ravel() for t in dW + db])

    def sub(v):
        W, b = unpack(v); l, dW, db = oracle.mlp_gradient(W, b, X[:n_bracket], y[:n_bracket])
        return np.concatenate([t.ravel() for t in dW + db])

    def err(v):
        W, b = unpack(v); return oracle.mlp_forward_loss(W, b, X, y)

    w0 = np.concatenate([t.ravel() for t in Ws + bs]).astype(np.float64)
    w, hist = ocg.minimise(w0, err, full, sub, iters, a0)
    return unpack(w), hist


def _compare(hist, want, tol_e, tol_a):
    assert len(hist) == len(want)
    for h, r in zip(hist[:-1], want[:-1]):
        assert abs(h["E"] - r["E"]) <= tol_e * abs(r["E"])
        assert (h["slopes"], h["losses"]) == (r["slopes"], r["losses"])         # the same sign decisions were taken
        for k in ("lo", "hi", "alpha"):
            assert abs(h[k] - r[k]) <= tol_a * abs(r[k]) + 1e-30, (k, h[k], r[k])
        assert abs(h["beta"] - r["beta"]) <= 50 * tol_a * max(r["beta"], 1e-3)
    assert abs(hist[-1]["E"] - want[-1]["E"]) <= tol_e * abs(want[-1]["E"])


@pytest.mark.parametrize("math_mode,tol", [(ul.MATH_FP32_SIMT, 1e-5), (ul.MATH_3XTF32, 1e-5)])
def test_small_network_five_iterations(math_mode, tol):
    sizes = [12, 9, 5]; n = 200; nb = 50
    Ws, bs = si.mlp_params(31, sizes)
    X, y = si.mlp_batch(31, sizes, n)
    (wantW, wantb), want = _checker_run(sizes, Ws, bs, X, y, nb, 5, 1e-3)
    opt = cg.ConjugateGradient(sizes, math_mode, n)
    opt.set_params(Ws, bs)
    hist = opt.minimise(dev(X), dev(y), nb, 5, 1e-3)
    _compare(hist, want, tol, 2e-3)
    gotW, gotb = opt.params()
    for a, b in zip(gotW + gotb, wantW + wantb):
        assert oracle.rel_l2(a, b) <= 1e-3
    assert hist[-1]["E"] < 0.95 * hist[0]["E"]


def test_paper_network_two_iterations():
    sizes = [400, 480, 3203]; n = 4096; nb = 512
    Ws, bs = si.mlp_params(2, sizes)
    X, y = si.mlp_batch(2, sizes, n)
    (wantW, wantb), want = _checker_run(sizes, Ws, bs, X, y, nb, 2, 1e-4)
    opt = cg.ConjugateGradient(sizes, ul.MATH_3XTF32, n)
    opt.set_params(Ws, bs)
    hist = opt.minimise(dev(X), dev(y), nb, 2, 1e-4)
    _compare(hist, want, 1e-5, 2e-3)
    assert hist[-1]["E"] < hist[0]["E"]


def test_vector_calls_against_numpy():
    n = 100003
    x = si.uniform_pm1(5, 7, n); y = si.uniform_pm1(5, 8, n)
    dx, dy = dev(x), dev(y)
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = torch.empty(ul.vec_dot_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    ul.vec_dot(n, dx, dy, out, ws, ws.numel())
    ref = float(np.dot(x.astype(np.float64), y.astype(np.float64)))
    assert abs(out.item() - ref) <= 1e-12 * np.sum(np.abs(x.astype(np.float64) * y))
    first = out.item()
    ul.vec_dot(n, dx, dy, out, ws, ws.numel())
    assert out.item() == first                                                     # fixed order: same bits
    dz = torch.empty_like(dx)
    ul.vec_axpby(n, 0.75, dx, -2.0, dy, dz)
    assert np.array_equal(dz.cpu().numpy(), np.float32(0.75) * x + np.float32(-2.0) * y) or \
        np.allclose(dz.cpu().numpy(), 0.75 * x.astype(np.float64) - 2.0 * y, rtol=0, atol=2e-7)
