"""Pins of the conjugate-gradient checker (oracle/cg.py) on functions with known answers."""
import math

import numpy as np
import pytest

from oracle import cg


def _quadratic(n, seed):
    rng = np.random.default_rng(seed)
    Q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    A = Q @ np.diag(np.linspace(1.0, 9.0, n)) @ Q.T
    b = rng.standard_normal(n)
    f = lambda w: 0.5 * w @ A @ w - b @ w
    g = lambda w: A @ w - b
    return A, b, f, g


def test_parabola_vertex_closed_forms():
    f = lambda x: 3.0 * (x - 1.25) ** 2 + 7.0
    assert abs(cg.parabola_vertex(0.0, f(0.0), 1.0, f(1.0), 2.0, f(2.0)) - 1.25) < 1e-14
    assert abs(cg.parabola_vertex(-3.0, f(-3.0), 0.5, f(0.5), 4.0, f(4.0)) - 1.25) < 1e-13
    assert cg.parabola_vertex(0.0, 0.0, 1.0, 1.0, 2.0, 2.0) is None            # a line
    assert cg.parabola_vertex(0.0, 0.0, 1.0, 1.0, 2.0, 0.0) is None            # opens downward


def test_bracket_contains_the_minimiser_and_counts_evaluations():
    for xmin in (0.003, 0.4, 1.0, 37.0):
        slope = lambda a: 2.0 * (a - xmin)
        lo, hi, n = cg.bracket(slope, 1.0)
        assert lo <= xmin <= hi and hi <= 2.0 * max(lo, 1e-300) + 1e-12 or lo == 0.0
        assert lo < hi
    lo, hi, n = cg.bracket(lambda a: 2.0 * (a - 37.0), 1.0)
    assert (lo, hi, n) == (32.0, 64.0, 7)                                        # 1, 2, 4, 8, 16, 32, 64
    lo, hi, n = cg.bracket(lambda a: 2.0 * (a - 0.3), 1.0)
    assert (lo, hi, n) == (0.25, 0.5, 3)                                         # 1, 0.5, 0.25
    lo, hi, n = cg.bracket(lambda a: 1.0, 1.0)                                   # never negative: gives up after 12 halvings
    assert lo == 0.0 and hi == 2.0 ** -12 and n == 13


def test_line_search_is_exact_on_a_quadratic():
    A, b, f, g = _quadratic(7, 0)
    w = np.zeros(7); d = -g(w)
    alpha, e, info = cg.line_search(lambda t: f(w + t * d), lambda t: float(g(w + t * d) @ d), 1.0)
    exact = -(g(w) @ d) / (d @ A @ d)                                            # textbook exact step
    assert abs(alpha - exact) <= 1e-12 * exact
    assert abs(e - f(w + exact * d)) <= 1e-12


def test_polak_ribiere_on_a_quadratic_is_conjugate_gradients():
    # with exact line searches PR equals Fletcher-Reeves, successive gradients are orthogonal, directions are
    # A-conjugate, and n steps solve the n x n system (textbook properties of linear CG)
    n = 9
    A, b, f, g = _quadratic(n, 1)
    grads, dirs = [], []
    def grad_fn(w):
        grads.append(g(w)); return f(w), g(w)
    w, hist = cg.minimise(np.zeros(n), f, grad_fn, g, n, 1.0)
    assert np.allclose(w, np.linalg.solve(A, b), atol=1e-8)
    for k in range(1, n):
        if np.linalg.norm(grads[k]) < 1e-7:
            break
        assert abs(grads[k] @ grads[k - 1]) <= 1e-6 * np.linalg.norm(grads[k]) * np.linalg.norm(grads[k - 1])
        fr = (grads[k] @ grads[k]) / (grads[k - 1] @ grads[k - 1])
        assert abs(hist[k]["beta"] - fr) <= 1e-5 * fr
    assert all(hist[k + 1]["E"] < hist[k]["E"] for k in range(n))


def test_beta_formula_and_reset():
    g0 = np.array([1.0, 2.0, -1.0]); g1 = np.array([0.5, -1.0, 2.0])
    assert cg.pr_beta(g1, g0) == max(0.0, (g1 @ (g1 - g0)) / (g0 @ g0))
    assert cg.pr_beta(0.5 * g0, g0) == 0.0                                       # g1.(g1-g0) < 0: restart


def test_descends_on_a_tiny_network_with_a_subset_for_bracketing():
    import oracle
    import synth_inputs as si
    sizes = [12, 9, 5]; n = 200
    Ws, bs = si.mlp_params(31, sizes)
    X, y = si.mlp_batch(31, sizes, n)
    shapes = [w.shape for w in Ws] + [b.shape for b in bs]
    def unpack(v):
        out, o = [], 0
        for s in shapes:
            k = int(np.prod(s)); out.append(v[o:o + k].reshape(s).astype(np.float32)); o += k
        return out[:2], out[2:]
    def full(v):
        W, b = unpack(v); l, dW, db = oracle.mlp_gradient(W, b, X, y)
        return l, np.concatenate([t.ravel() for t in dW + db])
    def sub(v):
        W, b = unpack(v); l, dW, db = oracle.mlp_gradient(W, b, X[:50], y[:50])
        return np.concatenate([t.ravel() for t in dW + db])
    w0 = np.concatenate([t.ravel() for t in Ws + bs]).astype(np.float64)
    w, hist = cg.minimise(w0, lambda v: full(v)[0], full, sub, 6, 1e-3)
    E = [h["E"] for h in hist]
    assert all(b <= a for a, b in zip(E, E[1:])) and E[-1] < 0.95 * E[0]
