"""CPU checker of the training iteration of Section 4.2: Polak-Ribiere conjugate-gradient directions with a line
search made of an exponential step-size scheme that brackets the minimum by the sign of the directional
derivative (estimated on a subset of the patterns) and one quadratic interpolation of the error.

TEST INFRASTRUCTURE ONLY, float64 numpy, independent of the CUDA path.  The paper gives the ingredients but no
constants and no order of evaluation; the reading taken here is:

  direction   d_0 = -g_0;  d_k = -g_k + beta_k d_{k-1},  beta_k = max(0, g_k.(g_k - g_{k-1}) / g_{k-1}.g_{k-1})
  bracketing  slope(a) = grad_subset(w + a d) . d.  From a_0, while slope(a_j) < 0: a_{j+1} = 2 a_j (at most
              `max_doublings` times).  If already slope(a_0) >= 0: a is halved until the slope is negative (at most
              `max_halvings` times).  Result: lo (last step with negative slope, 0 if none) < hi (first step with
              slope >= 0).  If no step with slope >= 0 was found, hi is the last step tried.  If the subset sees no
              negative slope at all (it disagrees with the direction), the bracketing is repeated with the slope
              on all patterns.
  interpolation  E at lo, mid = (lo + hi)/2, hi on ALL patterns; vertex of the parabola through the three points,
              kept if the parabola opens upward and the vertex lies in [lo, hi]; E at the vertex; the step taken is
              the best of the evaluated points (lo is only eligible when lo > 0).
  next a_0    the step just taken.

The functions take callbacks, so the pins can run them on functions with known answers (quadratics).
"""
from __future__ import annotations

import numpy as np


def pr_beta(g_new, g_old):
    """Polak-Ribiere coefficient, reset to 0 when negative."""
    return max(0.0, float(np.dot(g_new, g_new - g_old)) / float(np.dot(g_old, g_old)))


def bracket(slope, a0, max_doublings=30, max_halvings=12):
    """(lo, hi, n_slope_evaluations) as described in the module docstring.  slope(a) -> float."""
    a = float(a0)
    s = slope(a)
    n = 1
    if s < 0.0:
        lo = a
        for _ in range(max_doublings):
            a = 2.0 * a
            s = slope(a)
            n += 1
            if s >= 0.0:
                return lo, a, n
            lo = a
        return lo / 2.0 if lo > a0 else 0.0, a, n      # never turned upward: [previous, last]
    hi = a
    for _ in range(max_halvings):
        a = 0.5 * a
        s = slope(a)
        n += 1
        if s < 0.0:
            return a, hi, n
        hi = a
    return 0.0, hi, n


def parabola_vertex(xa, fa, xb, fb, xc, fc):
    """Abscissa of the vertex of the parabola through three points, or None if it does not open upward."""
    d1 = (fb - fa) / (xb - xa)
    d2 = (fc - fb) / (xc - xb)
    curv = (d2 - d1) / (xc - xa)
    if not np.isfinite(curv) or curv <= 0.0:
        return None
    return 0.5 * (xa + xb) - 0.5 * d1 / curv


def line_search(loss, slope, a0, slope_all=None):
    """Step along the direction: returns (alpha, E(alpha), info).  slope: on the bracketing subset; slope_all: on all
    patterns, used when the subset finds no negative slope."""
    lo, hi, n_slopes = bracket(slope, a0)
    if lo == 0.0 and slope_all is not None:
        lo, hi, n2 = bracket(slope_all, a0)
        n_slopes += n2
    mid = 0.5 * (lo + hi)
    pts = [(lo, loss(lo)), (mid, loss(mid)), (hi, loss(hi))]
    v = parabola_vertex(pts[0][0], pts[0][1], pts[1][0], pts[1][1], pts[2][0], pts[2][1])
    if v is not None and lo <= v <= hi and v > 0.0:
        pts.append((v, loss(v)))
    cand = [p for p in pts if p[0] > 0.0]
    alpha, e = min(cand, key=lambda p: p[1])
    return alpha, e, {"lo": lo, "hi": hi, "vertex": v, "slopes": n_slopes, "losses": len(pts)}


def minimise(w0, loss_fn, grad_fn, grad_subset_fn, iters, a0):
    """loss_fn(w) -> E; grad_fn(w) -> (E, g) on all patterns; grad_subset_fn(w) -> g on the bracketing subset.
    Returns (w, history) with history[k] = dict(E=error before step k, alpha=..., beta=..., lo, hi, ...)."""
    w = np.array(w0, dtype=np.float64)
    e, g = grad_fn(w)
    d = -g
    hist = []
    a = float(a0)
    beta = 0.0
    for _ in range(iters):
        if float(np.dot(g, d)) >= 0.0:          # not a descent direction: restart along the negative gradient
            d = -g; beta = 0.0
        alpha, e_new, info = line_search(lambda t: loss_fn(w + t * d), lambda t: float(np.dot(grad_subset_fn(w + t * d), d)), a,
                                         lambda t: float(np.dot(grad_fn(w + t * d)[1], d)))
        hist.append(dict(E=e, alpha=alpha, beta=beta, **info))
        w = w + alpha * d
        a = alpha
        e, g_new = grad_fn(w)
        beta = pr_beta(g_new, g)
        d = -g_new + beta * d
        g = g_new
    hist.append(dict(E=e))
    return w, hist
