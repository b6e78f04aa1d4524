"""Training iteration of Section 4.2 around the error / gradient calls of the library: Polak-Ribiere
conjugate-gradient directions, and a line search that brackets the minimum along the direction with an exponential
step-size scheme -- using only the SIGN of the directional derivative, estimated on a subset of the patterns -- and
then takes one quadratic interpolation of the error.

Everything that touches a parameter vector runs on the device through the C-ABI (ulsnn_mlp_gradient,
ulsnn_mlp_forward_loss, ulsnn_vec_dot, ulsnn_vec_axpby); this module only sequences the calls and does the scalar
arithmetic of the search (a handful of floats per iteration) on the host.

Reading of the paper's description taken here (the paper names the ingredients, not the constants):
  d_0 = -g_0;  d_k = -g_k + beta_k d_{k-1},  beta_k = max(0, g_k.(g_k - g_{k-1}) / g_{k-1}.g_{k-1});
  a direction with g.d >= 0 is replaced by -g;
  steps double from a_0 while the subset's slope grad(w + a d).d is negative (at most 30 times), or halve while it is
  not (at most 12 times); if the subset never sees a negative slope the bracketing is redone on all patterns;
  the error on all patterns at lo, (lo+hi)/2, hi gives a parabola whose vertex, if the parabola opens upward and the
  vertex lies inside the bracket, is evaluated too; the best evaluated step is taken and becomes the next a_0.
"""
from __future__ import annotations

import math

from . import binding as ul

_PAD = 64       # floats: every tensor of the flat parameter vector starts on a 256-byte boundary


class ConjugateGradient:
    def __init__(self, sizes, math_mode, max_patterns):
        import torch
        self.torch = torch
        self.sizes = [int(s) for s in sizes]
        self.L = len(self.sizes) - 1
        self.net = ul.Mlp(self.sizes, math_mode, max_patterns)
        shapes = [(self.sizes[l + 1], self.sizes[l]) for l in range(self.L)] + [(self.sizes[l + 1],) for l in range(self.L)]
        self.offsets, off = [], 0
        for s in shapes:
            self.offsets.append(off)
            off += (math.prod(s) + _PAD - 1) // _PAD * _PAD
        self.n = off
        self.shapes = shapes
        z = lambda: torch.zeros(self.n, device="cuda")
        self.w, self.g, self.g_prev, self.d, self.trial, self.gs = z(), z(), z(), z(), z(), z()
        nb = ul.vec_dot_workspace_bytes(self.n)
        self._dot_ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
        self._dot_out = torch.zeros(1, dtype=torch.float64, device="cuda")
        self._loss = torch.zeros(1, dtype=torch.float64, device="cuda")

    def _views(self, flat):
        t = [flat[o:o + math.prod(s)].view(s) for o, s in zip(self.offsets, self.shapes)]
        return t[:self.L], t[self.L:]

    def set_params(self, Ws, bs):
        W, b = self._views(self.w)
        for dst, src in zip(W + b, list(Ws) + list(bs)):
            dst.copy_(self.torch.as_tensor(src).to(dst.device))

    def params(self):
        W, b = self._views(self.w)
        return [t.cpu().numpy() for t in W], [t.cpu().numpy() for t in b]

    # ---- device work
    def _dot(self, x, y) -> float:
        ul.vec_dot(self.n, x, y, self._dot_out, self._dot_ws, self._dot_ws.numel())
        return float(self._dot_out.item())

    def _set_trial(self, alpha):
        ul.vec_axpby(self.n, 1.0, self.w, float(alpha), self.d, self.trial)

    def _gradient(self, flat_w, flat_g, X, y, n) -> float:
        W, b = self._views(flat_w)
        dW, db = self._views(flat_g)
        self.net.gradient(W, b, X, X.shape[1], y, n, False, dW, db, self._loss)
        return float(self._loss.item())

    def _error(self, flat_w, X, y, n) -> float:
        W, b = self._views(flat_w)
        self.net.forward_loss(W, b, X, X.shape[1], y, n, self._loss)
        return float(self._loss.item())

    # ---- the search (scalar logic on the host)
    @staticmethod
    def _bracket(slope, a0, max_doublings=30, max_halvings=12):
        a = float(a0)
        count = 1
        if slope(a) < 0.0:
            lo = a
            for _ in range(max_doublings):
                a *= 2.0
                count += 1
                if slope(a) >= 0.0:
                    return lo, a, count
                lo = a
            return (lo / 2.0 if lo > a0 else 0.0), a, count
        hi = a
        for _ in range(max_halvings):
            a *= 0.5
            count += 1
            if slope(a) < 0.0:
                return a, hi, count
            hi = a
        return 0.0, hi, count

    @staticmethod
    def _vertex(xa, fa, xb, fb, xc, fc):
        s1 = (fb - fa) / (xb - xa)
        s2 = (fc - fb) / (xc - xb)
        curvature = (s2 - s1) / (xc - xa)
        if not math.isfinite(curvature) or curvature <= 0.0:
            return None
        return 0.5 * (xa + xb) - 0.5 * s1 / curvature

    def minimise(self, X, y, n_bracket, iters, a0):
        """X [n x sizes[0]], y int32 [n] device tensors; the first n_bracket patterns estimate slope signs.
        Returns the history: one dict per iteration (error before the step, step, beta, bracket) and a last one
        with the final error."""
        n = int(X.shape[0])
        Xs, ys = X[:n_bracket], y[:n_bracket]

        def slope_subset(alpha):
            self._set_trial(alpha)
            self._gradient(self.trial, self.gs, Xs, ys, n_bracket)
            return self._dot(self.gs, self.d)

        def slope_all(alpha):
            self._set_trial(alpha)
            self._gradient(self.trial, self.gs, X, y, n)
            return self._dot(self.gs, self.d)

        def error(alpha):
            self._set_trial(alpha)
            return self._error(self.trial, X, y, n)

        e = self._gradient(self.w, self.g, X, y, n)
        ul.vec_axpby(self.n, -1.0, self.g, 0.0, self.g, self.d)                 # d = -g
        hist, a, beta = [], float(a0), 0.0
        for _ in range(iters):
            if self._dot(self.g, self.d) >= 0.0:
                ul.vec_axpby(self.n, -1.0, self.g, 0.0, self.g, self.d)
                beta = 0.0
            lo, hi, slopes = self._bracket(slope_subset, a)
            if lo == 0.0:
                lo, hi, more = self._bracket(slope_all, a)
                slopes += more
            mid = 0.5 * (lo + hi)
            pts = [(lo, error(lo)), (mid, error(mid)), (hi, error(hi))]
            v = self._vertex(pts[0][0], pts[0][1], pts[1][0], pts[1][1], pts[2][0], pts[2][1])
            if v is not None and lo <= v <= hi and v > 0.0:
                pts.append((v, error(v)))
            alpha, _ = min((p for p in pts if p[0] > 0.0), key=lambda p: p[1])
            hist.append(dict(E=e, alpha=alpha, beta=beta, lo=lo, hi=hi, vertex=v, slopes=slopes, losses=len(pts)))
            ul.vec_axpby(self.n, 1.0, self.w, float(alpha), self.d, self.w)       # w += alpha d
            a = alpha
            self.g_prev.copy_(self.g)
            e = self._gradient(self.w, self.g, X, y, n)
            gg_old = self._dot(self.g_prev, self.g_prev)
            beta = max(0.0, (self._dot(self.g, self.g) - self._dot(self.g, self.g_prev)) / gg_old)
            ul.vec_axpby(self.n, -1.0, self.g, float(beta), self.d, self.d)       # d = -g + beta d
        hist.append(dict(E=e))
        return hist
