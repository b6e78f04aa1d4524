"""CPU checker ("oracle"): ctypes front end of ulsnn_oracle.c.

TEST INFRASTRUCTURE ONLY.  The product package never imports this; only the
tests, the smoke check and the bench's CPU-baseline leg do.  It shares no code
with the CUDA path.  Everything is computed in float64 from the fp32 inputs,
directly from the definitions of Sections 3.1 and 4.1 (see the C file's header
for what pins it).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ulsnn_oracle.c")
_LIB = os.path.join(_HERE, "libulsnn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C checker with gcc (-O2, OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        subprocess.check_call(cmd)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_sgemm_entry.restype = ctypes.c_double
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _f32(a):
    a = np.asarray(a)
    assert a.dtype == np.float32, a.dtype
    return a


def _ptr(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct)) if a is not None else None


def _trans(t) -> int:
    t = str(t).upper()
    assert t in ("N", "T"), t
    return 1 if t == "T" else 0


def sgemm(transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C=None, ldc=0) -> np.ndarray:
    """C_out = alpha*op(A)*op(B) + beta*C in float64, dense [M, N] (Section 3.1)."""
    A = _f32(A); B = _f32(B)
    out = np.empty((M, N), dtype=np.float64)
    if beta != 0.0:
        C = _f32(C)
    _load().oracle_sgemm(
        ctypes.c_int(_trans(transA)), ctypes.c_int(_trans(transB)),
        ctypes.c_int64(M), ctypes.c_int64(N), ctypes.c_int64(K), ctypes.c_double(alpha),
        _ptr(A, ctypes.c_float), ctypes.c_int64(lda), _ptr(B, ctypes.c_float), ctypes.c_int64(ldb),
        ctypes.c_double(beta), _ptr(C if beta != 0.0 else None, ctypes.c_float), ctypes.c_int64(ldc),
        _ptr(out, ctypes.c_double))
    return out


def sgemm_entry(transA, transB, K, alpha, A, lda, B, ldb, beta, C, ldc, i, j) -> float:
    A = _f32(A); B = _f32(B)
    return float(_load().oracle_sgemm_entry(
        ctypes.c_int(_trans(transA)), ctypes.c_int(_trans(transB)), ctypes.c_int64(K),
        ctypes.c_double(alpha), _ptr(A, ctypes.c_float), ctypes.c_int64(lda),
        _ptr(B, ctypes.c_float), ctypes.c_int64(ldb), ctypes.c_double(beta),
        _ptr(_f32(C) if beta != 0.0 else None, ctypes.c_float), ctypes.c_int64(ldc),
        ctypes.c_int64(i), ctypes.c_int64(j)))


def _flatten(Ws, bs):
    sizes = [int(Ws[0].shape[1])] + [int(w.shape[0]) for w in Ws]
    for l, w in enumerate(Ws):
        assert w.shape == (sizes[l + 1], sizes[l]) and bs[l].shape == (sizes[l + 1],)
    Wflat = np.ascontiguousarray(np.concatenate([_f32(w).ravel() for w in Ws]))
    bflat = np.ascontiguousarray(np.concatenate([_f32(b).ravel() for b in bs]))
    return np.asarray(sizes, dtype=np.int32), Wflat, bflat


def _unflatten(sizes, dW, db):
    outW, outb, ow, ob = [], [], 0, 0
    for l in range(len(sizes) - 1):
        nw = int(sizes[l]) * int(sizes[l + 1])
        outW.append(dW[ow:ow + nw].reshape(int(sizes[l + 1]), int(sizes[l]))); ow += nw
        outb.append(db[ob:ob + int(sizes[l + 1])]); ob += int(sizes[l + 1])
    return outW, outb


def mlp_forward_loss(Ws, bs, X, labels) -> float:
    """Summed cross-entropy of softmax(W_L h + b_L) over all patterns (no 1/n)."""
    sizes, Wflat, bflat = _flatten(Ws, bs)
    X = np.ascontiguousarray(_f32(X)); labels = np.ascontiguousarray(labels, dtype=np.int32)
    loss = ctypes.c_double(0.0)
    rc = _load().oracle_mlp_forward_loss(
        ctypes.c_int(len(Ws)), _ptr(sizes, ctypes.c_int32), _ptr(Wflat, ctypes.c_float),
        _ptr(bflat, ctypes.c_float), _ptr(X, ctypes.c_float), ctypes.c_int64(X.shape[1]),
        _ptr(labels, ctypes.c_int32), ctypes.c_int64(X.shape[0]), ctypes.byref(loss))
    assert rc == 0
    return loss.value


def mlp_gradient(Ws, bs, X, labels):
    """(loss, [dW_l], [db_l]) summed over patterns, float64."""
    sizes, Wflat, bflat = _flatten(Ws, bs)
    X = np.ascontiguousarray(_f32(X)); labels = np.ascontiguousarray(labels, dtype=np.int32)
    dW = np.zeros(Wflat.size, dtype=np.float64); db = np.zeros(bflat.size, dtype=np.float64)
    loss = ctypes.c_double(0.0)
    rc = _load().oracle_mlp_gradient(
        ctypes.c_int(len(Ws)), _ptr(sizes, ctypes.c_int32), _ptr(Wflat, ctypes.c_float),
        _ptr(bflat, ctypes.c_float), _ptr(X, ctypes.c_float), ctypes.c_int64(X.shape[1]),
        _ptr(labels, ctypes.c_int32), ctypes.c_int64(X.shape[0]),
        _ptr(dW, ctypes.c_double), _ptr(db, ctypes.c_double), ctypes.byref(loss))
    assert rc == 0
    gW, gb = _unflatten(sizes, dW, db)
    return loss.value, gW, gb


def mlp_sse_gradient(Ws, bs, X, T, want_grad=True):
    """The paper's own head (tanh outputs, summed squared error, Eqs. 1 and 3)."""
    sizes, Wflat, bflat = _flatten(Ws, bs)
    X = np.ascontiguousarray(_f32(X)); T = np.ascontiguousarray(_f32(T))
    dW = np.zeros(Wflat.size, dtype=np.float64); db = np.zeros(bflat.size, dtype=np.float64)
    loss = ctypes.c_double(0.0)
    rc = _load().oracle_mlp_sse_gradient(
        ctypes.c_int(len(Ws)), _ptr(sizes, ctypes.c_int32), _ptr(Wflat, ctypes.c_float),
        _ptr(bflat, ctypes.c_float), _ptr(X, ctypes.c_float), ctypes.c_int64(X.shape[1]),
        _ptr(T, ctypes.c_float), ctypes.c_int64(T.shape[1]), ctypes.c_int64(X.shape[0]),
        ctypes.c_int(1 if want_grad else 0),
        _ptr(dW, ctypes.c_double), _ptr(db, ctypes.c_double), ctypes.byref(loss))
    assert rc == 0
    gW, gb = _unflatten(sizes, dW, db)
    return loss.value, gW, gb


def mlp_probe(Ws, bs, X, want_probs=True, want_hidden=True):
    """Per-pattern softmax probabilities and last-hidden activations (float64)."""
    sizes, Wflat, bflat = _flatten(Ws, bs)
    X = np.ascontiguousarray(_f32(X))
    n = X.shape[0]
    probs = np.empty((n, int(sizes[-1])), dtype=np.float64) if want_probs else None
    hid = np.empty((n, int(sizes[-2])), dtype=np.float64) if want_hidden else None
    rc = _load().oracle_mlp_probe(
        ctypes.c_int(len(Ws)), _ptr(sizes, ctypes.c_int32), _ptr(Wflat, ctypes.c_float),
        _ptr(bflat, ctypes.c_float), _ptr(X, ctypes.c_float), ctypes.c_int64(X.shape[1]),
        ctypes.c_int64(n), _ptr(probs, ctypes.c_double), _ptr(hid, ctypes.c_double))
    assert rc == 0
    return probs, hid


def sgemm_abs(transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C=None, ldc=0) -> np.ndarray:
    """|alpha| * |op(A)| * |op(B)| + |beta| * |C|: the magnitude sums the forward error of the product is proportional to."""
    A = _f32(A); B = _f32(B)
    out = np.empty((M, N), dtype=np.float64)
    if beta != 0.0:
        C = _f32(C)
    _load().oracle_sgemm_abs(
        ctypes.c_int(_trans(transA)), ctypes.c_int(_trans(transB)),
        ctypes.c_int64(M), ctypes.c_int64(N), ctypes.c_int64(K), ctypes.c_double(alpha),
        _ptr(A, ctypes.c_float), ctypes.c_int64(lda), _ptr(B, ctypes.c_float), ctypes.c_int64(ldb),
        ctypes.c_double(beta), _ptr(C if beta != 0.0 else None, ctypes.c_float), ctypes.c_int64(ldc),
        _ptr(out, ctypes.c_double))
    return out


def mlp_gradient_abs(Ws, bs, X, labels=None, T=None):
    """([aW_l], [ab_l]): the summed gradient's back-propagation with every term in absolute value (softmax head when
    `labels` is given, the paper's tanh + squared-error head when `T` is).  What rounding errors are proportional to."""
    sizes, Wflat, bflat = _flatten(Ws, bs)
    X = np.ascontiguousarray(_f32(X))
    head = 0 if T is None else 1
    if head == 0:
        labels = np.ascontiguousarray(labels, dtype=np.int32)
    else:
        T = np.ascontiguousarray(_f32(T))
    aW = np.zeros(Wflat.size, dtype=np.float64); ab = np.zeros(bflat.size, dtype=np.float64)
    rc = _load().oracle_mlp_gradient_abs(
        ctypes.c_int(len(Ws)), _ptr(sizes, ctypes.c_int32), _ptr(Wflat, ctypes.c_float),
        _ptr(bflat, ctypes.c_float), _ptr(X, ctypes.c_float), ctypes.c_int64(X.shape[1]),
        _ptr(labels if head == 0 else None, ctypes.c_int32), _ptr(T if head == 1 else None, ctypes.c_float),
        ctypes.c_int64(T.shape[1] if head == 1 else 0), ctypes.c_int64(X.shape[0]), ctypes.c_int(head),
        _ptr(aW, ctypes.c_double), _ptr(ab, ctypes.c_double))
    assert rc == 0
    return _unflatten(sizes, aW, ab)


def perturb_inputs(Ws, bs, X, T=None, eps=2.0 ** -14, seed=0):
    """Copies of the parameters, the patterns and (if given) the dense targets with every entry multiplied by
    1 + eps*u, u uniform in [-1, 1) from numpy's default_rng(seed), drawn tensor by tensor in the order
    W_0.., b_0.., X, T, evaluated in float64 and rounded to fp32.  Labels are not perturbed."""
    rng = np.random.default_rng(seed)

    def pert(a):
        a = _f32(a)
        return (a.astype(np.float64) * (1.0 + eps * rng.uniform(-1.0, 1.0, a.shape))).astype(np.float32)

    Wp = [pert(w) for w in Ws]
    bp = [pert(b) for b in bs]
    Xp = pert(X)
    Tp = pert(T) if T is not None else None
    return Wp, bp, Xp, Tp


def gradient_condition(Ws, bs, X, labels=None, T=None, eps=2.0 ** -14, seeds=(12345, 12346)):
    """Estimated relative condition number of every tensor of the summed gradient with respect to componentwise
    relative perturbations of its inputs: ||g(inputs*(1+eta)) - g(inputs)||_2 / ||g(inputs)||_2 divided by the
    root-mean-square size eps/sqrt(3) of the random eta, the larger of the values of the given seeds.
    Returns ([cond dW_l], [cond db_l]).  A finite-precision evaluation commits relative errors of the size of its
    unit roundoff in inputs and intermediates, so its attainable relative error is proportional to this number."""
    def grad(Wq, bq, Xq, Tq):
        return mlp_gradient(Wq, bq, Xq, labels) if T is None else mlp_sse_gradient(Wq, bq, Xq, Tq)

    _, gW, gb = grad(Ws, bs, X, T)
    rms = eps / np.sqrt(3.0)
    best = None
    for seed in seeds:
        Wp, bp, Xp, Tp = perturb_inputs(Ws, bs, X, T, eps, seed)
        _, pW, pb = grad(Wp, bp, Xp, Tp)
        c = []
        for a, b in zip(pW + pb, gW + gb):
            r = np.linalg.norm(b.ravel())
            c.append(float(np.linalg.norm((a - b).ravel()) / r / rms) if r > 0 else 0.0)
        best = c if best is None else [max(u, v) for u, v in zip(best, c)]
    return best[:len(Ws)], best[len(Ws):]


def sgd_step(w, g, lr) -> np.ndarray:
    """W - lr*grad evaluated in float64 and rounded once to fp32 (Section 4.2)."""
    w = np.ascontiguousarray(_f32(w)); g = np.ascontiguousarray(_f32(g))
    out = np.empty_like(w)
    _load().oracle_sgd_step(ctypes.c_int64(w.size), _ptr(w, ctypes.c_float), _ptr(g, ctypes.c_float),
                            ctypes.c_double(lr), _ptr(out, ctypes.c_float))
    return out


def rel_l2(x, ref) -> float:
    """||x - ref||_2 / ||ref||_2 in float64 (absolute norm if ref is all zero)."""
    x = np.asarray(x, dtype=np.float64).ravel(); ref = np.asarray(ref, dtype=np.float64).ravel()
    d = np.linalg.norm(x - ref); r = np.linalg.norm(ref)
    return float(d / r) if r > 0 else float(d)
