"""Pins for the CPU checker: none of the expected values below comes from the
checker itself.  A dropped term, a wrong sign, a transposed operand or a wrong
index in oracle/ulsnn_oracle.c fails at least one of these."""
import json
import math
import os

import numpy as np
import pytest

import oracle
import synth_inputs as si

GOLD = os.path.join(os.path.dirname(__file__), "golden")
_ENV = {"log": math.log, "exp": math.exp, "tanh": math.tanh, "sqrt": math.sqrt}


def _ev(x):
    if isinstance(x, list):
        return [_ev(v) for v in x]
    return float(eval(x, {"__builtins__": {}}, _ENV)) if isinstance(x, str) else float(x)


# ----------------------------------------------------------------------------- SGEMM (Section 3.1)

def _brute(transA, transB, M, N, K, alpha, A, B, beta, C):
    """Pure-Python triple loop on Python ints/floats (exact for small integers)."""
    out = [[0.0] * N for _ in range(M)]
    for i in range(M):
        for j in range(N):
            s = 0
            for k in range(K):
                a = A[k][i] if transA == "T" else A[i][k]
                b = B[j][k] if transB == "T" else B[k][j]
                s += a * b
            out[i][j] = alpha * s + (beta * C[i][j] if beta != 0 else 0)
    return out


@pytest.mark.parametrize("transA", ["N", "T"])
@pytest.mark.parametrize("transB", ["N", "T"])
@pytest.mark.parametrize("beta", [0.0, 1.0, -2.0])
def test_sgemm_small_integers_exact(transA, transB, beta):
    rng = np.random.default_rng(7)
    M, N, K = 5, 4, 3
    lda, ldb, ldc = 9, 8, 7          # leading dimensions larger than the widths
    ra, ca = (K, M) if transA == "T" else (M, K)
    rb, cb = (N, K) if transB == "T" else (K, N)
    A = np.full((ra, lda), 1e30, np.float32); A[:, :ca] = rng.integers(-4, 5, (ra, ca))
    B = np.full((rb, ldb), 1e30, np.float32); B[:, :cb] = rng.integers(-4, 5, (rb, cb))
    C = np.full((M, ldc), 1e30, np.float32); C[:, :N] = rng.integers(-4, 5, (M, N))
    got = oracle.sgemm(transA, transB, M, N, K, 3.0, A, lda, B, ldb, beta, C, ldc)
    want = _brute(transA, transB, M, N, K, 3.0, A[:, :ca].tolist(), B[:, :cb].tolist(), beta, C[:, :N].tolist())
    assert np.array_equal(got, np.asarray(want, dtype=np.float64))


def test_sgemm_hand_example():
    # [[1,2],[3,4]] * [[5,6],[7,8]] = [[19,22],[43,50]]
    A = np.array([[1, 2], [3, 4]], np.float32); B = np.array([[5, 6], [7, 8]], np.float32)
    assert oracle.sgemm("N", "N", 2, 2, 2, 1.0, A, 2, B, 2, 0.0).tolist() == [[19, 22], [43, 50]]
    # A^T * B = [[26,30],[38,44]];  A * B^T = [[17,23],[39,53]];  A^T * B^T = [[23,31],[34,46]]
    assert oracle.sgemm("T", "N", 2, 2, 2, 1.0, A, 2, B, 2, 0.0).tolist() == [[26, 30], [38, 44]]
    assert oracle.sgemm("N", "T", 2, 2, 2, 1.0, A, 2, B, 2, 0.0).tolist() == [[17, 23], [39, 53]]
    assert oracle.sgemm("T", "T", 2, 2, 2, 1.0, A, 2, B, 2, 0.0).tolist() == [[23, 31], [34, 46]]


def test_sgemm_transpose_identity_and_library():
    # (A B)^T = B^T A^T ties the four forms together; numpy's float64 matmul is the library routine.
    A, B, _ = si.gemm_operands(1, 37, 29, 29, 23, 1, 1)
    AB = oracle.sgemm("N", "N", 37, 23, 29, 1.0, A, 29, B, 23, 0.0)
    BtAt = oracle.sgemm("T", "T", 23, 37, 29, 1.0, B, 23, A, 29, 0.0)
    assert np.allclose(AB.T, BtAt, rtol=0, atol=1e-13)
    assert np.allclose(AB, A.astype(np.float64) @ B.astype(np.float64), rtol=0, atol=1e-12)
    At = np.ascontiguousarray(A.T); Bt = np.ascontiguousarray(B.T)
    assert np.allclose(oracle.sgemm("T", "N", 37, 23, 29, 1.0, At, 37, B, 23, 0.0), AB, rtol=0, atol=1e-13)
    assert np.allclose(oracle.sgemm("N", "T", 37, 23, 29, 1.0, A, 29, Bt, 29, 0.0), AB, rtol=0, atol=1e-13)
    assert oracle.sgemm_entry("N", "T", 29, 1.0, A, 29, Bt, 29, 0.0, None, 0, 5, 7) == pytest.approx(AB[5, 7], abs=1e-13)


def test_sgemm_beta_zero_ignores_c_and_edge_sizes():
    A = np.ones((2, 3), np.float32); B = np.ones((3, 2), np.float32)
    C = np.full((2, 2), np.nan, np.float32)
    assert oracle.sgemm("N", "N", 2, 2, 3, 1.0, A, 3, B, 2, 0.0, C, 2).tolist() == [[3, 3], [3, 3]]
    # K = 0: C = beta*C ; alpha = 0: A and B (NaN) are not read
    C2 = np.array([[1, 2], [3, 4]], np.float32)
    assert oracle.sgemm("N", "N", 2, 2, 0, 1.0, A, 3, B, 2, 2.0, C2, 2).tolist() == [[2, 4], [6, 8]]
    An = np.full((2, 3), np.nan, np.float32)
    assert oracle.sgemm("N", "N", 2, 2, 3, 0.0, An, 3, B, 2, 1.0, C2, 2).tolist() == [[1, 2], [3, 4]]


# ----------------------------------------------------------------------------- network: hand-worked example

@pytest.mark.parametrize("label", [0, 1])
def test_hand_worked_2_1_2(label):
    g = json.load(open(os.path.join(GOLD, "hand_net_2_1_2.json")))
    W1 = np.asarray(_ev(g["W1"]), np.float32); b1 = np.asarray(_ev(g["b1"]), np.float32)
    W2 = np.asarray(_ev(g["W2"]), np.float32); b2 = np.asarray(_ev(g["b2"]), np.float32)
    X = np.asarray([g["x"]], np.float32); y = np.asarray([label], np.int32)
    e = g["expected"]
    loss, dW, db = oracle.mlp_gradient([W1, W2], [b1, b2], X, y)
    assert loss == pytest.approx(_ev(e["loss_label%d" % label]), abs=2e-7)
    assert oracle.mlp_forward_loss([W1, W2], [b1, b2], X, y) == pytest.approx(loss, abs=1e-15)
    ex = e["label%d" % label]
    assert np.allclose(db[1], _ev(ex["db2"]), atol=2e-7)
    assert np.allclose(dW[1], _ev(ex["dW2"]), atol=2e-7)
    assert np.allclose(db[0], _ev(ex["db1"]), atol=2e-7)
    assert np.allclose(dW[0], _ev(ex["dW1"]), atol=2e-7)
    probs, hid = oracle.mlp_probe([W1, W2], [b1, b2], X)
    assert hid[0, 0] == pytest.approx(_ev(e["h"]), abs=1e-7)
    assert np.allclose(probs[0], [2 / 3, 1 / 3], atol=2e-7)


# ----------------------------------------------------------------------------- finite differences

def _random_net(seed, sizes, bias_scale=0.3):
    Ws, bs = si.mlp_params(seed, sizes)
    bs = [si.uniform_pm1(seed, 900 + l, b.size) * np.float32(bias_scale) for l, b in enumerate(bs)]
    return Ws, bs


def _fd_check(loss_fn, grad, params, step=2.0 ** -10, tol=1e-4):
    """Central differences of loss_fn for every parameter.  The step is a power of two so that
    p+step and p-step are exact in fp32 for the O(1) parameters used here."""
    num = []
    for t in params:
        flat = t.reshape(-1)
        gnum = np.zeros(flat.size)
        for i in range(flat.size):
            keep = flat[i]
            flat[i] = np.float32(keep + np.float32(step)); up = loss_fn(); hi = float(flat[i])
            flat[i] = np.float32(keep - np.float32(step)); dn = loss_fn(); lo = float(flat[i])
            flat[i] = keep
            gnum[i] = (up - dn) / (hi - lo)
        num.append(gnum)
    num = np.concatenate(num); ana = np.concatenate([np.asarray(g).ravel() for g in grad])
    rel = np.linalg.norm(num - ana) / np.linalg.norm(ana)
    assert rel < tol, rel
    # also elementwise, so a single wrong entry cannot hide in the norm
    assert np.allclose(num, ana, rtol=2e-3, atol=2e-4 * np.abs(ana).max())


@pytest.mark.parametrize("sizes", [[5, 4, 3], [4, 3, 3, 2], [3, 2]])
def test_finite_differences_softmax_ce(sizes):
    Ws, bs = _random_net(11, sizes)
    X, y = si.mlp_batch(11, sizes, 7)
    loss, dW, db = oracle.mlp_gradient(Ws, bs, X, y)
    _fd_check(lambda: oracle.mlp_forward_loss(Ws, bs, X, y), dW + db, Ws + bs)


@pytest.mark.parametrize("sizes", [[5, 4, 3], [4, 3, 3, 2]])
def test_finite_differences_paper_head_and_sign(sizes):
    # Eqs. 1 and 3: tanh outputs, E = sum (y - t)^2.
    Ws, bs = _random_net(12, sizes)
    X, _ = si.mlp_batch(12, sizes, 6)
    T = si.uniform_pm1(12, 77, 6 * sizes[-1]).reshape(6, sizes[-1])
    loss, dW, db = oracle.mlp_sse_gradient(Ws, bs, X, T)
    _fd_check(lambda: oracle.mlp_sse_gradient(Ws, bs, X, T, want_grad=False)[0], dW + db, Ws + bs)
    # E itself, from Eq. 1/3 with numpy (library matmul + tanh)
    a = X.astype(np.float64)
    for l, (W, b) in enumerate(zip(Ws, bs)):
        a = np.tanh(a @ W.astype(np.float64).T + b.astype(np.float64))
    assert loss == pytest.approx(((a - T) ** 2).sum(), rel=1e-12)


def test_paper_matrix_identities_sse_head():
    # Section 4.2 with the paper's head: Y_D = (1-Y*Y)*(T-Y), H_D = (1-H*H)*(Y_D W_ho),
    # G_ih = H_D^T X, G_ho = Y_D^T H; these are -1/2 of the derivative of Eq. 3.
    sizes = [6, 5, 4]
    Ws, bs = si.mlp_params(13, sizes)            # no biases, as in the paper
    X, _ = si.mlp_batch(13, sizes, 9)
    T = si.uniform_pm1(13, 78, 9 * 4).reshape(9, 4)
    _, dW, _ = oracle.mlp_sse_gradient(Ws, bs, X, T)
    Xd = X.astype(np.float64); W1 = Ws[0].astype(np.float64); W2 = Ws[1].astype(np.float64)
    H = np.tanh(Xd @ W1.T); Y = np.tanh(H @ W2.T)
    YD = (1 - Y * Y) * (T - Y); HD = (1 - H * H) * (YD @ W2)
    assert np.allclose(dW[0], -2.0 * (HD.T @ Xd), rtol=1e-11, atol=1e-13)
    assert np.allclose(dW[1], -2.0 * (YD.T @ H), rtol=1e-11, atol=1e-13)


def test_paper_matrix_identities_softmax_head_via_oracle_sgemm():
    # Same identities with delta_out = softmax - onehot, the products done by the checker's own SGEMM
    # (ties the two halves of the checker together and checks the per-pattern code against the matrix form).
    sizes = [7, 6, 5]
    Ws, bs = _random_net(14, sizes)
    n = 11
    X, y = si.mlp_batch(14, sizes, n)
    loss, dW, db = oracle.mlp_gradient(Ws, bs, X, y)
    probs, hid = oracle.mlp_probe(Ws, bs, X)
    D2 = probs.copy(); D2[np.arange(n), y] -= 1.0
    D2f = D2.astype(np.float32); Hf = hid.astype(np.float32)    # fp32 copies for the SGEMM interface
    G2 = oracle.sgemm("T", "N", 5, 6, n, 1.0, D2f, 5, Hf, 6, 0.0)
    assert np.allclose(G2, dW[1], rtol=0, atol=1e-6)
    back = oracle.sgemm("N", "N", n, 6, 5, 1.0, D2f, 5, Ws[1], 6, 0.0)
    D1 = ((1 - hid * hid) * back).astype(np.float32)
    G1 = oracle.sgemm("T", "N", 6, 7, n, 1.0, D1, 6, X, 7, 0.0)
    assert np.allclose(G1, dW[0], rtol=0, atol=1e-6)
    assert np.allclose(D2.sum(0), db[1], atol=1e-12) and np.allclose(D1.sum(0), db[0], atol=1e-6)
    assert loss == pytest.approx(-np.log(probs[np.arange(n), y]).sum(), rel=1e-12)


# ----------------------------------------------------------------------------- invariants and closed forms

def test_softmax_rows_sum_to_one_and_bias_gradient_sums_to_zero():
    sizes = [20, 16, 33]
    Ws, bs = _random_net(15, sizes)
    X, y = si.mlp_batch(15, sizes, 50)
    probs, _ = oracle.mlp_probe(Ws, bs, X)
    assert np.allclose(probs.sum(1), 1.0, atol=1e-14) and (probs > 0).all()
    _, _, db = oracle.mlp_gradient(Ws, bs, X, y)
    assert abs(db[-1].sum()) < 1e-12


@pytest.mark.parametrize("sizes,n", [([256, 128, 64], 300), ([12, 8, 8, 5], 40)])
def test_zero_weights_closed_form(sizes, n):
    Ws = [np.zeros((sizes[l + 1], sizes[l]), np.float32) for l in range(len(sizes) - 1)]
    bs = [np.zeros(sizes[l + 1], np.float32) for l in range(len(sizes) - 1)]
    X, y = si.mlp_batch(16, sizes, n)
    loss, dW, db = oracle.mlp_gradient(Ws, bs, X, y)
    no = sizes[-1]
    assert loss == pytest.approx(n * math.log(no), rel=1e-14)
    assert all(np.all(g == 0) for g in dW)               # h = 0 and W = 0 kill every outer product
    assert all(np.all(g == 0) for g in db[:-1])
    counts = np.bincount(y, minlength=no)
    assert np.allclose(db[-1], n / no - counts, atol=1e-12)


def test_config3_closed_form_constant():
    # all-zero weights at the paper-scale shape: loss = n_p * ln(3203)
    assert 65536 * math.log(3203) == pytest.approx(528996.3127, abs=1e-3)


def test_additivity_over_patterns_and_permutation():
    sizes = [10, 9, 8, 7]
    Ws, bs = _random_net(17, sizes)
    n = 24
    X, y = si.mlp_batch(17, sizes, n)
    loss, dW, db = oracle.mlp_gradient(Ws, bs, X, y)
    # sum of single-pattern gradients
    accW = [np.zeros_like(g) for g in dW]; accb = [np.zeros_like(g) for g in db]; accl = 0.0
    for p in range(n):
        l1, w1, b1 = oracle.mlp_gradient(Ws, bs, X[p:p + 1], y[p:p + 1])
        accl += l1
        for a, g in zip(accW, w1): a += g
        for a, g in zip(accb, b1): a += g
    assert accl == pytest.approx(loss, rel=1e-13)
    for a, g in zip(accW + accb, dW + db):
        assert np.allclose(a, g, rtol=1e-12, atol=1e-13)
    # ragged chunking 5 + 11 + 8
    accW = [np.zeros_like(g) for g in dW]
    for lo, hi in [(0, 5), (5, 16), (16, 24)]:
        _, w1, _ = oracle.mlp_gradient(Ws, bs, X[lo:hi], y[lo:hi])
        for a, g in zip(accW, w1): a += g
    for a, g in zip(accW, dW):
        assert np.allclose(a, g, rtol=1e-12, atol=1e-13)
    # permutation of the patterns
    perm = np.random.default_rng(3).permutation(n)
    loss2, dW2, _ = oracle.mlp_gradient(Ws, bs, X[perm], y[perm])
    assert loss2 == pytest.approx(loss, rel=1e-13)
    for a, g in zip(dW2, dW):
        assert np.allclose(a, g, rtol=1e-12, atol=1e-13)


def test_leading_dimension_of_x_is_respected():
    sizes = [6, 5, 4]
    Ws, bs = _random_net(18, sizes)
    X, y = si.mlp_batch(18, sizes, 8)
    l0, w0, _ = oracle.mlp_gradient(Ws, bs, X, y)
    # a view with junk columns must be made contiguous by the wrapper: same numbers
    big = np.full((8, 11), 7.0, np.float32); big[:, :6] = X
    l1, w1, _ = oracle.mlp_gradient(Ws, bs, big[:, :6], y)
    assert l1 == l0 and all(np.array_equal(a, b) for a, b in zip(w0, w1))


def test_sgd_step_closed_form():
    w = np.array([1.0, -2.0, 0.5, 3.0], np.float32); g = np.array([4.0, 8.0, -16.0, 0.0], np.float32)
    assert oracle.sgd_step(w, g, 0.25).tolist() == [0.0, -4.0, 4.5, 3.0]
    # within half an ulp of the exact real-number result
    w = si.uniform_pm1(19, 1, 1000); g = si.uniform_pm1(19, 2, 1000)
    out = oracle.sgd_step(w, g, 1e-3)
    exact = w.astype(np.float64) - 1e-3 * g.astype(np.float64)
    assert np.all(np.abs(out.astype(np.float64) - exact) <= 0.5 * np.spacing(np.abs(exact).astype(np.float32)).astype(np.float64) + 1e-300)


def test_untrained_classifier_loss_is_near_ln_classes():
    # N(0,1/fan_in) weights: logits are O(1), so the summed loss sits a little above n*ln(n_o)
    sizes = [256, 128, 64]
    Ws, bs = si.mlp_params(0, sizes)
    X, y = si.mlp_batch(0, sizes, 512)
    loss = oracle.mlp_forward_loss(Ws, bs, X, y)
    assert 512 * math.log(64) < loss < 1.2 * 512 * math.log(64)


# ----------------------------------------------------------------------------- magnitude sums and condition numbers

@pytest.mark.parametrize("transA", ["N", "T"])
@pytest.mark.parametrize("transB", ["N", "T"])
def test_sgemm_abs_small_integers_exact(transA, transB):
    # |alpha| sum_k |a||b| + |beta||c| against a pure-Python loop; equal to the product itself when nothing is negative
    rng = np.random.default_rng(11)
    M, N, K = 4, 3, 5
    ra, ca = (K, M) if transA == "T" else (M, K)
    rb, cb = (N, K) if transB == "T" else (K, N)
    A = rng.integers(-4, 5, (ra, ca)).astype(np.float32); B = rng.integers(-4, 5, (rb, cb)).astype(np.float32)
    C = rng.integers(-4, 5, (M, N)).astype(np.float32)
    got = oracle.sgemm_abs(transA, transB, M, N, K, -3.0, A, ca, B, cb, -2.0, C, N)
    want = _brute(transA, transB, M, N, K, 3.0, np.abs(A).tolist(), np.abs(B).tolist(), 2.0, np.abs(C).tolist())
    assert np.array_equal(got, np.asarray(want, dtype=np.float64))
    pos = oracle.sgemm(transA, transB, M, N, K, 3.0, np.abs(A), ca, np.abs(B), cb, 2.0, np.abs(C), N)
    assert np.array_equal(got, pos)


def test_gradient_magnitudes_hand_worked_2_1_2():
    # the hand-worked network: softmax (2/3, 1/3), label 0 -> output magnitudes (2/3 + 1, 1/3), h = 1/2,
    # hidden magnitude (1 - h^2) * (|2 ln 2| * 5/3 + 0 * 1/3)
    with open(os.path.join(GOLD, "hand_net_2_1_2.json")) as f:
        g = json.load(f)
    W1 = np.asarray(_ev(g["W1"]), np.float32); W2 = np.asarray(_ev(g["W2"]), np.float32)
    b1 = np.asarray(_ev(g["b1"]), np.float32); b2 = np.asarray(_ev(g["b2"]), np.float32)
    X = np.asarray([_ev(g["x"])], np.float32)
    aW, ab = oracle.mlp_gradient_abs([W1, W2], [b1, b2], X, labels=np.asarray([0], np.int32))
    m1 = 0.75 * (2 * math.log(2) * 5 / 3)
    # fp32 storage of ln(3)/2 and 2 ln 2 moves the values by ~1e-8 relative
    assert np.allclose(ab[1], [5 / 3, 1 / 3], rtol=1e-6) and np.allclose(aW[1], [[5 / 6], [1 / 6]], rtol=1e-6)
    assert np.allclose(ab[0], [m1], rtol=1e-6) and np.allclose(aW[0], [[m1, 0.0]], rtol=1e-6)


@pytest.mark.parametrize("head", ["softmax", "sse"])
def test_gradient_magnitudes_bound_the_gradient(head):
    sizes, n = [6, 5, 4, 3], 40
    Ws, bs = si.mlp_params(21, sizes)
    bs = [(0.3 * si.uniform_pm1(21, 11 + i, b.size)).astype(np.float32) for i, b in enumerate(bs)]
    X, y = si.mlp_batch(21, sizes, n)
    T = si.mlp_targets(21, sizes, n)
    if head == "softmax":
        _, gW, gb = oracle.mlp_gradient(Ws, bs, X, y); aW, ab = oracle.mlp_gradient_abs(Ws, bs, X, labels=y)
    else:
        _, gW, gb = oracle.mlp_sse_gradient(Ws, bs, X, T); aW, ab = oracle.mlp_gradient_abs(Ws, bs, X, T=T)
    for g_, a_ in zip(gW + gb, aW + ab):
        assert (a_ >= np.abs(g_) * (1 - 1e-12)).all() and (a_ > 0).all()
    # one pattern, one weight matrix, squared-error head: every entry is a single product, so magnitude = |gradient|
    _, g1W, g1b = oracle.mlp_sse_gradient(Ws[:1], bs[:1], X[:1], T[:1, :sizes[1]])
    a1W, a1b = oracle.mlp_gradient_abs(Ws[:1], bs[:1], X[:1], T=T[:1, :sizes[1]])
    assert np.allclose(a1W[0], np.abs(g1W[0]), rtol=1e-13) and np.allclose(a1b[0], np.abs(g1b[0]), rtol=1e-13)


def test_gradient_condition_of_a_gradient_linear_in_the_pattern():
    # all-zero parameters, one pattern: dW = (1/n_o - onehot) x^T does not depend on W and is linear in x, so its
    # relative change under x -> x~ is ||x~ - x|| / ||x|| exactly; db does not depend on x at all
    sizes = [7, 4]
    W = [np.zeros((4, 7), np.float32)]; b = [np.zeros(4, np.float32)]
    X = (0.25 + si.uniform01(5, si.TID_X, 7)).reshape(1, 7).astype(np.float32)
    y = np.asarray([2], np.int32)
    eps, seeds = 2.0 ** -14, (12345, 12346)
    cW, cb = oracle.gradient_condition(W, b, X, labels=y, eps=eps, seeds=seeds)
    want = 0.0
    for s in seeds:
        _, _, Xp, _ = oracle.perturb_inputs(W, b, X, None, eps, s)
        want = max(want, np.linalg.norm((Xp.astype(np.float64) - X).ravel()) / np.linalg.norm(X.astype(np.float64).ravel()))
    assert abs(cW[0] - want / (eps / math.sqrt(3))) < 1e-6 * cW[0]
    assert 0.3 < cW[0] < 3.0 and cb[0] == 0.0


def test_condition_reference_of_the_benchmark_network_is_stored():
    with open(os.path.join(GOLD, "cond_ref.json")) as f:
        ref = json.load(f)
    vals = ref["softmax"]["dW"] + ref["softmax"]["db"] + ref["sse"]["dW"] + ref["sse"]["db"]
    assert ref["cond_ref"] == max(vals) and all(0.5 < v < 3.0 for v in vals)
    # a 1/16 sample of the stored configuration reproduces the weight-gradient values, which set the maximum, to
    # 15 % (they do not depend on the batch; the top bias gradient's does: its label counts are exact)
    sizes = [400, 480, 3203]
    Ws, bs = si.mlp_params(2, sizes)
    X, y = si.mlp_batch(2, sizes, 512)
    cW, cb = oracle.gradient_condition(Ws, bs, X, labels=y, seeds=(12345,))
    for got, want in zip(cW + cb[:1], ref["softmax"]["dW"] + ref["softmax"]["db"][:1]):
        assert abs(got - want) < 0.15 * want
