"""Seeded random shapes through every math mode: SGEMM forms (Section 3.1) and small networks with both output heads
(Section 4.2), each checked against the CPU checker.  The shape lists mix tile multiples with their neighbours
(127/128/129, 255/256/257), tiny sizes and one long K."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_1911_05181_b200 import binding as ul
from helpers import TOL, GpuNet, dev, gpu_sgemm, tolerance_at

pytestmark = pytest.mark.gpu

MATHS = [ul.MATH_3XTF32, ul.MATH_TF32, ul.MATH_BF16, ul.MATH_FP32_SIMT]


@pytest.mark.parametrize("seed", [1, 2])
def test_random_sgemm_shapes(seed):
    rng = np.random.default_rng(seed)
    for it in range(40):
        M = int(rng.choice([1, 7, 64, 127, 128, 129, 255, 256, 257, 300, 511, 640, 1000]))
        N = int(rng.choice([1, 5, 8, 31, 32, 33, 64, 100, 128, 200, 255, 256, 257, 320, 481, 700]))
        K = int(rng.choice([1, 3, 8, 31, 32, 33, 63, 64, 65, 100, 256, 257, 480, 1000, 3203, 9000]))
        if M * N * K > 6e7:
            K = max(1, int(6e7 / (M * N)))
        ta, tb = str(rng.choice(["N", "T"])), str(rng.choice(["N", "T"]))
        pad = int(rng.choice([0, 0, 1, 3, 4, 8]))
        alpha = float(rng.choice([1.0, -0.5, 2.0])); beta = float(rng.choice([0.0, 1.0, 0.25]))
        ra, ca = (K, M) if ta == "T" else (M, K)
        rb, cb = (N, K) if tb == "T" else (K, N)
        lda, ldb, ldc = ca + pad, cb + pad, N + pad
        A, B, C = si.gemm_operands(100 * seed + it, ra, lda, rb, ldb, M, ldc)
        want = oracle.sgemm(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C.copy(), ldc)
        for math in MATHS:
            C1 = C.copy()
            if beta == 0.0:
                C1[:, :N] = np.nan
            got = gpu_sgemm(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C1, ldc, math)
            assert oracle.rel_l2(got[:, :N], want) <= TOL[math], (ta, tb, M, N, K, pad, alpha, beta, math)
            if pad:
                assert np.array_equal(got[:, N:], C[:, N:])


def test_random_networks_both_heads():
    rng = np.random.default_rng(3)
    for it in range(16):
        L = int(rng.integers(1, 4))
        sizes = [int(rng.choice([3, 8, 20, 33, 64, 100, 129, 256, 400])) for _ in range(L + 1)]
        n = int(rng.choice([1, 5, 64, 127, 128, 129, 300, 1000, 2500]))
        seed = 500 + it
        Ws, bs = si.mlp_params(seed, sizes)
        bs = [(0.2 * si.uniform_pm1(seed, 11 + i, b.size)).astype(np.float32) for i, b in enumerate(bs)]
        X, y = si.mlp_batch(seed, sizes, n)
        T = si.mlp_targets(seed, sizes, n, 0, False)
        want = oracle.mlp_gradient(Ws, bs, X, y)
        want_sse = oracle.mlp_sse_gradient(Ws, bs, X, T)
        # Every tensor is compared at the stated tolerance times max(1, its condition number / that of the benchmark
        # network's worst tensor): layers of a few units make gradients whose relative sensitivity to perturbations
        # of the inputs is several times the benchmark's, and no evaluation in finite precision can be held to more
        cond = oracle.gradient_condition(Ws, bs, X, labels=y)
        cond_sse = oracle.gradient_condition(Ws, bs, X, T=T)
        for math in MATHS:
            g = GpuNet(sizes, math, n); g.set_params(Ws, bs)
            got = g.gradient(X, y)
            g.net.gradient_sse(g.W, g.b, dev(X), sizes[0], dev(T), sizes[-1], n, False, g.dW, g.db, g.loss)
            torch.cuda.synchronize()
            got_sse = (float(g.loss.item()), [t.cpu().numpy() for t in g.dW], [t.cpu().numpy() for t in g.db])
            for head, a, b, c in (("softmax", got, want, cond), ("sse", got_sse, want_sse, cond_sse)):
                assert abs(a[0] - b[0]) <= TOL[math] * abs(b[0]), (sizes, n, math, head)
                for u, v, k in zip(a[1] + a[2], b[1] + b[2], c[0] + c[1]):
                    assert oracle.rel_l2(u, v) <= tolerance_at(math, k, head), (sizes, n, math, head, k)
            assert g.net.last_device_status() == ul.OK
            g.net.close()
