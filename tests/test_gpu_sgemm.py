"""SGEMM parity (Section 3.1) of the CUDA path against the CPU checker, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_1911_05181_b200 import binding as ul
from helpers import TOL, gpu_sgemm, dev

pytestmark = pytest.mark.gpu

MATHS = [ul.MATH_FP32_SIMT, ul.MATH_3XTF32, ul.MATH_TF32, ul.MATH_BF16]


def _stored(trans_a, trans_b, M, N, K, pad, seed=1):
    ra, ca = (K, M) if trans_a == "T" else (M, K)
    rb, cb = (N, K) if trans_b == "T" else (K, N)
    lda, ldb, ldc = ca + pad, cb + pad, N + pad
    A, B, C = si.gemm_operands(seed, ra, lda, rb, ldb, M, ldc)
    return A, lda, B, ldb, C, ldc


def _check(ta, tb, M, N, K, alpha, beta, pad, math, use_plain=False):
    A, lda, B, ldb, C, ldc = _stored(ta, tb, M, N, K, pad)
    C0 = C.copy()
    if beta == 0.0:
        C[:, :N] = np.nan                       # beta == 0 must not read C
    got = gpu_sgemm(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, math, use_plain)
    want = oracle.sgemm(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C0, ldc)
    err = oracle.rel_l2(got[:, :N], want)
    assert err <= TOL[math], (err, ta, tb, M, N, K, math)
    if pad:                                      # columns beyond N are the caller's: untouched
        assert np.array_equal(got[:, N:], C[:, N:])


@pytest.mark.parametrize("math", MATHS)
@pytest.mark.parametrize("ta", ["N", "T"])
@pytest.mark.parametrize("tb", ["N", "T"])
def test_all_forms_ragged(math, ta, tb):
    # several 128-wide tiles plus a ragged tail in every dimension; ld > width
    _check(ta, tb, 300, 391, 203, 1.0, 0.0, 5, math)
    _check(ta, tb, 257, 130, 77, -0.5, 1.0, 3, math)


@pytest.mark.parametrize("math", MATHS)
@pytest.mark.parametrize("ta,tb", [("N", "T"), ("N", "N"), ("T", "N"), ("T", "T")])
def test_tma_friendly_shapes(math, ta, tb):
    # leading dimensions that are multiples of 4 and 16-byte aligned bases: the tensor-core route
    _check(ta, tb, 384, 512, 256, 1.0, 0.0, 0, math)
    _check(ta, tb, 200, 260, 132, 2.0, 1.0, 4, math)


@pytest.mark.parametrize("math", MATHS)
@pytest.mark.parametrize("size", [256, 1024])
def test_square(math, size):
    _check("N", "N", size, size, size, 1.0, 1.0, 0, math)


@pytest.mark.parametrize("math", MATHS)
def test_split_k_long_sum(math):
    # few output tiles, long K: the split-K path with its fixed-order reduction (the weight-gradient shape)
    _check("T", "N", 96, 200, 20000, 1.0, 1.0, 0, math)
    _check("T", "N", 130, 60, 9000, 1.5, 0.0, 4, math)


@pytest.mark.parametrize("math", MATHS)
def test_tiny_and_degenerate(math):
    _check("N", "N", 1, 1, 1, 1.0, 0.0, 0, math)
    _check("N", "T", 3, 2, 5, 1.0, 1.0, 1, math)
    # K == 0 -> C = beta*C ; alpha == 0 -> C = beta*C without reading A, B
    A = np.full((4, 4), np.nan, np.float32); C = si.uniform_pm1(3, 9, 16).reshape(4, 4)
    out = gpu_sgemm("N", "N", 4, 4, 0, 1.0, A, 4, A, 4, 2.0, C.copy(), 4, math)
    assert np.array_equal(out, 2.0 * C)
    out = gpu_sgemm("N", "N", 4, 4, 4, 0.0, A, 4, A, 4, 0.0, np.full((4, 4), np.nan, np.float32), 4, math)
    assert np.array_equal(out, np.zeros((4, 4), np.float32))
    out = gpu_sgemm("N", "N", 4, 4, 4, 0.0, A, 4, A, 4, 1.0, C.copy(), 4, math)
    assert np.array_equal(out, C)


def test_plain_entry_point_uses_internal_scratch_and_repeats_bitwise():
    A, lda, B, ldb, C, ldc = _stored("T", "N", 100, 180, 12000, 0)
    want = oracle.sgemm("T", "N", 100, 180, 12000, 1.0, A, lda, B, ldb, 0.0)
    r1 = gpu_sgemm("T", "N", 100, 180, 12000, 1.0, A, lda, B, ldb, 0.0, C.copy(), ldc, ul.MATH_3XTF32, use_plain=True)
    r2 = gpu_sgemm("T", "N", 100, 180, 12000, 1.0, A, lda, B, ldb, 0.0, C.copy(), ldc, ul.MATH_3XTF32, use_plain=True)
    assert oracle.rel_l2(r1, want) <= 1e-5
    assert np.array_equal(r1, r2)


def test_workspace_too_small_is_reported():
    A, lda, B, ldb, C, ldc = _stored("T", "N", 96, 200, 20000, 0)
    st = ul.sgemm_ex("T", "N", 96, 200, 20000, 1.0, dev(A), lda, dev(B), ldb, 0.0, dev(C), ldc, ul.MATH_FP32_SIMT,
                     None, 0, check=False)
    assert st == ul.ERR_WORKSPACE_TOO_SMALL


@pytest.mark.parametrize("math", MATHS)
@pytest.mark.parametrize("shape", [(65536, 480, 400, "N", "T"), (8192, 3203, 480, "N", "T"), (480, 3203, 65536, "T", "N"),
                                   (4096, 4096, 4096, "N", "N")])
def test_paper_shapes_sampled(math, shape):
    """The skinny shapes of the network (patterns x hidden x inputs, ...) at full K, checked on sampled entries,
    each a full-length double dot product of the checker."""
    M, N, K, ta, tb = shape
    A, lda, B, ldb, C, ldc = _stored(ta, tb, M, N, K, 0)
    got = gpu_sgemm(ta, tb, M, N, K, 1.0, A, lda, B, ldb, 0.0, C.copy(), ldc, math)
    rng = np.random.default_rng(5)
    ii = rng.integers(0, M, 512); jj = rng.integers(0, N, 512)
    ii[:4] = [0, M - 1, 0, M - 1]; jj[:4] = [0, 0, N - 1, N - 1]
    want = np.array([oracle.sgemm_entry(ta, tb, K, 1.0, A, lda, B, ldb, 0.0, None, 0, int(i), int(j)) for i, j in zip(ii, jj)])
    err = oracle.rel_l2(got[ii, jj], want)
    assert err <= TOL[math], err


@pytest.mark.parametrize("math", [ul.MATH_3XTF32, ul.MATH_TF32])
def test_operands_tma_cannot_address_are_rebuffered_onto_the_tensor_cores(math):
    """Packed rows of 3203 floats (the class count of the paper's network is prime) and a base pointer that is not
    16-byte aligned: with the workspace ulsnn_sgemm_workspace_bytes_for asks for, the product runs on the tensor-core
    engine after a copy with padded rows (Section 3.3's re-buffering); with less, on the FFMA kernel.  Both are right."""
    for ta, tb, M, N, K, off in (("N", "N", 700, 3203, 480, 0), ("T", "N", 480, 3203, 2100, 0), ("N", "T", 300, 130, 203, 1),
                                 ("T", "T", 129, 65, 77, 3)):
        ra, ca = (K, M) if ta == "T" else (M, K)
        rb, cb = (N, K) if tb == "T" else (K, N)
        A, B, C = si.gemm_operands(31, ra, ca, rb, cb, M, N)
        want = oracle.sgemm(ta, tb, M, N, K, 1.0, A, ca, B, cb, 0.5, C.copy(), N)
        # device copies shifted by `off` floats: bases that are 4-byte but not 16-byte aligned
        bufA = torch.empty(A.size + 8, device="cuda"); bufB = torch.empty(B.size + 8, device="cuda")
        dA = bufA[off:off + A.size].view(ra, ca); dB = bufB[off:off + B.size].view(rb, cb)
        dA.copy_(torch.from_numpy(A)); dB.copy_(torch.from_numpy(B))
        plain = ul.sgemm_workspace_bytes(ta, tb, M, N, K, math)
        need = ul.sgemm_workspace_bytes_for(ta, tb, M, N, K, dA, ca, dB, cb, math)
        assert need > plain
        for nbytes, tc_expected in ((need, True), (plain, False)):
            ws = torch.empty(max(nbytes, 1) + 256, dtype=torch.uint8, device="cuda")
            wp = (ws.data_ptr() + 255) // 256 * 256
            dC = dev(C)
            c0 = ul.launch_counts()
            ul.sgemm_ex(ta, tb, M, N, K, 1.0, dA, ca, dB, cb, 0.5, dC, N, math, wp if nbytes else None, nbytes)
            torch.cuda.synchronize()
            c1 = ul.launch_counts()
            assert (c1["tc_gemm"] > c0["tc_gemm"]) == tc_expected and (c1["simt_gemm"] > c0["simt_gemm"]) == (not tc_expected)
            tol = TOL[math] if tc_expected else TOL[ul.MATH_FP32_SIMT]
            assert oracle.rel_l2(dC.cpu().numpy(), want) <= tol, (ta, tb, M, N, K, off, nbytes)
        # the allocating entry point takes the re-buffered route by itself
        if math == ul.MATH_3XTF32:
            dC = dev(C)
            c0 = ul.launch_counts()
            ul.sgemm(ta, tb, M, N, K, 1.0, dA, ca, dB, cb, 0.5, dC, N)
            torch.cuda.synchronize()
            assert ul.launch_counts()["tc_gemm"] > c0["tc_gemm"]
            assert oracle.rel_l2(dC.cpu().numpy(), want) <= TOL[math]
