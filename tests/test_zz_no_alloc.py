"""ulsnn_sgemm_noalloc: SGEMM for callers that may not allocate device memory.

A caller that runs under a fixed memory budget, or inside a host framework that owns every allocation, cannot hand
ulsnn_sgemm_ex a workspace and cannot live with the allocate-on-first-need of ulsnn_sgemm.  The no-alloc entry point
takes its split-K scratch from a fixed 8 MiB array inside the library instead.  These tests call it through the C-ABI
and hold its output against ulsnn_sgemm_ex on the same operands, twice in a row (the second call finds the array dirty
from the first, and from a different product).  The file name makes pytest collect it last.
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_1911_05181_b200 import binding as ul
from helpers import TOL, dev

pytestmark = pytest.mark.gpu


def _operands(ta, tb, M, N, K, seed):
    ra, ca = (K, M) if ta == "T" else (M, K)
    rb, cb = (N, K) if tb == "T" else (K, N)
    A, B, C = si.gemm_operands(seed, ra, ca, rb, cb, M, N)
    return A, ca, B, cb, C, N


def _ex(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, math):
    dA, dB = dev(A), dev(B)
    nbytes = ul.sgemm_workspace_bytes_for(ta, tb, M, N, K, dA, lda, dB, ldb, math)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    wp = (ws.data_ptr() + 255) // 256 * 256
    dC = dev(C)
    ul.sgemm_ex(ta, tb, M, N, K, alpha, dA, lda, dB, ldb, beta, dC, ldc, math, wp if nbytes else None, nbytes)
    torch.cuda.synchronize()
    return dC.cpu().numpy(), nbytes


def _noalloc(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, math):
    dA, dB, dC = dev(A), dev(B), dev(C)      # inputs and outputs still come from the caller
    torch.cuda.synchronize()
    ul.sgemm_noalloc(ta, tb, M, N, K, alpha, dA, lda, dB, ldb, beta, dC, ldc, math)
    torch.cuda.synchronize()
    return dC.cpu().numpy()


@pytest.mark.parametrize("math", [ul.MATH_3XTF32, ul.MATH_FP32_SIMT, ul.MATH_TF32])
def test_two_calls_in_a_row_match_the_workspace_entry_point(math):
    # two different split-K products back to back: the second one reuses the array the first one filled
    cases = [("T", "N", 96, 200, 20000, 1.0, 1.0, 7), ("T", "N", 130, 64, 9000, 1.5, 0.0, 8)]
    for ta, tb, M, N, K, alpha, beta, seed in cases:
        A, lda, B, ldb, C, ldc = _operands(ta, tb, M, N, K, seed)
        want, nbytes = _ex(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, math)
        assert 0 < nbytes <= ul.sgemm_noalloc_max_scratch_bytes()        # the case really uses the scratch
        got = _noalloc(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, math)
        assert oracle.rel_l2(got, want) <= TOL[math]
        assert np.array_equal(got, want)                                  # same slice plan, same order: same bits
        again = _noalloc(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, math)
        assert np.array_equal(again, got)
        ref = oracle.sgemm(ta, tb, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc)
        assert oracle.rel_l2(got, ref) <= TOL[math]


def test_products_without_split_and_oversized_products():
    # no split-K needed: the array is not touched, the result is that of the workspace entry point
    A, lda, B, ldb, C, ldc = _operands("N", "T", 300, 260, 132, 9)
    want, nbytes = _ex("N", "T", 300, 260, 132, 1.0, A, lda, B, ldb, 0.0, C, ldc, ul.MATH_3XTF32)
    assert nbytes == 0
    got = _noalloc("N", "T", 300, 260, 132, 1.0, A, lda, B, ldb, 0.0, C, ldc, ul.MATH_3XTF32)
    assert np.array_equal(got, want)
    # the weight-gradient shape of the 400-480-3203 network wants 98 MB of partials: refused, nothing launched
    M, N, K = 480, 3203, 65536
    assert ul.sgemm_workspace_bytes("T", "N", M, N, K, ul.MATH_3XTF32) > ul.sgemm_noalloc_max_scratch_bytes()
    a = torch.zeros(K, M, device="cuda"); b = torch.zeros(K, N + 1, device="cuda")
    c = torch.full((M, N), 7.0, device="cuda")
    st = ul.sgemm_noalloc("T", "N", M, N, K, 1.0, a, M, b, N + 1, 0.0, c, N, ul.MATH_3XTF32, check=False)
    assert st == ul.ERR_TOO_LARGE
    torch.cuda.synchronize()
    assert bool((c == 7.0).all())


def test_sixteen_bit_mode_padded_rows_and_degenerate_products():
    """The branches the two-call test leaves out.  The 16-bit mode keeps its bfloat16 operand copies in the array as well, so
    only small products fit; operands whose rows TMA cannot address are re-buffered in the array when copies and partials
    fit; K == 0 and alpha == 0 touch neither operands nor array.  Each is held bit for bit against the workspace entry point."""
    # 16-bit mode, accepted: copies of A (128 x 2048) and B (2048 x 96) plus partials are well below 8 MiB
    for _ in range(2):
        A, lda, B, ldb, C, ldc = _operands("N", "N", 128, 96, 2048, 11)
        want, nbytes = _ex("N", "N", 128, 96, 2048, 1.0, A, lda, B, ldb, 0.5, C, ldc, ul.MATH_BF16)
        assert 0 < nbytes <= ul.sgemm_noalloc_max_scratch_bytes()
        got = _noalloc("N", "N", 128, 96, 2048, 1.0, A, lda, B, ldb, 0.5, C, ldc, ul.MATH_BF16)
        assert np.array_equal(got, want)
        assert oracle.rel_l2(got, oracle.sgemm("N", "N", 128, 96, 2048, 1.0, A, lda, B, ldb, 0.5, C, ldc)) <= TOL[ul.MATH_BF16]
    # 16-bit mode, rejected: the copies alone (2 x 2048 x 2048 bfloat16 = 16 MiB) exceed the array
    z = torch.zeros(2048, 2048, device="cuda"); c = torch.full((2048, 2048), 3.0, device="cuda")
    assert ul.sgemm_noalloc("N", "N", 2048, 2048, 2048, 1.0, z, 2048, z, 2048, 0.0, c, 2048, ul.MATH_BF16, check=False) == ul.ERR_TOO_LARGE
    torch.cuda.synchronize()
    assert bool((c == 3.0).all())
    # rows of 130 floats (not a multiple of 4): copies and partials fit, both entry points take the re-buffered route
    for math in (ul.MATH_3XTF32, ul.MATH_TF32):
        A, lda, B, ldb, C, ldc = _operands("T", "N", 130, 66, 9000, 12)
        want, nbytes = _ex("T", "N", 130, 66, 9000, 1.5, A, lda, B, ldb, 1.0, C, ldc, math)
        assert 0 < nbytes <= ul.sgemm_noalloc_max_scratch_bytes()
        got = _noalloc("T", "N", 130, 66, 9000, 1.5, A, lda, B, ldb, 1.0, C, ldc, math)
        assert np.array_equal(got, want)
        assert oracle.rel_l2(got, oracle.sgemm("T", "N", 130, 66, 9000, 1.5, A, lda, B, ldb, 1.0, C, ldc)) <= TOL[math]
    # K == 0 and alpha == 0: C = beta * C, operands never read (they hold NaN)
    nan = np.full((8, 8), np.nan, np.float32); C = si.uniform_pm1(3, 9, 64).reshape(8, 8)
    for math in (ul.MATH_3XTF32, ul.MATH_BF16):
        assert np.array_equal(_noalloc("N", "N", 8, 8, 0, 1.0, nan, 8, nan, 8, 2.0, C.copy(), 8, math), 2.0 * C)
        assert np.array_equal(_noalloc("N", "N", 8, 8, 8, 0.0, nan, 8, nan, 8, 1.0, C.copy(), 8, math), C)
