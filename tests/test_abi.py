"""The C-ABI library loads without a GPU, exports what include/ulsnn.h declares, and rejects bad
arguments on the host before touching the device."""
import ctypes
import os
import re

import pytest

from paper_1911_05181_b200 import binding as ul, buildlib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    buildlib.build()


def test_every_declared_symbol_is_exported():
    hdr = open(os.path.join(ROOT, "include", "ulsnn.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = sorted(set(re.findall(r"\b(ulsnn_[a-z0-9_]+)\s*\(", hdr)))
    assert len(declared) >= 14
    lib = ctypes.CDLL(ul.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(declared) == sorted(ul.EXPORTS)


def test_version_and_status_strings():
    assert ul.version() >= 100
    assert ul.status_string(ul.OK) == "ok"
    for s in (ul.ERR_INVALID_ARG, ul.ERR_UNSUPPORTED_ARCH, ul.ERR_WORKSPACE_TOO_SMALL, ul.ERR_CUDA,
              ul.ERR_DEVICE_TIMEOUT, ul.ERR_TOO_LARGE):
        assert ul.status_string(s) not in ("ok", "unknown status")


@pytest.mark.parametrize("args", [
    ("X", "N", 4, 4, 4, 4, 4, 4),      # bad trans
    ("N", "Q", 4, 4, 4, 4, 4, 4),
    ("N", "N", -1, 4, 4, 4, 4, 4),     # negative size
    ("N", "N", 4, 4, -2, 4, 4, 4),
    ("N", "N", 4, 4, 8, 7, 4, 4),      # lda < K
    ("T", "N", 8, 4, 4, 7, 4, 4),      # lda < M when A is transposed
    ("N", "N", 4, 8, 4, 4, 7, 8),      # ldb < N
    ("N", "T", 4, 4, 8, 8, 7, 4),      # ldb < K when B is transposed
    ("N", "N", 4, 8, 4, 4, 8, 7),      # ldc < N
])
def test_sgemm_rejects_bad_arguments_on_the_host(args):
    ta, tb, M, N, K, lda, ldb, ldc = args
    fake = 4096   # never dereferenced: validation comes first
    assert ul.sgemm(ta, tb, M, N, K, 1.0, fake, lda, fake, ldb, 0.0, fake, ldc, stream=0, check=False) == ul.ERR_INVALID_ARG
    assert ul.sgemm_ex(ta, tb, M, N, K, 1.0, fake, lda, fake, ldb, 0.0, fake, ldc, ul.MATH_FP32_SIMT, None, 0,
                       stream=0, check=False) == ul.ERR_INVALID_ARG


def test_sgemm_bad_math_and_empty_products():
    fake = 4096
    assert ul.sgemm_ex("N", "N", 4, 4, 4, 1.0, fake, 4, fake, 4, 0.0, fake, 4, 7, None, 0, stream=0, check=False) == ul.ERR_INVALID_ARG
    # M == 0 or N == 0: nothing to do, no device needed
    assert ul.sgemm("N", "N", 0, 4, 4, 1.0, fake, 4, fake, 4, 0.0, fake, 4, stream=0, check=False) == ul.OK
    assert ul.sgemm("N", "N", 4, 0, 4, 1.0, fake, 4, fake, 1, 0.0, fake, 1, stream=0, check=False) == ul.OK


def test_workspace_queries_are_host_only():
    assert ul.sgemm_workspace_bytes("N", "N", 4096, 4096, 4096, ul.MATH_FP32_SIMT) == 0
    # short-and-wide with a long K is split: slices x M x ld4(N) floats
    b = ul.sgemm_workspace_bytes("T", "N", 480, 3203, 65536, ul.MATH_FP32_SIMT)
    assert b > 0 and b % 256 == 0 and b % (480 * 3204 * 4) < 256
    with pytest.raises(ul.UlsnnError):
        ul.sgemm_workspace_bytes("N", "N", -1, 4, 4)
    small = ul.mlp_workspace_bytes([256, 128, 64], ul.MATH_FP32_SIMT, 4096)
    big = ul.mlp_workspace_bytes([400, 480, 3203], ul.MATH_FP32_SIMT, 65536)
    assert 0 < small < big
    # logits alone are 65536 x 3204 floats
    assert big > 65536 * 3204 * 4
    for bad in ([4], [4, 0, 3], [4, -1]):
        with pytest.raises(ul.UlsnnError):
            ul.mlp_workspace_bytes(bad, ul.MATH_FP32_SIMT, 16)
    with pytest.raises(ul.UlsnnError):
        ul.mlp_workspace_bytes([4, 3], ul.MATH_FP32_SIMT, 0)
    with pytest.raises(ul.UlsnnError):
        ul.mlp_workspace_bytes([4, 3], 9, 16)


def test_mlp_create_rejects_bad_workspace():
    lib = ul.lib()
    arr = (ctypes.c_int32 * 3)(8, 4, 2)
    d = ul._Desc(2, arr, ul.MATH_FP32_SIMT, 32)
    h = ctypes.c_void_p(None)
    need = ul.mlp_workspace_bytes([8, 4, 2], ul.MATH_FP32_SIMT, 32)
    assert lib.ulsnn_mlp_create(ctypes.byref(h), ctypes.byref(d), None, need) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_mlp_create(ctypes.byref(h), ctypes.byref(d), 4096 + 16, need) == ul.ERR_INVALID_ARG      # misaligned
    assert lib.ulsnn_mlp_create(ctypes.byref(h), ctypes.byref(d), 4096, need - 1) == ul.ERR_WORKSPACE_TOO_SMALL
    assert lib.ulsnn_mlp_create(ctypes.byref(h), ctypes.byref(d), 4096, need) == ul.OK and h.value
    # calls on the handle validate before using the device
    fake = ctypes.c_void_p(4096)
    ptrs = (ctypes.c_void_p * 2)(4096, 4096)
    assert lib.ulsnn_mlp_forward_loss(h, ptrs, ptrs, fake, 8, fake, 33, fake, None) == ul.ERR_INVALID_ARG     # n > max_patterns
    assert lib.ulsnn_mlp_forward_loss(h, ptrs, ptrs, fake, 7, fake, 4, fake, None) == ul.ERR_INVALID_ARG      # ldx < n_0
    assert lib.ulsnn_mlp_gradient(h, ptrs, ptrs, fake, 8, fake, 4, 0, None, ptrs, fake, None) == ul.ERR_INVALID_ARG
    nulls = (ctypes.c_void_p * 2)(4096, None)
    assert lib.ulsnn_mlp_gradient(h, nulls, ptrs, fake, 8, fake, 4, 0, ptrs, ptrs, fake, None) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_sgd_step(h, ptrs, ptrs, nulls, ptrs, 0.1, None) == ul.ERR_INVALID_ARG
    lib.ulsnn_mlp_destroy(h)


def test_fill_rejects_bad_arguments():
    lib = ul.lib()
    assert lib.ulsnn_fill_uniform(4096, -1, 0, 0, 0, 0, None) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_fill_uniform(4096, 4, 0, 0, 0, 5, None) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_fill_labels(4096, 4, 0, 0, 0, 0, None) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_fill_uniform(None, 0, 0, 0, 0, 0, None) == ul.OK


def test_vector_calls_reject_bad_arguments_on_the_host():
    fake = 4096
    out = ctypes.c_size_t(0)
    lib = ul.lib()
    assert lib.ulsnn_vec_dot_workspace_bytes(-1, ctypes.byref(out)) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_vec_dot_workspace_bytes(5000, ctypes.byref(out)) == ul.OK and out.value >= 6 * 8
    assert lib.ulsnn_vec_dot(10, fake, fake, None, fake, 4096, None) == ul.ERR_INVALID_ARG        # no output
    assert lib.ulsnn_vec_dot(10, None, fake, fake, fake, 4096, None) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_vec_dot(5000, fake, fake, fake, fake, 8, None) == ul.ERR_WORKSPACE_TOO_SMALL
    assert lib.ulsnn_vec_axpby(-3, 1.0, fake, 1.0, fake, fake, None) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_vec_axpby(0, 1.0, None, 1.0, None, None, None) == ul.OK


def test_squared_error_head_rejects_bad_arguments_on_the_host():
    sizes = [8, 4, 3]
    nbytes = ul.mlp_workspace_bytes(sizes, ul.MATH_FP32_SIMT, 16)
    arr = (ctypes.c_int32 * 3)(*sizes)
    d = ul._Desc(2, arr, ul.MATH_FP32_SIMT, 16)
    h = ctypes.c_void_p(None)
    assert ul.lib().ulsnn_mlp_create(ctypes.byref(h), ctypes.byref(d), 4096, nbytes) == ul.OK     # 4096: aligned, never touched
    fake = 8192
    ptrs = (ctypes.c_void_p * 2)(fake, fake)
    lib = ul.lib()
    assert lib.ulsnn_mlp_forward_sse(h, ptrs, ptrs, fake, 8, None, 3, 4, fake, None) == ul.ERR_INVALID_ARG      # no targets
    assert lib.ulsnn_mlp_forward_sse(h, ptrs, ptrs, fake, 8, fake, 2, 4, fake, None) == ul.ERR_INVALID_ARG      # ldt < classes
    assert lib.ulsnn_mlp_forward_sse(h, ptrs, ptrs, fake, 7, fake, 3, 4, fake, None) == ul.ERR_INVALID_ARG      # ldx < inputs
    assert lib.ulsnn_mlp_gradient_sse(h, ptrs, ptrs, fake, 8, fake, 3, 17, 0, ptrs, ptrs, fake, None) == ul.ERR_INVALID_ARG   # n > max
    assert lib.ulsnn_mlp_gradient_sse(h, ptrs, ptrs, fake, 8, fake, 3, 4, 0, None, ptrs, fake, None) == ul.ERR_INVALID_ARG
    lib.ulsnn_mlp_destroy(h)


def test_sixteen_bit_mode_workspaces():
    # the bf16 SGEMM always needs room for its two operand copies (rows padded to 8 elements), split or not
    b = ul.sgemm_workspace_bytes("N", "N", 4096, 4096, 4096, ul.MATH_BF16)
    assert b == 2 * 4096 * 4096 * 2
    b = ul.sgemm_workspace_bytes("N", "T", 100, 50, 30, ul.MATH_BF16)
    assert b % 256 == 0 and b >= 100 * 32 * 2 + 50 * 32 * 2
    # the network keeps bfloat16 activations, exponentials and deltas: well under the fp32 modes' workspace
    half = ul.mlp_workspace_bytes([400, 480, 3203], ul.MATH_BF16, 65536)
    full = ul.mlp_workspace_bytes([400, 480, 3203], ul.MATH_TF32, 65536)
    assert 65536 * 3208 * 2 < half < 0.7 * full
    with pytest.raises(ul.UlsnnError):
        ul.mlp_workspace_bytes([400, 480, 3203], 4, 65536)


def test_per_device_tables_key_on_the_device_ordinal():
    # every per-device cache of the library (architecture check, SM count, status-word address, kernel attributes,
    # scratch buffers) is indexed by this slot: distinct devices get distinct slots, ordinals outside the table none
    slots = [ul.device_cache_slot(d) for d in range(64)]
    assert slots == list(range(64))
    assert ul.device_cache_slot(-1) == -1 and ul.device_cache_slot(64) == -1 and ul.device_cache_slot(1 << 20) == -1


def test_workspace_query_for_given_operands_is_host_only():
    # no device: no operand is addressable by TMA and no tensor-core route exists, so the query equals the plain one;
    # bad arguments are refused
    for math in (ul.MATH_3XTF32, ul.MATH_TF32, ul.MATH_FP32_SIMT):
        got = ul.sgemm_workspace_bytes_for("T", "N", 96, 200, 20000, 256, 96, 512, 200, math)
        assert got >= 0
    out = ctypes.c_size_t(0)
    lib = ul.lib()
    assert lib.ulsnn_sgemm_workspace_bytes_for(b"N", b"N", 4, 4, 4, None, 3, None, 4, 0, ctypes.byref(out)) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_sgemm_workspace_bytes_for(b"N", b"N", 4, 4, 4, None, 4, None, 4, 0, None) == ul.ERR_INVALID_ARG
    assert lib.ulsnn_sgemm_workspace_bytes_for(b"N", b"N", 4, 4, 4, None, 4, None, 4, 9, ctypes.byref(out)) == ul.ERR_INVALID_ARG
