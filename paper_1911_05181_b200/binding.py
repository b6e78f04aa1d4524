"""ctypes binding of the C-ABI in include/ulsnn.h: same names, argument marshalling only.

Every function takes device buffers as objects with a `data_ptr()` method (torch tensors) or as
integer addresses, and a stream as `None` (torch's current stream), a `torch.cuda.Stream` or an
integer handle.  Nothing is computed here; a missing library is an error, never a fallback.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libulsnn.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED_ARCH = -2
ERR_WORKSPACE_TOO_SMALL = -3
ERR_CUDA = -4
ERR_DEVICE_TIMEOUT = -5
ERR_TOO_LARGE = -6

MATH_3XTF32 = 0
MATH_TF32 = 1
MATH_FP32_SIMT = 2
MATH_BF16 = 3
MATH_NAMES = {MATH_3XTF32: "3xtf32", MATH_TF32: "tf32", MATH_FP32_SIMT: "fp32_simt", MATH_BF16: "bf16"}

EXPORTS = [
    "ulsnn_status_string", "ulsnn_version", "ulsnn_sgemm", "ulsnn_sgemm_ex", "ulsnn_sgemm_workspace_bytes",
    "ulsnn_mlp_workspace_bytes", "ulsnn_mlp_create", "ulsnn_mlp_destroy", "ulsnn_mlp_forward_loss",
    "ulsnn_mlp_gradient", "ulsnn_sgd_step", "ulsnn_last_device_status", "ulsnn_fill_uniform",
    "ulsnn_fill_labels", "ulsnn_launch_counts", "ulsnn_mlp_enable_timing", "ulsnn_mlp_phase_times",
    "ulsnn_sgemm_noalloc", "ulsnn_sgemm_noalloc_max_scratch_bytes", "ulsnn_mlp_forward_sse", "ulsnn_mlp_gradient_sse",
    "ulsnn_vec_dot_workspace_bytes", "ulsnn_vec_dot", "ulsnn_vec_axpby",
    "ulsnn_sgemm_workspace_bytes_for", "ulsnn_debug_wait_timeout", "ulsnn_debug_device_cache_slot",
    "ulsnn_mlp_set_gradient_events",
]


class UlsnnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, status_string(status), status))


class _Desc(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("sizes", ctypes.POINTER(ctypes.c_int32)),
                ("math", ctypes.c_int), ("max_patterns", ctypes.c_int64)]


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libulsnn.so is not built: run `python -m paper_1911_05181_b200.buildlib`")
        l = ctypes.CDLL(LIB_PATH)
        vp, i64, f32, i32, u64, sz = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_float, ctypes.c_int32,
                                      ctypes.c_uint64, ctypes.c_size_t)
        l.ulsnn_status_string.restype = ctypes.c_char_p
        l.ulsnn_status_string.argtypes = [ctypes.c_int]
        l.ulsnn_version.restype = ctypes.c_int
        l.ulsnn_sgemm.argtypes = [ctypes.c_char, ctypes.c_char, i64, i64, i64, f32, vp, i64, vp, i64, f32, vp, i64, vp]
        l.ulsnn_sgemm_ex.argtypes = l.ulsnn_sgemm.argtypes[:-1] + [ctypes.c_int, vp, sz, vp]
        l.ulsnn_sgemm_noalloc.argtypes = l.ulsnn_sgemm.argtypes[:-1] + [ctypes.c_int, vp]
        l.ulsnn_sgemm_noalloc_max_scratch_bytes.restype = sz
        l.ulsnn_sgemm_noalloc_max_scratch_bytes.argtypes = []
        l.ulsnn_sgemm_workspace_bytes.argtypes = [ctypes.c_char, ctypes.c_char, i64, i64, i64, ctypes.c_int,
                                                  ctypes.POINTER(sz)]
        l.ulsnn_sgemm_workspace_bytes_for.argtypes = [ctypes.c_char, ctypes.c_char, i64, i64, i64, vp, i64, vp, i64,
                                                      ctypes.c_int, ctypes.POINTER(sz)]
        l.ulsnn_debug_wait_timeout.argtypes = [u64, vp]
        l.ulsnn_debug_device_cache_slot.argtypes = [ctypes.c_int]
        l.ulsnn_debug_device_cache_slot.restype = ctypes.c_int
        l.ulsnn_mlp_workspace_bytes.argtypes = [ctypes.POINTER(_Desc), ctypes.POINTER(sz)]
        l.ulsnn_mlp_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(_Desc), vp, sz]
        l.ulsnn_mlp_destroy.argtypes = [vp]
        l.ulsnn_mlp_destroy.restype = None
        pp = ctypes.POINTER(vp)
        l.ulsnn_mlp_forward_loss.argtypes = [vp, pp, pp, vp, i64, vp, i64, vp, vp]
        l.ulsnn_mlp_gradient.argtypes = [vp, pp, pp, vp, i64, vp, i64, ctypes.c_int, pp, pp, vp, vp]
        l.ulsnn_mlp_forward_sse.argtypes = [vp, pp, pp, vp, i64, vp, i64, i64, vp, vp]
        l.ulsnn_mlp_gradient_sse.argtypes = [vp, pp, pp, vp, i64, vp, i64, i64, ctypes.c_int, pp, pp, vp, vp]
        l.ulsnn_vec_dot_workspace_bytes.argtypes = [i64, ctypes.POINTER(sz)]
        l.ulsnn_vec_dot.argtypes = [i64, vp, vp, vp, vp, sz, vp]
        l.ulsnn_vec_axpby.argtypes = [i64, f32, vp, f32, vp, vp, vp]
        l.ulsnn_sgd_step.argtypes = [vp, pp, pp, pp, pp, f32, vp]
        l.ulsnn_last_device_status.argtypes = [vp, vp]
        l.ulsnn_mlp_set_gradient_events.argtypes = [vp, pp]
        l.ulsnn_fill_uniform.argtypes = [vp, i64, u64, u64, u64, ctypes.c_int, vp]
        l.ulsnn_fill_labels.argtypes = [vp, i64, u64, u64, u64, i32, vp]
        l.ulsnn_launch_counts.argtypes = [ctypes.POINTER(i64)]
        l.ulsnn_launch_counts.restype = None
        l.ulsnn_mlp_enable_timing.argtypes = [vp, ctypes.c_int]
        l.ulsnn_mlp_phase_times.argtypes = [vp, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(f32), ctypes.POINTER(i64)]
        _lib = l
    return _lib


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(s):
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _ptr_array(seq):
    arr = (ctypes.c_void_p * len(seq))(*[_ptr(t) for t in seq])
    return arr


def _check(status: int, where: str):
    if status != OK:
        raise UlsnnError(status, where)


def status_string(status: int) -> str:
    return lib().ulsnn_status_string(status).decode()


def version() -> int:
    return lib().ulsnn_version()


def launch_counts():
    out = (ctypes.c_int64 * 4)()
    lib().ulsnn_launch_counts(out)
    return {"simt_gemm": out[0], "tc_gemm": out[1], "small": out[2], "fill": out[3]}


def sgemm(transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream=None, check=True):
    st = lib().ulsnn_sgemm(transA.encode(), transB.encode(), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb,
                           beta, _ptr(C), ldc, _stream(stream))
    if check:
        _check(st, "ulsnn_sgemm")
    return st


def sgemm_workspace_bytes(transA, transB, M, N, K, math=MATH_3XTF32) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().ulsnn_sgemm_workspace_bytes(transA.encode(), transB.encode(), M, N, K, math, ctypes.byref(out)),
           "ulsnn_sgemm_workspace_bytes")
    return out.value


def sgemm_workspace_bytes_for(transA, transB, M, N, K, A, lda, B, ldb, math=MATH_3XTF32) -> int:
    """Workspace for these operands (A, B: tensors or addresses, inspected for alignment only)."""
    out = ctypes.c_size_t(0)
    _check(lib().ulsnn_sgemm_workspace_bytes_for(transA.encode(), transB.encode(), M, N, K, _ptr(A), lda, _ptr(B), ldb,
                                                 math, ctypes.byref(out)), "ulsnn_sgemm_workspace_bytes_for")
    return out.value


def debug_wait_timeout(limit_cycles: int, stream=None) -> int:
    return lib().ulsnn_debug_wait_timeout(int(limit_cycles), _stream(stream))


def device_cache_slot(device: int) -> int:
    return int(lib().ulsnn_debug_device_cache_slot(int(device)))


def last_device_status(stream=None) -> int:
    """Status word of the current device (synchronises the stream, clears the word)."""
    return lib().ulsnn_last_device_status(None, _stream(stream))


def sgemm_ex(transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, math=MATH_3XTF32,
             workspace=None, workspace_bytes=0, stream=None, check=True):
    st = lib().ulsnn_sgemm_ex(transA.encode(), transB.encode(), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb,
                              beta, _ptr(C), ldc, math, _ptr(workspace), workspace_bytes, _stream(stream))
    if check:
        _check(st, "ulsnn_sgemm_ex")
    return st


def sgemm_noalloc_max_scratch_bytes() -> int:
    return int(lib().ulsnn_sgemm_noalloc_max_scratch_bytes())


def sgemm_noalloc(transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, math=MATH_3XTF32, stream=None,
                  check=True):
    """ulsnn_sgemm_noalloc: the product of sgemm_ex with the split-K scratch taken from the library's fixed array."""
    st = lib().ulsnn_sgemm_noalloc(transA.encode(), transB.encode(), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb,
                                   beta, _ptr(C), ldc, math, _stream(stream))
    if check:
        _check(st, "ulsnn_sgemm_noalloc")
    return st


def vec_dot_workspace_bytes(n) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().ulsnn_vec_dot_workspace_bytes(n, ctypes.byref(out)), "ulsnn_vec_dot_workspace_bytes")
    return out.value


def vec_dot(n, x, y, out, workspace, workspace_bytes, stream=None):
    _check(lib().ulsnn_vec_dot(n, _ptr(x), _ptr(y), _ptr(out), _ptr(workspace), workspace_bytes, _stream(stream)), "ulsnn_vec_dot")


def vec_axpby(n, a, x, b, y, out, stream=None):
    _check(lib().ulsnn_vec_axpby(n, a, _ptr(x), b, _ptr(y), _ptr(out), _stream(stream)), "ulsnn_vec_axpby")


def fill_uniform(dst, n, seed, tensor_id, offset=0, mode=0, stream=None):
    _check(lib().ulsnn_fill_uniform(_ptr(dst), n, seed, tensor_id, offset, mode, _stream(stream)), "ulsnn_fill_uniform")


def fill_labels(dst, n, seed, tensor_id, offset, n_classes, stream=None):
    _check(lib().ulsnn_fill_labels(_ptr(dst), n, seed, tensor_id, offset, n_classes, _stream(stream)), "ulsnn_fill_labels")


def mlp_workspace_bytes(sizes, math, max_patterns) -> int:
    arr = (ctypes.c_int32 * len(sizes))(*[int(s) for s in sizes])
    d = _Desc(len(sizes) - 1, arr, math, max_patterns)
    out = ctypes.c_size_t(0)
    _check(lib().ulsnn_mlp_workspace_bytes(ctypes.byref(d), ctypes.byref(out)), "ulsnn_mlp_workspace_bytes")
    return out.value


class Mlp:
    """Handle of ulsnn_mlp_create plus the workspace it borrows (a torch uint8 tensor on the current device)."""

    def __init__(self, sizes, math=MATH_3XTF32, max_patterns=65536, workspace=None):
        self.sizes = [int(s) for s in sizes]
        self.math = math
        self.max_patterns = int(max_patterns)
        self.L = len(self.sizes) - 1
        self.workspace_bytes = mlp_workspace_bytes(self.sizes, math, self.max_patterns)
        if workspace is None:
            import torch
            workspace = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device="cuda")
        self._ws = workspace
        base = _ptr(workspace)
        self._ws_ptr = (base + 255) // 256 * 256
        arr = (ctypes.c_int32 * len(self.sizes))(*self.sizes)
        d = _Desc(self.L, arr, math, self.max_patterns)
        h = ctypes.c_void_p(None)
        _check(lib().ulsnn_mlp_create(ctypes.byref(h), ctypes.byref(d), self._ws_ptr, self.workspace_bytes),
               "ulsnn_mlp_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().ulsnn_mlp_destroy(self._h)
            self._h = None

    __del__ = close

    def forward_loss(self, W, b, X, ldx, labels, n_patterns, loss_out, stream=None, check=True):
        st = lib().ulsnn_mlp_forward_loss(self._h, _ptr_array(W), _ptr_array(b), _ptr(X), ldx, _ptr(labels),
                                          n_patterns, _ptr(loss_out), _stream(stream))
        if check:
            _check(st, "ulsnn_mlp_forward_loss")
        return st

    def gradient(self, W, b, X, ldx, labels, n_patterns, accumulate, dW, db, loss_out, stream=None, check=True):
        st = lib().ulsnn_mlp_gradient(self._h, _ptr_array(W), _ptr_array(b), _ptr(X), ldx, _ptr(labels), n_patterns,
                                      1 if accumulate else 0, _ptr_array(dW), _ptr_array(db), _ptr(loss_out),
                                      _stream(stream))
        if check:
            _check(st, "ulsnn_mlp_gradient")
        return st

    def forward_sse(self, W, b, X, ldx, T, ldt, n_patterns, loss_out, stream=None, check=True):
        st = lib().ulsnn_mlp_forward_sse(self._h, _ptr_array(W), _ptr_array(b), _ptr(X), ldx, _ptr(T), ldt,
                                         n_patterns, _ptr(loss_out), _stream(stream))
        if check:
            _check(st, "ulsnn_mlp_forward_sse")
        return st

    def gradient_sse(self, W, b, X, ldx, T, ldt, n_patterns, accumulate, dW, db, loss_out, stream=None, check=True):
        st = lib().ulsnn_mlp_gradient_sse(self._h, _ptr_array(W), _ptr_array(b), _ptr(X), ldx, _ptr(T), ldt, n_patterns,
                                          1 if accumulate else 0, _ptr_array(dW), _ptr_array(db), _ptr(loss_out),
                                          _stream(stream))
        if check:
            _check(st, "ulsnn_mlp_gradient_sse")
        return st

    def sgd_step(self, W, b, dW, db, lr, stream=None, check=True):
        st = lib().ulsnn_sgd_step(self._h, _ptr_array(W), _ptr_array(b), _ptr_array(dW), _ptr_array(db), lr,
                                  _stream(stream))
        if check:
            _check(st, "ulsnn_sgd_step")
        return st

    def enable_timing(self, on=True):
        _check(lib().ulsnn_mlp_enable_timing(self._h, 1 if on else 0), "ulsnn_mlp_enable_timing")

    def phase_times(self):
        """[(ms, M, N, K)] of the products of the most recent forward_loss / gradient call (timing must be on)."""
        cap = 64
        n = ctypes.c_int(cap); ms = (ctypes.c_float * cap)(); mnk = (ctypes.c_int64 * (3 * cap))()
        _check(lib().ulsnn_mlp_phase_times(self._h, ctypes.byref(n), ms, mnk), "ulsnn_mlp_phase_times")
        return [(ms[i], mnk[3 * i], mnk[3 * i + 1], mnk[3 * i + 2]) for i in range(n.value)]

    def set_gradient_events(self, events):
        """events: one torch.cuda.Event (already recorded once, so that it exists) or None per weight matrix, or None."""
        if events is None:
            _check(lib().ulsnn_mlp_set_gradient_events(self._h, None), "ulsnn_mlp_set_gradient_events")
            return
        arr = (ctypes.c_void_p * len(events))(*[(e.cuda_event if e is not None else None) for e in events])
        _check(lib().ulsnn_mlp_set_gradient_events(self._h, arr), "ulsnn_mlp_set_gradient_events")

    def last_device_status(self, stream=None) -> int:
        return lib().ulsnn_last_device_status(self._h, _stream(stream))
