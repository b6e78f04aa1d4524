"""Shared plumbing of the GPU tests: numpy <-> device tensors and calls through the C-ABI binding."""
import json
import os

import numpy as np
import torch

from paper_1911_05181_b200 import binding as ul

# relative L2, per tensor; the 16-bit mode keeps 8 mantissa bits against TF32's 10: four times its tolerance
TOL = {ul.MATH_3XTF32: 1e-5, ul.MATH_FP32_SIMT: 1e-5, ul.MATH_TF32: 5e-3, ul.MATH_BF16: 2e-2}


with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "cond_ref.json")) as _f:
    COND_REF = json.load(_f)


def tolerance_at(math, cond, head="softmax"):
    """Tolerance for a gradient tensor whose condition number (oracle.gradient_condition) is `cond`.  The attainable
    relative error of a finite-precision evaluation is proportional to the condition number; the stated tolerances
    are those of the benchmark network, whose worst tensor has COND_REF: a tensor that is worse conditioned than that
    is held to the same multiple of its own condition number, a better conditioned one to the stated tolerance."""
    ref = max(COND_REF[head]["dW"] + COND_REF[head]["db"])
    return TOL[math] * max(1.0, cond / ref)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_sgemm(transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, math, use_plain=False):
    """A, B, C: numpy arrays as stored (rows x ld).  Returns the full stored C after the call."""
    dA, dB, dC = dev(A), dev(B), dev(C)
    if use_plain:
        ul.sgemm(transA, transB, M, N, K, alpha, dA, lda, dB, ldb, beta, dC, ldc)
    else:
        # the workspace these operands need, re-buffered copies of operands TMA cannot address included
        nbytes = ul.sgemm_workspace_bytes_for(transA, transB, M, N, K, dA, lda, dB, ldb, math)
        ws = torch.empty(max(nbytes, 1) + 256, dtype=torch.uint8, device="cuda")
        wp = (ws.data_ptr() + 255) // 256 * 256
        ul.sgemm_ex(transA, transB, M, N, K, alpha, dA, lda, dB, ldb, beta, dC, ldc, math, wp if nbytes else None, nbytes)
    torch.cuda.synchronize()
    return dC.cpu().numpy()


class GpuNet:
    def __init__(self, sizes, math, max_patterns):
        self.sizes = list(sizes)
        self.net = ul.Mlp(sizes, math, max_patterns)
        L = len(sizes) - 1
        self.dW = [torch.full((sizes[l + 1], sizes[l]), float("nan"), device="cuda") for l in range(L)]
        self.db = [torch.full((sizes[l + 1],), float("nan"), device="cuda") for l in range(L)]
        self.loss = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")

    def set_params(self, Ws, bs):
        self.W = [dev(w) for w in Ws]
        self.b = [dev(b) for b in bs]

    def gradient(self, X, y, accumulate=False, ldx=None):
        dX = X if isinstance(X, torch.Tensor) else dev(X)
        dy = y if isinstance(y, torch.Tensor) else dev(y)
        n = dX.shape[0]
        self.net.gradient(self.W, self.b, dX, ldx or (dX.shape[1] if n else self.sizes[0]), dy, n, accumulate,
                          self.dW, self.db, self.loss)
        torch.cuda.synchronize()
        return (float(self.loss.item()), [g.cpu().numpy() for g in self.dW], [g.cpu().numpy() for g in self.db])

    def forward_loss(self, X, y):
        dX, dy = dev(X), dev(y)
        self.net.forward_loss(self.W, self.b, dX, dX.shape[1], dy, dX.shape[0], self.loss)
        torch.cuda.synchronize()
        return float(self.loss.item())
