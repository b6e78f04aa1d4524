"""Seeded synthetic inputs shared by the tests, the bench and the CPU checker.

This module holds no arithmetic of the method itself: it only turns
(seed, tensor id, flat index) into reproducible numbers, so that any slice of
any tensor can be produced independently, on the host (here, numpy) and on the
device (the library's fill kernels implement the same counter-based hash and
are tested bit-for-bit against this file).

Recipe (stands in for the paper's 20x20-pixel / 3203-class character data,
Section 6.1, which is not available):

    h            = mix64(seed, tensor_id, index)            (64-bit hash)
    uniform[0,1) = (h >> 40) * 2**-24                        (exact in fp32)
    uniform[-1,1)= 2*u - 1                                   (exact in fp32)
    label        = (h >> 11) mod n_classes
    normal(0,s)  = s * sqrt(-2 ln u1) * cos(2 pi u2), u1,u2 from two hashes,
                   evaluated in float64 on the host, rounded once to fp32
"""
from __future__ import annotations

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_C_TENSOR = np.uint64(0xD1B54A32D192ED03)
_MIX1 = np.uint64(0xBF58476D1CE4E5B9)
_MIX2 = np.uint64(0x94D049BB133111EB)

# Tensor ids used by every config (kept here so host and device agree).
TID_X = 1
TID_LABELS = 2
TID_TARGETS = 3
TID_W0 = 16        # W_l uses TID_W0 + 2*l, b_l uses TID_W0 + 2*l + 1
TID_GEMM_A = 100
TID_GEMM_B = 101
TID_GEMM_C = 102


def mix64(seed: int, tensor_id: int, index: np.ndarray) -> np.ndarray:
    """64-bit counter hash: a splitmix64-style finaliser of a linear key."""
    with np.errstate(over="ignore"):
        idx = np.asarray(index, dtype=np.uint64)
        key = (np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * _GOLD
               + np.uint64(tensor_id) * _C_TENSOR + idx + np.uint64(1))
        z = key
        z = (z ^ (z >> np.uint64(30))) * _MIX1
        z = (z ^ (z >> np.uint64(27))) * _MIX2
        z = z ^ (z >> np.uint64(31))
        # second round decorrelates neighbouring counters of neighbouring tensors
        z = z + _GOLD
        z = (z ^ (z >> np.uint64(30))) * _MIX1
        z = (z ^ (z >> np.uint64(27))) * _MIX2
        z = z ^ (z >> np.uint64(31))
    return z


def _counter(n: int, offset: int) -> np.ndarray:
    return np.arange(offset, offset + n, dtype=np.uint64)


def uniform01(seed: int, tensor_id: int, n: int, offset: int = 0) -> np.ndarray:
    """n fp32 values in [0,1), multiples of 2**-24."""
    h = mix64(seed, tensor_id, _counter(n, offset))
    return ((h >> np.uint64(40)).astype(np.float32) * np.float32(2.0 ** -24)).astype(np.float32)


def uniform_pm1(seed: int, tensor_id: int, n: int, offset: int = 0) -> np.ndarray:
    """n fp32 values in [-1,1), multiples of 2**-23."""
    u = uniform01(seed, tensor_id, n, offset)
    return (np.float32(2.0) * u - np.float32(1.0)).astype(np.float32)


def labels(seed: int, tensor_id: int, n: int, n_classes: int, offset: int = 0) -> np.ndarray:
    """n int32 class labels in [0, n_classes)."""
    h = mix64(seed, tensor_id, _counter(n, offset))
    return ((h >> np.uint64(11)) % np.uint64(n_classes)).astype(np.int32)


def normal(seed: int, tensor_id: int, n: int, std: float) -> np.ndarray:
    """n fp32 draws from N(0, std**2) by Box-Muller in float64 (host only)."""
    c = _counter(n, 0)
    h1 = mix64(seed, tensor_id, c * np.uint64(2))
    h2 = mix64(seed, tensor_id, c * np.uint64(2) + np.uint64(1))
    u1 = ((h1 >> np.uint64(11)).astype(np.float64) + 1.0) * 2.0 ** -53   # (0,1]
    u2 = (h2 >> np.uint64(11)).astype(np.float64) * 2.0 ** -53           # [0,1)
    g = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (std * g).astype(np.float32)


def mlp_params(seed: int, sizes):
    """Weights W_l ~ N(0, 1/fan_in) as [n_out, n_in] fp32, biases zero."""
    Ws, bs = [], []
    for l in range(len(sizes) - 1):
        fan_in, fan_out = int(sizes[l]), int(sizes[l + 1])
        w = normal(seed, TID_W0 + 2 * l, fan_in * fan_out, 1.0 / np.sqrt(fan_in))
        Ws.append(w.reshape(fan_out, fan_in))
        bs.append(np.zeros(fan_out, dtype=np.float32))
    return Ws, bs


def mlp_batch(seed: int, sizes, n_patterns: int, offset: int = 0):
    """Inputs X [n_patterns, n_0] uniform[0,1) and int32 labels; `offset` is in patterns."""
    n0, nL = int(sizes[0]), int(sizes[-1])
    X = uniform01(seed, TID_X, n_patterns * n0, offset * n0).reshape(n_patterns, n0)
    y = labels(seed, TID_LABELS, n_patterns, nL, offset)
    return X, y


def mlp_targets(seed: int, sizes, n_patterns: int, offset: int = 0, coded: bool = False):
    """Dense target matrix T [n_patterns, n_L] for the squared-error head: uniform[-1,1), or, with coded=True,
    the +1 / -1 code of the pattern's label (one output unit per class)."""
    nL = int(sizes[-1])
    if coded:
        y = labels(seed, TID_LABELS, n_patterns, nL, offset)
        T = np.full((n_patterns, nL), -1.0, dtype=np.float32)
        T[np.arange(n_patterns), y] = 1.0
        return T
    return uniform_pm1(seed, TID_TARGETS, n_patterns * nL, offset * nL).reshape(n_patterns, nL)


def gemm_operands(seed: int, rows_a: int, cols_a: int, rows_b: int, cols_b: int,
                  rows_c: int, cols_c: int):
    """Stored operands (as laid out in memory, before op()) uniform[-1,1)."""
    A = uniform_pm1(seed, TID_GEMM_A, rows_a * cols_a).reshape(rows_a, cols_a)
    B = uniform_pm1(seed, TID_GEMM_B, rows_b * cols_b).reshape(rows_b, cols_b)
    C = uniform_pm1(seed, TID_GEMM_C, rows_c * cols_c).reshape(rows_c, cols_c)
    return A, B, C
