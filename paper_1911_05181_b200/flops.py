"""Flop accounting of the paper (2 flops per multiply-add; elementwise,
epilogue and reduction work is not counted, Section 6.3).

    SGEMM            2*M*N*K                                  (Section 3.1)
    error (forward)  2*n_p*(n_i + n_o)*n_h                    (Section 6.2)
    gradient         n_p*(4*n_i*n_h + 6*n_h*n_o)              (Section 6.2)

For more than one hidden layer the same reasoning gives 2 flops per weight for
the forward product, 2 for the weight-gradient product and, for every layer but
the first, 2 more for propagating the deltas down (no delta is formed for the
inputs, which is why the first layer counts 4 and not 6).
"""
from __future__ import annotations


def sgemm_flops(M: int, N: int, K: int) -> int:
    return 2 * M * N * K


def n_params(sizes, with_bias: bool = False) -> int:
    n = sum(int(sizes[l]) * int(sizes[l + 1]) for l in range(len(sizes) - 1))
    if with_bias:
        n += sum(int(s) for s in sizes[1:])
    return n


def forward_flops_per_pattern(sizes) -> int:
    return 2 * n_params(sizes)


def gradient_flops_per_pattern(sizes) -> int:
    first = int(sizes[0]) * int(sizes[1])
    rest = n_params(sizes) - first
    return 4 * first + 6 * rest


def forward_flops(sizes, n_patterns: int) -> int:
    return n_patterns * forward_flops_per_pattern(sizes)


def gradient_flops(sizes, n_patterns: int) -> int:
    return n_patterns * gradient_flops_per_pattern(sizes)
