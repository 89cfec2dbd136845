"""CPU oracle for the fused mixed-precision linear layer  Y = A . dequant(Wq).

TEST INFRASTRUCTURE, NOT PRODUCT.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline / reference legs may import this package.  It shares no
code with the CUDA library and never imports it; the CUDA path never imports
this.  Everything here is the plain definition written out in fp64 with numpy
(one library matmul is the contraction step); nothing is blocked, fused or
reordered.

What the method computes (it reaches this result exactly, up to rounding order,
so the oracle *is* the definition):

    q[k][n]   4-bit code of column n in row k of the AWQ-packed words        (W4)
              or the int8 weight itself                                       (W8)
    z[g][n]   4-bit zero point of group g = k // group_size                   (W4 only)
    s[g][n]   fp16 scale of group g
    w[k][n] = s[g][n] * (q[k][n] - z[g][n])        asymmetric dequantization, Eq. (2)
    w[k][n] = s[g][n] *  q[k][n]                    symmetric dequantization,  Eq. (1)
    y[m][n] = sum_k a[m][k] * w[k][n]               C = A x B of Section 2.1
    B[m][n] = sum_k |a[m][k] * w[k][n]|             magnitude sum used by the tolerance

Groups run along K (every `group_size` weights of one output column share one
scale and zero point, Section 4.2).  The zero point is used as stored (no +1
offset).  The 4-bit packing is the AWQ checkpoint encoding: bits [4i, 4i+4) of
word j hold column 8j + (0,2,4,6,1,3,5,7)[i].

Parity pins (tests/test_oracle_*.py): a hand-worked packed word, exact rational
arithmetic on tiny problems, integer-matmul special cases, one-hot activations,
linearity, q == z, and the magnitude bound.  No function here is unpinned.
"""
from __future__ import annotations

import numpy as np

# Column held by nibble position i of a word (Section 2.2 names the AWQ format;
# the order itself is the AWQ checkpoint convention).
_POSITION_TO_COLUMN = (0, 2, 4, 6, 1, 3, 5, 7)


def unpack_awq(words: np.ndarray) -> np.ndarray:
    """uint32 [R, C/8] -> uint8 [R, C]: the 4-bit codes in logical column order."""
    words = np.asarray(words, dtype=np.uint32)
    rows, nwords = words.shape
    out = np.empty((rows, nwords, 8), dtype=np.uint8)
    for position, column in enumerate(_POSITION_TO_COLUMN):
        out[:, :, column] = (words >> np.uint32(4 * position)) & np.uint32(0xF)
    return out.reshape(rows, nwords * 8)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exactly (bf16 is the top half of fp32)."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def _expand_groups(per_group: np.ndarray, group_size: int) -> np.ndarray:
    """[K/g, N] -> [K, N]: row k takes the value of group k // group_size."""
    return np.repeat(per_group, group_size, axis=0)


def dequant_w4(qweight, scales_f16, qzeros, group_size: int) -> np.ndarray:
    """Eq. (2): w = s_g (q - z_g), in fp64.  Returns float64 [K, N]."""
    q = unpack_awq(qweight).astype(np.float64)
    z = unpack_awq(qzeros).astype(np.float64)
    s = np.asarray(scales_f16, dtype=np.float16).astype(np.float64)
    K = q.shape[0]
    assert K % group_size == 0 and z.shape == (K // group_size, q.shape[1]) and s.shape == z.shape
    return _expand_groups(s, group_size) * (q - _expand_groups(z, group_size))


def dequant_w8(w_i8, scales_f16, group_size: int) -> np.ndarray:
    """Eq. (1): w = s_g q, in fp64.  Returns float64 [K, N]."""
    q = np.asarray(w_i8, dtype=np.int8).astype(np.float64)
    s = np.asarray(scales_f16, dtype=np.float16).astype(np.float64)
    K = q.shape[0]
    assert K % group_size == 0 and s.shape == (K // group_size, q.shape[1])
    return _expand_groups(s, group_size) * q


def linear(a_bf16_bits, w_f64):
    """y = a @ w and B = |a| @ |w| in fp64 (Section 2.1: C = A x B)."""
    a = bf16_bits_to_f64(a_bf16_bits)
    y = a @ w_f64
    bound = np.abs(a) @ np.abs(w_f64)
    return y, bound


def linear_w4a16(a_bf16_bits, qweight, scales_f16, qzeros, group_size: int = 128,
                 columns=None):
    """W4A16 layer.  `columns` (optional index array) restricts the output columns."""
    w = dequant_w4(qweight, scales_f16, qzeros, group_size) if columns is None else \
        _dequant_w4_columns(qweight, scales_f16, qzeros, group_size, np.asarray(columns))
    return linear(a_bf16_bits, w)


def linear_w8a16(a_bf16_bits, w_i8, scales_f16, group_size: int = 128, columns=None):
    """W8A16 layer.  `columns` (optional index array) restricts the output columns."""
    if columns is not None:
        columns = np.asarray(columns)
        w_i8 = np.asarray(w_i8)[:, columns]
        scales_f16 = np.asarray(scales_f16)[:, columns]
    return linear(a_bf16_bits, dequant_w8(w_i8, scales_f16, group_size))


def _dequant_w4_columns(qweight, scales_f16, qzeros, group_size, columns):
    """Eq. (2) for a subset of columns: decode only the words those columns live in."""
    words = np.unique(columns // 8)
    q = unpack_awq(np.asarray(qweight)[:, words]).astype(np.float64)
    z = unpack_awq(np.asarray(qzeros)[:, words]).astype(np.float64)
    local = np.searchsorted(words, columns // 8) * 8 + columns % 8
    s = np.asarray(scales_f16, dtype=np.float16)[:, columns].astype(np.float64)
    return _expand_groups(s, group_size) * (q[:, local] - _expand_groups(z[:, local], group_size))


def solve(problem, columns=None):
    """(y_ref, B) for a `workloads.Problem`-shaped object (duck-typed: attributes only)."""
    if problem.bits == 4:
        return linear_w4a16(problem.a_bf16, problem.qweight, problem.scales_f16,
                            problem.qzeros, problem.group_size, columns)
    return linear_w8a16(problem.a_bf16, problem.w_i8, problem.scales_f16,
                        problem.group_size, columns)
