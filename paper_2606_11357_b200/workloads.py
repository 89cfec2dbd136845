"""Seeded synthetic inputs for the fused W4A16 / W8A16 linear layer.

This module only *draws* and *encodes* inputs.  It holds none of the method's
arithmetic (no unpacking, no dequantization, no contraction): the CPU oracle and
the CUDA library each decode these arrays with code of their own.  Both sides
are handed the very same numpy arrays, so no random-number stream has to be
reproduced across languages.

Formats produced (the quantized-weight format of Section 2.2 of the paper, in
the AWQ checkpoint encoding):

* activations : bf16 bit patterns, ``uint16 [M, K]``, row-major.
* W4A16       : ``qweight uint32 [K, N/8]`` (eight 4-bit codes per word along
  N; bits ``[4i, 4i+4)`` of word ``j`` hold column ``8j + AWQ_ORDER[i]``),
  ``scales fp16 [K/g, N]``, ``qzeros uint32 [K/g, N/8]`` (same nibble order).
* W8A16       : ``w int8 [K, N]``, ``scales fp16 [K/g, N]``, no zero point.

Draw order per problem (fixed, so a seed names one input set): activations,
weight codes, zero points, scales.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

GROUP_SIZE = 128
# Position i of a packed word holds logical column AWQ_ORDER[i] of its 8-column run.
AWQ_ORDER = (0, 2, 4, 6, 1, 3, 5, 7)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + (((u >> 16) & 1) + 0x7FFF)
    return (u >> 16).astype(np.uint16)


def awq_pack_words(codes: np.ndarray) -> np.ndarray:
    """Encode 4-bit codes ``uint8 [R, C]`` (C % 8 == 0) as AWQ words ``uint32 [R, C/8]``."""
    codes = np.asarray(codes)
    assert codes.ndim == 2 and codes.shape[1] % 8 == 0
    assert codes.max(initial=0) <= 15
    c8 = codes.reshape(codes.shape[0], -1, 8).astype(np.uint32)
    words = np.zeros(c8.shape[:2], dtype=np.uint32)
    for pos, col in enumerate(AWQ_ORDER):
        words |= c8[:, :, col] << np.uint32(4 * pos)
    return words


@dataclass
class Problem:
    """One linear-layer problem: inputs in the formats the library accepts."""
    name: str
    bits: int                 # 4 or 8
    M: int
    K: int
    N: int
    group_size: int
    seed: int
    a_bf16: np.ndarray        # uint16 [M, K]
    scales_f16: np.ndarray    # float16 [K/g, N]
    qweight: np.ndarray | None = None   # uint32 [K, N/8]   (bits == 4)
    qzeros: np.ndarray | None = None    # uint32 [K/g, N/8] (bits == 4)
    w_i8: np.ndarray | None = None      # int8 [K, N]       (bits == 8)
    # Raw draws kept for tests that want to look at them (never fed to a decoder).
    raw: dict = field(default_factory=dict)


def _activations(rng, M, K, outlier_frac=0.0, outlier_gain=20.0):
    a = rng.standard_normal((M, K), dtype=np.float32)
    if outlier_frac > 0.0:
        idx = rng.choice(K, size=int(round(outlier_frac * K)), replace=False)
        a[:, idx] *= np.float32(outlier_gain)       # scaled before rounding to bf16
    return f32_to_bf16_bits(a)


def make_w4(M, K, N, seed, *, name="w4", group_size=GROUP_SIZE, outlier_frac=0.0,
            scale_range=(0.001, 0.02), keep_raw=False) -> Problem:
    """AWQ-style W4A16 problem: codes U{0..15}, zero points U{0..15}, fp16 scales U[lo, hi]."""
    assert K % group_size == 0 and N % 8 == 0
    rng = np.random.default_rng(seed)
    a = _activations(rng, M, K, outlier_frac)
    q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    z = rng.integers(0, 16, size=(K // group_size, N), dtype=np.uint8)
    s = rng.uniform(scale_range[0], scale_range[1], size=(K // group_size, N)).astype(np.float32)
    p = Problem(name, 4, M, K, N, group_size, seed, a, s.astype(np.float16),
                qweight=awq_pack_words(q), qzeros=awq_pack_words(z))
    if keep_raw:
        p.raw = {"q": q, "z": z}
    return p


def make_w8(M, K, N, seed, *, name="w8", group_size=GROUP_SIZE,
            scale_range=(0.0005, 0.005), keep_raw=False) -> Problem:
    """Symmetric W8A16 problem: int8 codes U{-127..127}, fp16 scales U[lo, hi], no zero point."""
    assert K % group_size == 0
    rng = np.random.default_rng(seed)
    a = _activations(rng, M, K)
    w = rng.integers(-127, 128, size=(K, N), dtype=np.int8)
    s = rng.uniform(scale_range[0], scale_range[1], size=(K // group_size, N)).astype(np.float32)
    p = Problem(name, 8, M, K, N, group_size, seed, a, s.astype(np.float16), w_i8=w)
    if keep_raw:
        p.raw = {"q": w}
    return p


# ---------------------------------------------------------------------------
# The five benchmark configurations (shapes, distributions and structure).
# ---------------------------------------------------------------------------
LLAMA3_8B_SHAPES = ((4096, 4096), (4096, 1024), (4096, 14336), (14336, 4096))  # (K, N)


def config0() -> Problem:
    """W4A16 GEMV 1x4096x4096, seed 0."""
    return make_w4(1, 4096, 4096, 0, name="cfg0_gemv_w4_1x4096x4096")


def config1(M: int, K: int, N: int) -> Problem:
    """Decode GEMV sweep over Llama-3-8B-shaped layers, M in {1, 4, 16}."""
    seed = 1000 + 100 * LLAMA3_8B_SHAPES.index((K, N)) + M
    return make_w4(M, K, N, seed, name=f"cfg1_gemv_w4_{M}x{K}x{N}")


def config2(M: int = 2048, K: int = 4096, N: int = 14336) -> Problem:
    """Prefill GEMM with 1 % outlier K-channels (x20)."""
    return make_w4(M, K, N, 2, name=f"cfg2_gemm_w4_{M}x{K}x{N}", outlier_frac=0.01)


def config3_gemm(M: int = 1024, K: int = 4096, N: int = 4096) -> Problem:
    return make_w8(M, K, N, 3, name=f"cfg3_gemm_w8_{M}x{K}x{N}")


def config3_gemv(M: int = 1, K: int = 4096, N: int = 14336) -> Problem:
    return make_w8(M, K, N, 31, name=f"cfg3_gemv_w8_{M}x{K}x{N}")


def config4_gemm(M: int = 512, K: int = 32768, N: int = 4096) -> Problem:
    return make_w4(M, K, N, 4, name=f"cfg4_gemm_w4_{M}x{K}x{N}")


def config4_gemv(M: int = 1, K: int = 4096, N: int = 32768) -> Problem:
    return make_w4(M, K, N, 41, name=f"cfg4_gemv_w4_{M}x{K}x{N}")
