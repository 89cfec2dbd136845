"""Pins for the oracle's arithmetic: exact rationals, integer special cases, invariants."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import tilefuse_oracle as orc
from paper_2606_11357_b200 import workloads as wl
from helpers import bf16_bits_to_f64, loop_pack_awq, read_golden_dequant

ORDER = [0, 2, 4, 6, 1, 3, 5, 7]


def _nibble(words, r, c):
    """Scalar decode of logical column c of row r, from the format rule."""
    return (int(words[r, c // 8]) >> (4 * ORDER.index(c % 8))) & 0xF


def brute_force(p):
    """Exact rational evaluation of the definition with scalar loops (tiny shapes only)."""
    a = bf16_bits_to_f64(p.a_bf16)
    g = p.group_size
    y = [[Fraction(0)] * p.N for _ in range(p.M)]
    b = [[Fraction(0)] * p.N for _ in range(p.M)]
    for n in range(p.N):
        for k in range(p.K):
            s = Fraction(float(p.scales_f16[k // g, n]))
            if p.bits == 4:
                w = s * (_nibble(p.qweight, k, n) - _nibble(p.qzeros, k // g, n))
            else:
                w = s * int(p.w_i8[k, n])
            for m in range(p.M):
                t = Fraction(float(a[m, k])) * w
                y[m][n] += t
                b[m][n] += abs(t)
    return y, b


@pytest.mark.parametrize("maker,M,K,N", [(wl.make_w4, 1, 128, 8), (wl.make_w4, 3, 256, 24),
                                         (wl.make_w8, 2, 256, 5), (wl.make_w8, 1, 128, 16)])
def test_against_exact_rationals(maker, M, K, N):
    p = maker(M, K, N, seed=5)
    y, b = orc.solve(p)
    ye, be = brute_force(p)
    for m in range(M):
        for n in range(N):
            assert abs(Fraction(float(y[m, n])) - ye[m][n]) <= Fraction(1, 10**12) * (be[m][n] + 1)
            assert abs(Fraction(float(b[m, n])) - be[m][n]) <= Fraction(1, 10**12) * (be[m][n] + 1)


@pytest.mark.parametrize("kind,q,z,s,a,w,aw", read_golden_dequant())
def test_hand_worked_values(kind, q, z, s, a, w, aw):
    """One weight at row k0 of a [128 x 8] problem, one-hot activation: y = a*w exactly."""
    K, N, k0, n0 = 128, 8, 77, 5
    a_bits = np.zeros((1, K), dtype=np.uint16)
    a_bits[0, k0] = wl.f32_to_bf16_bits(np.array([a], dtype=np.float32))[0]
    scales = np.full((1, N), s, dtype=np.float16)
    assert float(scales[0, 0]) == s                       # the fixture's scale is exact in fp16
    if kind == "w4":
        codes = np.zeros((K, N), dtype=np.uint8)
        codes[k0, n0] = q
        zeros = np.zeros((1, N), dtype=np.uint8)
        zeros[0, n0] = z
        wmat = orc.dequant_w4(loop_pack_awq(codes), scales, loop_pack_awq(zeros), 128)
        y, b = orc.linear_w4a16(a_bits, loop_pack_awq(codes), scales, loop_pack_awq(zeros), 128)
    else:
        codes = np.zeros((K, N), dtype=np.int8)
        codes[k0, n0] = q
        wmat = orc.dequant_w8(codes, scales, 128)
        y, b = orc.linear_w8a16(a_bits, codes, scales, 128)
    assert wmat[k0, n0] == w
    assert y[0, n0] == aw and b[0, n0] == abs(aw)


def test_unit_scale_zero_offset_is_integer_matmul():
    """s = 1, z = 0, integer activations: the layer is an exact integer matrix product."""
    rng = np.random.default_rng(3)
    M, K, N = 5, 384, 40
    ai = rng.integers(-8, 9, size=(M, K))
    q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    a_bits = wl.f32_to_bf16_bits(ai.astype(np.float32))
    ones = np.ones((K // 128, N), dtype=np.float16)
    zero = np.zeros((K // 128, N), dtype=np.uint8)
    y, b = orc.linear_w4a16(a_bits, loop_pack_awq(q), ones, loop_pack_awq(zero), 128)
    assert np.array_equal(y, (ai.astype(np.int64) @ q.astype(np.int64)).astype(np.float64))
    assert np.array_equal(b, (np.abs(ai).astype(np.int64) @ q.astype(np.int64)).astype(np.float64))


def test_zero_point_eight_is_signed_int4():
    rng = np.random.default_rng(4)
    K, N = 256, 16
    q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    z = np.full((K // 128, N), 8, dtype=np.uint8)
    w = orc.dequant_w4(loop_pack_awq(q), np.ones((K // 128, N), np.float16), loop_pack_awq(z), 128)
    assert np.array_equal(w, q.astype(np.float64) - 8.0)


def test_w8_integer_matmul_and_full_range():
    rng = np.random.default_rng(5)
    M, K, N = 4, 256, 12
    ai = rng.integers(-4, 5, size=(M, K))
    w8 = rng.integers(-128, 128, size=(K, N), dtype=np.int8)
    w8[0, 0], w8[1, 0] = -128, 127
    y, _ = orc.linear_w8a16(wl.f32_to_bf16_bits(ai.astype(np.float32)), w8,
                            np.ones((K // 128, N), np.float16), 128)
    assert np.array_equal(y, (ai.astype(np.int64) @ w8.astype(np.int64)).astype(np.float64))


def test_groups_run_along_k_and_scale_is_per_column():
    """A scale or zero point placed in group 1 / column 3 affects rows 128..255 of column 3 only."""
    K, N = 384, 8
    q = np.full((K, N), 5, dtype=np.uint8)
    z = np.zeros((3, N), dtype=np.uint8)
    s = np.ones((3, N), dtype=np.float16)
    z[1, 3] = 2
    s[2, 6] = 0.5
    w = orc.dequant_w4(loop_pack_awq(q), s, loop_pack_awq(z), 128)
    want = np.full((K, N), 5.0)
    want[128:256, 3] = 3.0
    want[256:384, 6] = 2.5
    assert np.array_equal(w, want)


@pytest.mark.parametrize("maker", [wl.make_w4, wl.make_w8])
def test_one_hot_rows_pick_single_weights(maker):
    p = maker(1, 256, 24, seed=9)
    w = orc.dequant_w4(p.qweight, p.scales_f16, p.qzeros, 128) if p.bits == 4 else \
        orc.dequant_w8(p.w_i8, p.scales_f16, 128)
    for k in (0, 127, 128, 255):
        a = np.zeros((1, p.K), dtype=np.uint16)
        a[0, k] = 0x3F80                                   # bf16 1.0
        y, b = orc.linear(a, w)
        assert np.array_equal(y[0], w[k]) and np.array_equal(b[0], np.abs(w[k]))


def test_q_equals_z_gives_exact_zero():
    p = wl.make_w4(3, 512, 64, seed=12)
    zeros = orc.unpack_awq(p.qzeros)
    q = np.repeat(zeros, 128, axis=0)                       # q == z everywhere
    y, b = orc.linear_w4a16(p.a_bf16, loop_pack_awq(q.tolist()), p.scales_f16, p.qzeros, 128)
    assert not y.any() and not b.any()


@pytest.mark.parametrize("maker", [wl.make_w4, wl.make_w8])
def test_linear_in_the_activations(maker):
    p = maker(2, 384, 32, seed=21)
    w = orc.dequant_w4(p.qweight, p.scales_f16, p.qzeros, 128) if p.bits == 4 else \
        orc.dequant_w8(p.w_i8, p.scales_f16, 128)
    a0, a1 = p.a_bf16[0:1], p.a_bf16[1:2]
    # 2*a0 and a0 + (power-of-two multiple) stay exactly representable in bf16
    a_sum = wl.f32_to_bf16_bits((2.0 * bf16_bits_to_f64(a0)).astype(np.float32))
    y0, _ = orc.linear(a0, w)
    y1, _ = orc.linear(a1, w)
    y2, _ = orc.linear(a_sum, w)
    assert np.allclose(y2, 2.0 * y0, rtol=1e-13, atol=0)
    both, _ = orc.linear(p.a_bf16, w)
    assert np.array_equal(both[0:1], y0) and np.array_equal(both[1:2], y1)
    # additivity checked in fp64 space, away from bf16 rounding of the sum
    a = bf16_bits_to_f64(p.a_bf16)
    assert np.allclose((0.25 * a[0] - 3.0 * a[1]) @ w, 0.25 * y0[0] - 3.0 * y1[0], rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("maker", [wl.make_w4, wl.make_w8])
def test_bound_dominates_and_matches_float64_product(maker):
    p = maker(3, 640, 40, seed=30)
    y, b = orc.solve(p)
    assert y.shape == (3, 40) and b.shape == (3, 40)
    assert np.all(b >= np.abs(y) - 1e-12)
    w = orc.dequant_w4(p.qweight, p.scales_f16, p.qzeros, 128) if p.bits == 4 else \
        orc.dequant_w8(p.w_i8, p.scales_f16, 128)
    a = bf16_bits_to_f64(p.a_bf16)
    ref = np.einsum("mk,kn->mn", a, w)                      # a second contraction routine
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)
    # transposition guard: contracting over the wrong axis cannot even broadcast here
    assert w.shape == (640, 40) and a.shape == (3, 640)


@pytest.mark.parametrize("maker", [wl.make_w4, wl.make_w8])
def test_column_subset_equals_full(maker):
    p = maker(2, 256, 48, seed=33)
    y, b = orc.solve(p)
    cols = np.array([47, 0, 9, 10, 33, 8])
    ys, bs = orc.solve(p, columns=cols)
    assert np.array_equal(ys, y[:, cols]) and np.array_equal(bs, b[:, cols])
