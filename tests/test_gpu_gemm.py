"""Parity of tf_gemm_w4a16 / tf_gemm_w8a16 (tcgen05 path) with the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import tilefuse_oracle as orc
from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import workloads as wl
from helpers import bf16_bits_to_f64
import gpu_util as gu

pytestmark = pytest.mark.gpu

# (M, K, N): single tile, ragged M and N, several token tiles, several n tiles, odd strip count, deep K
SMALL = [(32, 128, 128), (1, 128, 8), (16, 256, 64), (33, 256, 136), (100, 384, 200), (128, 512, 256),
         (200, 256, 384), (256, 1024, 128), (300, 640, 320), (513, 512, 1000), (64, 4096, 192)]


@pytest.mark.parametrize("M,K,N", SMALL)
def test_gemm_w4_small(M, K, N):
    p = wl.make_w4(M, K, N, seed=M * 100003 + K + N)
    gu.check_against_oracle(p, gu.run(p, "gemm"))


@pytest.mark.parametrize("M,K,N", SMALL)
def test_gemm_w8_small(M, K, N):
    p = wl.make_w8(M, K, N, seed=M * 100003 + K + N)
    p.w_i8[0, 0], p.w_i8[K - 1, N - 1] = -128, 127
    gu.check_against_oracle(p, gu.run(p, "gemm"))


@pytest.mark.parametrize("bits", [4, 8])
def test_unit_scales_integer_activations_are_exact(bits):
    """s = 1 and small-integer activations: operands, products and fp32 sums are all exact, so any
    misplaced element of either MMA operand (descriptor, swizzle, k permutation) changes the result."""
    M, K, N = 160, 512, 264
    rng = np.random.default_rng(2)
    ai = rng.integers(-4, 5, size=(M, K))
    p = (wl.make_w4 if bits == 4 else wl.make_w8)(M, K, N, seed=6, keep_raw=True)
    p.a_bf16 = wl.f32_to_bf16_bits(ai.astype(np.float32))
    p.scales_f16 = np.ones_like(p.scales_f16)
    y = bf16_bits_to_f64(gu.run(p, "gemm"))
    q = p.raw["q"].astype(np.int64)
    if bits == 4:
        q = q - np.repeat(p.raw["z"].astype(np.int64), 128, 0)
    exact = ai.astype(np.int64) @ q
    want = bf16_bits_to_f64(wl.f32_to_bf16_bits(exact.astype(np.float32)))
    assert np.array_equal(y, want)


def _round_to_bf16(v: np.ndarray) -> np.ndarray:
    """fp64 -> nearest bf16 value (8 significant bits, ties to even), returned as fp64."""
    m, e = np.frexp(v)                       # v = m * 2^e, 0.5 <= |m| < 1
    return np.ldexp(np.round(m * 256.0), e - 8)


@pytest.mark.parametrize("bits", [4, 8])
def test_one_hot_activations_pick_weights(bits):
    """a = e_k: y[n] is the GEMM's weight operand itself.  W4: bf16((q - z) * s), one rounding of the exact product
    with the fp16 scale.  W8: the scale is split into its upper 8 bits and the rest, w = bf16(q * hi + bf16(q * lo))."""
    K, N = 256, 136
    p = (wl.make_w4 if bits == 4 else wl.make_w8)(1, K, N, seed=77, keep_raw=True)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    ks = list(range(0, 256, 7)) + [255]
    a = np.zeros((len(ks), K), dtype=np.uint16)
    for i, k in enumerate(ks):
        a[i, k] = 0x3F80
    y = bf16_bits_to_f64(gu.run(p, "gemm", blob_dev=blob, a_bits=a))
    qi = p.raw["q"].astype(np.float64)
    s = np.repeat(p.scales_f16.astype(np.float64), 128, 0)
    if bits == 4:
        qi = qi - np.repeat(p.raw["z"].astype(np.float64), 128, 0)
        w = _round_to_bf16(qi * s)
    else:
        s_hi = s.astype(np.float32).view(np.uint32) & np.uint32(0xFFFF0000)         # truncated to bf16
        s_hi = s_hi.view(np.float32).astype(np.float64)
        w = _round_to_bf16(qi * s_hi + _round_to_bf16(qi * (s - s_hi)))
    assert np.array_equal(y, w[ks])


def test_q_equals_z_gives_exact_zero():
    M, K, N = 70, 512, 192
    p = wl.make_w4(M, K, N, seed=5)
    z = orc.unpack_awq(p.qzeros)
    p.qweight = wl.awq_pack_words(np.repeat(z, 128, axis=0))
    assert not bf16_bits_to_f64(gu.run(p, "gemm")).any()


@pytest.mark.parametrize("bits", [4, 8])
def test_deterministic(bits):
    p = (wl.make_w4 if bits == 4 else wl.make_w8)(384, 1024, 512, seed=9)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    assert np.array_equal(gu.run(p, "gemm", blob_dev=blob), gu.run(p, "gemm", blob_dev=blob))


def test_back_to_back_launches_are_independent():
    """GEMMs queued back to back with different activations and shapes give what they give alone."""
    stream = torch.cuda.Stream()
    cases = []
    for (M, K, N, seed) in [(256, 1024, 1024, 1), (256, 1024, 1024, 2), (64, 2048, 512, 3), (300, 512, 1000, 4)]:
        p = wl.make_w4(M, K, N, seed=seed)
        cases.append((p, torch.from_numpy(gu.pack(p)).cuda(), gu.to_device_bf16(p.a_bf16),
                      torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")))
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMM_W4A16, 4096, 4096, 4096), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for rep in range(3):
            for (p, blob, a, y) in cases:
                tf.tf_gemm_w4a16(blob, a, y, p.M, p.K, p.N, ws, stream=stream)
    stream.synchronize()
    assert tf.tf_device_status(ws, stream=stream) == 0
    for (p, blob, a, y) in cases:
        assert np.array_equal(gu.bits_of(y), gu.run(p, "gemm", blob_dev=blob))


def test_gemm_agrees_with_gemv_range():
    """M <= 16 is legal for the GEMM too; both kernels must satisfy the same bound."""
    p = wl.make_w4(16, 1024, 256, seed=12)
    gu.check_against_oracle(p, gu.run(p, "gemm"))
    gu.check_against_oracle(p, gu.run(p, "gemv"))


def test_mismatched_blob_reports_status_and_leaves_y():
    p = wl.make_w4(32, 256, 128, seed=1)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    a = gu.to_device_bf16(p.a_bf16)
    y = torch.full((32, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMM_W8A16, 32, 256, 128), dtype=torch.uint8, device="cuda")
    tf.tf_gemm_w8a16(blob, a, y, 32, 256, 128, ws)
    assert tf.tf_device_status(ws) == 4
    assert bool((y == 7.0).all())


def test_config2_prefill_gemm_full_matrix():
    p = wl.config2()
    ratio = gu.check_against_oracle(p, gu.run(p, "gemm"))
    print(f"cfg2 max err/tol = {ratio:.4f}")


def test_config3_w8_gemm_full_matrix():
    p = wl.config3_gemm()
    gu.check_against_oracle(p, gu.run(p, "gemm"))


def test_config4_w4_gemm_k32768():
    p = wl.config4_gemm()
    gu.check_against_oracle(p, gu.run(p, "gemm"))


def test_max_m_ragged():
    p = wl.make_w4(4096, 256, 200, seed=3)
    gu.check_against_oracle(p, gu.run(p, "gemm"))


def test_maximum_dimensions_on_sampled_columns():
    """M = 4096, K = N = 32768: the largest problem the GEMM accepts (256 x 16 tiles of 256 k-tiles each, split evenly
    over the SMs), checked against the oracle on 129 sampled columns.  Codes drawn as whole words: uniform, as in make_w4."""
    M, K, N = 4096, 32768, 32768
    rng = np.random.default_rng(4343)
    p = wl.Problem("w4max", 4, M, K, N, 128, 4343, wl._activations(rng, M, K),
                   rng.uniform(0.001, 0.02, size=(K // 128, N)).astype(np.float32).astype(np.float16),
                   qweight=rng.integers(0, 2**32, size=(K, N // 8), dtype=np.uint32),
                   qzeros=rng.integers(0, 2**32, size=(K // 128, N // 8), dtype=np.uint32))
    cols = np.unique(np.concatenate([np.arange(0, N, 257), [N - 1]]))
    gu.check_against_oracle(p, gu.run(p, "gemm"), columns=cols)
