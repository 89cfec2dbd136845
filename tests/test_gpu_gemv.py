"""Parity of tf_gemv_w4a16 / tf_gemv_w8a16 with the fp64 oracle, element by element."""
import copy

import numpy as np
import pytest
import torch

from oracle import tilefuse_oracle as orc
from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import workloads as wl
from helpers import bf16_bits_to_f64
import gpu_util as gu

pytestmark = pytest.mark.gpu

SMALL = [(1, 128, 8), (1, 128, 64), (2, 256, 72), (5, 384, 200), (8, 640, 128), (9, 512, 136),
         (16, 1152, 320), (3, 2048, 64), (1, 8192, 8), (16, 4096, 64), (7, 1024, 1000)]


@pytest.mark.parametrize("M,K,N", SMALL)
def test_gemv_w4_small(M, K, N):
    p = wl.make_w4(M, K, N, seed=M * 100003 + K + N)
    gu.check_against_oracle(p, gu.run(p, "gemv"))


@pytest.mark.parametrize("M,K,N", SMALL)
def test_gemv_w8_small(M, K, N):
    p = wl.make_w8(M, K, N, seed=M * 100003 + K + N)
    p.w_i8[0, 0], p.w_i8[K - 1, N - 1] = -128, 127
    gu.check_against_oracle(p, gu.run(p, "gemv"))


# ranges that pass over their k-tiles more than once, K a multiple of 128 x consumer warps: a warp of the integer path
# keeps the activation pieces of the k-tiles it has visited
PIECE_TABLE = [(1, 1024, 30000), (2, 1024, 30000), (1, 2048, 32768), (2, 2048, 20000), (1, 4096, 14336), (1, 4096, 32768),
               (2, 4096, 32768), (1, 3072, 20000)]


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("M,K,N", PIECE_TABLE)
def test_gemv_integer_path_with_piece_table(bits, M, K, N):
    if bits == 4:                               # int8 weights prepare their pieces per tile
        assert tf.tf_gemv_plan(bits, M, K, N)["i8"] == 2
    p = (wl.make_w4 if bits == 4 else wl.make_w8)(M, K, N, seed=M * 7 + K + N)
    y = gu.run(p, "gemv")
    gu.check_against_oracle(p, y)
    assert np.array_equal(y, gu.run(p, "gemv"))


@pytest.mark.parametrize("bits", [4, 8])
def test_one_hot_activations_pick_exact_weights(bits):
    """a = e_k: y[n] must be bf16(w[k][n]) exactly (one rounding at the output, none on the weights)."""
    K, N = 512, 136
    p = (wl.make_w4 if bits == 4 else wl.make_w8)(1, K, N, seed=77)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    w = orc.dequant_w4(p.qweight, p.scales_f16, p.qzeros, 128) if bits == 4 else \
        orc.dequant_w8(p.w_i8, p.scales_f16, 128)
    ks = [0, 1, 2, 3, 4, 15, 16, 63, 64, 127, 128, 255, 300, 511]
    a = np.zeros((len(ks), K), dtype=np.uint16)
    for i, k in enumerate(ks):
        a[i, k] = 0x3F80
    y = gu.run(p, "gemv", blob_dev=blob, a_bits=a)
    want = wl.f32_to_bf16_bits(w[ks].astype(np.float32))        # fp64 -> fp32 exact here (<= 24 bits)
    assert np.array_equal(bf16_bits_to_f64(y), bf16_bits_to_f64(want))


def test_q_equals_z_gives_exact_zero():
    M, K, N = 4, 1024, 192
    p = wl.make_w4(M, K, N, seed=5)
    z = orc.unpack_awq(p.qzeros)
    p.qweight = wl.awq_pack_words(np.repeat(z, 128, axis=0))
    y = gu.run(p, "gemv")
    assert not bf16_bits_to_f64(y).any()


def test_unit_scales_integer_activations_are_exact():
    """s = 1, integer activations: every partial sum is an integer below 2^24, so fp32 is exact."""
    M, K, N = 3, 512, 64
    rng = np.random.default_rng(2)
    ai = rng.integers(-4, 5, size=(M, K))
    p = wl.make_w4(M, K, N, seed=6, keep_raw=True)
    p.a_bf16 = wl.f32_to_bf16_bits(ai.astype(np.float32))
    p.scales_f16 = np.ones_like(p.scales_f16)
    y = bf16_bits_to_f64(gu.run(p, "gemv"))
    exact = ai.astype(np.int64) @ (p.raw["q"].astype(np.int64) - np.repeat(p.raw["z"].astype(np.int64), 128, 0))
    want = bf16_bits_to_f64(wl.f32_to_bf16_bits(exact.astype(np.float32)))
    assert np.array_equal(y, want)


@pytest.mark.parametrize("bits", [4, 8])
def test_deterministic_and_independent_of_stale_output(bits):
    p = (wl.make_w4 if bits == 4 else wl.make_w8)(16, 4096, 1024, seed=9)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    y1, y2 = gu.run(p, "gemv", blob_dev=blob), gu.run(p, "gemv", blob_dev=blob)
    assert np.array_equal(y1, y2)


@pytest.mark.parametrize("bits", [4, 8])
def test_back_to_back_launches_are_independent(bits):
    """Calls queued back to back on one stream (nothing in between, shared workspace, different shapes and
    activations) must each give what they give alone.  Shared-memory state of one launch must not leak into
    the next: this is the sequence a decode step issues."""
    stream = torch.cuda.Stream()
    maker = wl.make_w4 if bits == 4 else wl.make_w8
    op = tf.TF_OP_GEMV_W4A16 if bits == 4 else tf.TF_OP_GEMV_W8A16
    fn = tf.tf_gemv_w4a16 if bits == 4 else tf.tf_gemv_w8a16
    cases = []
    for (M, K, N, seed) in [(1, 4096, 9472, 1), (4, 4096, 9472, 2), (4, 4096, 9472, 3), (16, 4096, 2048, 4),
                            (1, 14336, 1024, 5), (4, 14336, 1024, 6), (8, 1024, 4096, 7), (2, 4096, 9472, 8)]:
        p = maker(M, K, N, seed=seed)
        cases.append((p, torch.from_numpy(gu.pack(p)).cuda(), gu.to_device_bf16(p.a_bf16),
                      torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")))
    ws = torch.zeros(tf.tf_workspace_size(op, 16, 4096, 4096), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for rep in range(3):
            for (p, blob, a, y) in cases:
                fn(blob, a, y, p.M, p.K, p.N, ws, stream=stream)
    stream.synchronize()
    assert tf.tf_device_status(ws, stream=stream) == 0
    for (p, blob, a, y) in cases:
        gu.check_against_oracle(p, gu.bits_of(y))
        alone = gu.run(p, "gemv", blob_dev=blob)
        assert np.array_equal(gu.bits_of(y), alone)


def test_mismatched_blob_reports_status_and_leaves_y():
    p = wl.make_w4(1, 256, 64, seed=1)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    a = gu.to_device_bf16(p.a_bf16)
    y = torch.full((1, 64), 7.0, dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMV_W8A16, 1, 256, 64), dtype=torch.uint8, device="cuda")
    tf.tf_gemv_w8a16(blob, a, y, 1, 256, 64, ws)                 # W4 blob handed to the W8 kernel
    assert tf.tf_device_status(ws) == 4
    assert bool((y == 7.0).all())


def test_config0_full_matrix():
    p = wl.config0()
    ratio = gu.check_against_oracle(p, gu.run(p, "gemv"))
    print(f"cfg0 max err/tol = {ratio:.4f}")


@pytest.mark.parametrize("K,N", wl.LLAMA3_8B_SHAPES)
@pytest.mark.parametrize("M", [1, 4, 16])
def test_config1_decode_sweep(M, K, N):
    p = wl.config1(M, K, N)
    gu.check_against_oracle(p, gu.run(p, "gemv"))


def test_config1_step_replayed_as_one_graph():
    """The twelve calls of the decode step the way the benchmark issues them: one stream, one workspace, captured
    once into a CUDA graph and replayed, every kernel free to start under its predecessor's tail.  Every result is
    checked against the oracle on the first and last columns and a seeded sample in between."""
    probs = [wl.config1(M, K, N) for M in (1, 4, 16) for (K, N) in wl.LLAMA3_8B_SHAPES]
    packed = [torch.from_numpy(gu.pack(p)).cuda() for p in probs]
    acts = [gu.to_device_bf16(p.a_bf16) for p in probs]
    ys = [torch.full((p.M, p.N), float("nan"), dtype=torch.bfloat16, device="cuda") for p in probs]
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, 16, 4096, 4096), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        for p, b, a, y in zip(probs, packed, acts, ys):            # first use outside the capture
            tf.tf_gemv_w4a16(b, a, y, p.M, p.K, p.N, ws, stream=stream)
        stream.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            for p, b, a, y in zip(probs, packed, acts, ys):
                tf.tf_gemv_w4a16(b, a, y, p.M, p.K, p.N, ws, stream=stream)
        for y in ys:
            y.fill_(float("nan"))
        for _ in range(3):
            graph.replay()
        stream.synchronize()
    assert tf.tf_device_status(ws) == 0
    rng = np.random.default_rng(17)
    for p, y in zip(probs, ys):
        cols = np.unique(np.concatenate([np.arange(0, 8), np.arange(p.N - 8, p.N), rng.integers(0, p.N, size=48)]))
        gu.check_against_oracle(p, gu.bits_of(y), columns=cols)


def test_config3_w8_gemv():
    p = wl.config3_gemv()
    gu.check_against_oracle(p, gu.run(p, "gemv"))


def test_config4_w4_gemv_32k_columns():
    p = wl.config4_gemv()
    gu.check_against_oracle(p, gu.run(p, "gemv"))


def test_max_k_gemv():
    p = wl.make_w4(2, 32768, 128, seed=44)
    gu.check_against_oracle(p, gu.run(p, "gemv"))


def test_maximum_dimensions_on_sampled_columns():
    """K = N = 32768, the largest shape the library accepts (131072 tiles, a 558 MB blob): one token (integer path,
    whole SM, piece table) and sixteen, checked against the oracle on 257 sampled columns (first, last and a stride
    that meets every column position of a strip).  The codes are drawn as whole 32-bit words: uniform codes, like
    make_w4's, at a fraction of the time."""
    K = N = 32768
    rng = np.random.default_rng(4242)
    p = wl.Problem("w4max", 4, 16, K, N, 128, 4242, wl._activations(rng, 16, K),
                   rng.uniform(0.001, 0.02, size=(K // 128, N)).astype(np.float32).astype(np.float16),
                   qweight=rng.integers(0, 2**32, size=(K, N // 8), dtype=np.uint32),
                   qzeros=rng.integers(0, 2**32, size=(K // 128, N // 8), dtype=np.uint32))
    blob = torch.from_numpy(gu.pack(p)).cuda()
    cols = np.unique(np.concatenate([np.arange(0, N, 129), [N - 1]]))
    for M in (16, 1):
        q = copy.copy(p)
        q.M, q.a_bf16 = M, p.a_bf16[:M].copy()
        y = gu.run(q, "gemv", blob_dev=blob)
        gu.check_against_oracle(q, y, columns=cols)
