"""The fused W4A16 GEMV on the AWQ arrays themselves (the layout arm of the Section 5.5 ablation): same
acceptance rule against the fp64 oracle as the pre-tiled kernels, including the group sizes below 128 that
the tile format does not cover."""
import numpy as np
import pytest
import torch

from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import workloads as wl
import gpu_util as gu
from helpers import bf16_bits_to_f64

pytestmark = pytest.mark.gpu


def run_raw(p, a_bits=None):
    a = gu.to_device_bf16(p.a_bf16 if a_bits is None else a_bits)
    M, K, N, g = a.shape[0], p.K, p.N, p.group_size
    qw = torch.from_numpy(p.qweight.view(np.int32)).cuda()
    sc = torch.from_numpy(p.scales_f16.view(np.int16)).cuda()
    qz = torch.from_numpy(p.qzeros.view(np.int32)).cuda()
    guard = 512
    ybuf = torch.full((guard + M * N + guard,), gu.CANARY, dtype=torch.int16, device="cuda")
    y = ybuf[guard:guard + M * N].view(torch.bfloat16).view(M, N)
    ws_bytes = tf.tf_gemv_awq_raw_workspace_size(M, K, N, g)
    assert ws_bytes > 0
    ws = torch.full((ws_bytes + 1024,), 0xA5, dtype=torch.uint8, device="cuda")   # no initial contents required
    tf.tf_gemv_awq_raw(qw, sc, qz, a, y, M, K, N, g, ws[:ws_bytes])
    torch.cuda.synchronize()
    raw = ybuf.cpu().numpy().view(np.uint16)
    assert np.all(raw[:guard] == gu.CANARY) and np.all(raw[guard + M * N:] == gu.CANARY), "write outside y"
    assert bool((ws[ws_bytes:] == 0xA5).all()), "write outside the workspace"
    return raw[guard:guard + M * N].reshape(M, N).copy()


SHAPES = [(1, 128, 8), (1, 256, 64), (2, 256, 72), (3, 384, 200), (4, 512, 256), (5, 640, 264), (8, 1024, 1000),
          (9, 512, 136), (16, 1152, 320), (1, 8192, 8), (16, 4096, 64), (7, 2048, 2056), (12, 640, 328)]


@pytest.mark.parametrize("M,K,N", SHAPES)
@pytest.mark.parametrize("g", [128, 64, 32])
def test_raw_gemv_matches_oracle(M, K, N, g):
    p = wl.make_w4(M, K, N, seed=M * 7919 + K + N + g, group_size=g)
    gu.check_against_oracle(p, run_raw(p))


@pytest.mark.parametrize("M,K,N", [(1, 4096, 4096), (4, 4096, 1024), (16, 4096, 14336), (1, 14336, 4096)])
def test_raw_gemv_layer_shapes_on_sampled_columns(M, K, N):
    p = wl.config1(M, K, N)
    y = run_raw(p)
    cols = np.unique(np.concatenate([np.arange(0, 16), np.arange(N - 16, N),
                                     np.random.default_rng(3).integers(0, N, size=96)]))
    gu.check_against_oracle(p, y, columns=cols)


def test_raw_gemv_q_equals_z_gives_exact_zero():
    from oracle import tilefuse_oracle as orc
    M, K, N, g = 4, 1024, 192, 64
    p = wl.make_w4(M, K, N, seed=5, group_size=g)
    p.qweight = wl.awq_pack_words(np.repeat(orc.unpack_awq(p.qzeros), g, axis=0))
    assert not bf16_bits_to_f64(run_raw(p)).any()


def test_raw_and_pretiled_agree_to_rounding():
    """Two routes to the same fp32-accumulated product: they may differ in summation order only."""
    p = wl.make_w4(8, 2048, 520, seed=21)
    y_raw, y_tiled = bf16_bits_to_f64(run_raw(p)), bf16_bits_to_f64(gu.run(p, "gemv"))
    assert np.max(np.abs(y_raw - y_tiled)) <= 2.0 ** -7 * np.max(np.abs(y_tiled))


def test_raw_gemv_one_hot_activations_pick_exact_weights():
    from oracle import tilefuse_oracle as orc
    K, N, g = 512, 136, 32
    p = wl.make_w4(1, K, N, seed=78, group_size=g)
    w = orc.dequant_w4(p.qweight, p.scales_f16, p.qzeros, g)
    ks = [0, 1, 2, 3, 4, 15, 16, 31, 32, 63, 64, 127, 128, 255, 300, 511]
    a = np.zeros((len(ks), K), dtype=np.uint16)
    for i, k in enumerate(ks):
        a[i, k] = 0x3F80
    y = run_raw(p, a_bits=a)
    want = wl.f32_to_bf16_bits(w[ks].astype(np.float32))
    assert np.array_equal(bf16_bits_to_f64(y), bf16_bits_to_f64(want))


def _awq_on_device(p):
    return (torch.from_numpy(p.qweight.view(np.int32)).cuda(), torch.from_numpy(p.scales_f16.view(np.int16)).cuda(),
            torch.from_numpy(p.qzeros.view(np.int32)).cuda())


@pytest.mark.parametrize("K,N,g", [(128, 8, 128), (384, 72, 128), (512, 200, 256), (1024, 1096, 64), (256, 136, 32), (4096, 4096, 128)])
def test_device_packer_writes_the_host_packers_bytes(K, N, g):
    """Pre-tiling on the GPU: byte for byte the blob tf_pack_awq writes (header, weights, scales, zeros, padding)."""
    p = wl.make_w4(1, K, N, seed=700 + K + g, group_size=g)
    want = tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, N, g)
    qw, sc, qz = _awq_on_device(p)
    guard = 256
    buf = torch.full((guard + want.nbytes + guard,), 0xA5, dtype=torch.uint8, device="cuda")
    tf.tf_pack_awq_device(qw, sc, qz, K, N, g, buf[guard:guard + want.nbytes])
    torch.cuda.synchronize()
    got = buf.cpu().numpy()
    assert np.all(got[:guard] == 0xA5) and np.all(got[guard + want.nbytes:] == 0xA5), "write outside the blob"
    assert np.array_equal(got[guard:guard + want.nbytes], want)


@pytest.mark.parametrize("M,K,N,g", [(24, 512, 200, 128), (130, 1024, 328, 64), (300, 2048, 1096, 128), (64, 256, 136, 32)])
def test_gemm_on_the_raw_awq_arrays(M, K, N, g):
    """The GEMM arm of the layout ablation: re-tiled on the fly, then the pre-tiled GEMM; parity against the oracle and
    bit-identical to the pre-tiled path on the offline blob."""
    p = wl.make_w4(M, K, N, seed=800 + M, group_size=g)
    qw, sc, qz = _awq_on_device(p)
    a = gu.to_device_bf16(p.a_bf16)
    y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(tf.tf_gemm_awq_raw_workspace_size(M, K, N, g), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        tf.tf_gemm_awq_raw(qw, sc, qz, a, y, M, K, N, g, ws)
    assert tf.tf_device_status(ws) == 0
    gu.check_against_oracle(p, gu.bits_of(y))
    blob = torch.from_numpy(gu.pack(p)).cuda()
    y2 = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    ws2 = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMM_W4A16, M, K, N), dtype=torch.uint8, device="cuda")
    tf.tf_gemm_w4a16_grouped(blob, a, y2, M, K, N, g, ws2)
    torch.cuda.synchronize()
    assert np.array_equal(gu.bits_of(y), gu.bits_of(y2))
