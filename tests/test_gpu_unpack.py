"""GPU unpack (the kernels' own decode helpers) must reproduce the packed inputs bit for bit."""
import numpy as np
import pytest
import torch

from oracle import tilefuse_oracle as orc
from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import workloads as wl
import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,N", [(128, 8), (384, 72), (256, 200), (1024, 1024), (4096, 4096)])
def test_unpack_w4_bit_exact(K, N):
    p = wl.make_w4(1, K, N, seed=K * 7 + N)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    q = torch.full((K, N), 0xEE, dtype=torch.uint8, device="cuda")
    z = torch.full((K // 128, N), 0xEE, dtype=torch.uint8, device="cuda")
    s = torch.zeros((K // 128, N), dtype=torch.float16, device="cuda")
    tf.tf_unpack_w4(blob, q, z, s, K, N)
    torch.cuda.synchronize()
    assert np.array_equal(q.cpu().numpy(), orc.unpack_awq(p.qweight))
    assert np.array_equal(z.cpu().numpy(), orc.unpack_awq(p.qzeros))
    assert np.array_equal(s.cpu().numpy().view(np.uint16), p.scales_f16.view(np.uint16))


@pytest.mark.parametrize("K,N", [(128, 8), (384, 72), (1024, 1000)])
def test_unpack_w8_bit_exact(K, N):
    p = wl.make_w8(1, K, N, seed=K + N)
    p.w_i8[0, 0], p.w_i8[K - 1, N - 1], p.w_i8[1, 1] = -128, 127, 0
    blob = torch.from_numpy(gu.pack(p)).cuda()
    q = torch.full((K, N), 0x5E, dtype=torch.int8, device="cuda")
    s = torch.zeros((K // 128, N), dtype=torch.float16, device="cuda")
    tf.tf_unpack_w8(blob, q, s, K, N)
    torch.cuda.synchronize()
    assert np.array_equal(q.cpu().numpy(), p.w_i8)
    assert np.array_equal(s.cpu().numpy().view(np.uint16), p.scales_f16.view(np.uint16))


def test_unpack_every_code_in_every_position():
    """All 16 codes at every (k mod 128, n mod 64) tile position."""
    K, N = 128, 64
    q = ((np.arange(K)[:, None] * 5 + np.arange(N)[None, :] * 3) % 16).astype(np.uint8)
    for shift in range(16):
        qq = (q + shift) % 16
        z = np.full((1, N), (shift * 7) % 16, dtype=np.uint8)
        blob = tf.tf_pack_awq(wl.awq_pack_words(qq), np.ones((1, N), np.float16), wl.awq_pack_words(z), K, N)
        out_q = torch.zeros((K, N), dtype=torch.uint8, device="cuda")
        out_z = torch.zeros((1, N), dtype=torch.uint8, device="cuda")
        tf.tf_unpack_w4(torch.from_numpy(blob).cuda(), out_q, out_z, None, K, N)
        assert np.array_equal(out_q.cpu().numpy(), qq) and np.array_equal(out_z.cpu().numpy(), z)


def test_mismatched_blob_leaves_outputs_untouched():
    p = wl.make_w4(1, 256, 64, seed=1)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    q = torch.full((256, 64), 0xEE, dtype=torch.uint8, device="cuda")
    tf.tf_unpack_w8(blob, q.view(torch.int8), None, 256, 64)      # W4 blob handed to the W8 decoder
    torch.cuda.synchronize()
    assert bool((q == 0xEE).all())
