"""tf_pack_awq / tf_pack_w8 on the host: header, determinism, and layout read back == oracle unpack."""
import numpy as np
import pytest

from oracle import tilefuse_oracle as orc
from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import build as tfbuild
from paper_2606_11357_b200 import workloads as wl
from helpers import read_blob, read_header


@pytest.fixture(scope="module", autouse=True)
def _built():
    tfbuild.build()


@pytest.mark.parametrize("K,N", [(128, 8), (256, 64), (384, 72), (128, 200), (512, 136)])
def test_w4_layout_round_trip(K, N):
    p = wl.make_w4(1, K, N, seed=K + N)
    blob = tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, N)
    h = read_header(blob)
    assert h["magic"] == 0x31424654 and h["version"] == 1 and h["bits"] == 4
    assert (h["K"], h["N"], h["group_size"]) == (K, N, 128)
    assert h["n_padded"] == -(-N // 64) * 64 and h["strips"] * 64 == h["n_padded"] and h["ktiles"] == K // 128
    assert h["tile_bytes"] == 4256 and h["tiles_offset"] == 256 and h["total_bytes"] == blob.nbytes
    q, z, s = read_blob(blob, 4, K, N)
    assert np.array_equal(q[:, :N], orc.unpack_awq(p.qweight))
    assert np.array_equal(z[:, :N], orc.unpack_awq(p.qzeros))
    assert np.array_equal(s[:, :N], p.scales_f16.view(np.uint16))
    # padded columns dequantize to exactly zero: q == z and s == 0
    assert not q[:, N:].any() and not z[:, N:].any() and not s[:, N:].any()
    assert np.array_equal(blob, tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, N))


@pytest.mark.parametrize("K,N", [(128, 8), (256, 64), (384, 72), (256, 136)])
def test_w8_layout_round_trip(K, N):
    p = wl.make_w8(1, K, N, seed=K + N)
    p.w_i8[0, 0], p.w_i8[K - 1, N - 1] = -128, 127
    blob = tf.tf_pack_w8(p.w_i8, p.scales_f16, K, N)
    h = read_header(blob)
    assert h["bits"] == 8 and h["tile_bytes"] == 8320 and h["total_bytes"] == blob.nbytes
    q, _, s = read_blob(blob, 8, K, N)
    assert np.array_equal(q[:, :N], p.w_i8)
    assert np.array_equal(s[:, :N], p.scales_f16.view(np.uint16))
    assert not q[:, N:].any() and not s[:, N:].any()


def test_group_size_multiple_of_tile_replicates_metadata():
    """group_size = 256: both k-tiles of a group carry the same scales and zeros."""
    K, N, g = 512, 64, 256
    p = wl.make_w4(1, K, N, seed=3, group_size=g)
    blob = tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, N, g)
    q, z, s = read_blob(blob, 4, K, N, g)
    assert np.array_equal(q, orc.unpack_awq(p.qweight))
    assert np.array_equal(z, np.repeat(orc.unpack_awq(p.qzeros), 2, axis=0))
    assert np.array_equal(s, np.repeat(p.scales_f16.view(np.uint16), 2, axis=0))


@pytest.mark.parametrize("g,tile_bytes", [(64, 4416), (32, 4736)])
@pytest.mark.parametrize("K,N", [(128, 8), (384, 72), (256, 200)])
def test_w4_group_sizes_below_the_tile(K, N, g, tile_bytes):
    """Group sizes 64 and 32: a tile carries two or four scale blocks followed by as many zero blocks."""
    p = wl.make_w4(1, K, N, seed=K + N + g, group_size=g)
    blob = tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, N, g)
    h = read_header(blob)
    assert h["group_size"] == g and h["tile_bytes"] == tile_bytes and h["total_bytes"] == blob.nbytes
    assert blob.nbytes == 256 + (-(-N // 64)) * (K // 128) * tile_bytes == tf.tf_packed_size(4, K, N, g)
    q, z, s = read_blob(blob, 4, K, N, g)
    assert np.array_equal(q[:, :N], orc.unpack_awq(p.qweight))
    assert np.array_equal(z[:, :N], orc.unpack_awq(p.qzeros))
    assert np.array_equal(s[:, :N], p.scales_f16.view(np.uint16))
    assert not q[:, N:].any() and not z[:, N:].any() and not s[:, N:].any()


def test_group_sizes_that_are_not_legal():
    assert tf.tf_packed_size(4, 1024, 64, 16) == 0 and tf.tf_packed_size(4, 1024, 64, 48) == 0
    assert tf.tf_packed_size(8, 1024, 64, 64) == 0           # below the tile: the 4-bit format only
    assert tf.tf_packed_size(4, 1024, 64, 64) > 0 and tf.tf_packed_size(4, 1024, 64, 32) > 0


def test_blob_is_tile_major_and_contiguous_per_strip():
    """Changing one weight changes bytes only inside that weight's tile payload."""
    K, N = 384, 128
    p = wl.make_w4(1, K, N, seed=8, keep_raw=True)
    base = tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, N)
    q2 = p.raw["q"].copy()
    k, n = 200, 70                                   # strip 1, k-tile 1
    q2[k, n] ^= 0xF
    other = tf.tf_pack_awq(wl.awq_pack_words(q2), p.scales_f16, p.qzeros, K, N)
    diff = np.nonzero(base != other)[0]
    lo = 256 + (1 * 3 + 1) * 4256
    assert len(diff) == 1 and lo <= diff[0] < lo + 4096
