"""tf_pack_concat: blobs side by side along N (fused QKV, fused gate + up).  The pin needs no GPU: the result must
be byte for byte what the packer gives for the column-concatenated inputs."""
import numpy as np
import pytest

from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import workloads as wl


def _concat_w4(parts):
    K, g = parts[0].K, parts[0].group_size
    N = sum(p.N for p in parts)
    return wl.Problem("fused", 4, parts[0].M, K, N, g, 0, parts[0].a_bf16,
                      np.concatenate([p.scales_f16 for p in parts], axis=1),
                      qweight=np.concatenate([p.qweight for p in parts], axis=1),
                      qzeros=np.concatenate([p.qzeros for p in parts], axis=1))


def _concat_w8(parts):
    K, g = parts[0].K, parts[0].group_size
    N = sum(p.N for p in parts)
    return wl.Problem("fused", 8, parts[0].M, K, N, g, 0, parts[0].a_bf16,
                      np.concatenate([p.scales_f16 for p in parts], axis=1),
                      w_i8=np.concatenate([p.w_i8 for p in parts], axis=1))


@pytest.mark.parametrize("widths", [(256, 64, 64), (128, 72), (64,), (192, 128, 8)])
def test_w4_concat_equals_pack_of_concatenated_inputs(widths):
    K = 384
    parts = [wl.make_w4(1, K, n, seed=40 + i) for i, n in enumerate(widths)]
    blobs = [tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, p.N) for p in parts]
    whole = _concat_w4(parts)
    expect = tf.tf_pack_awq(whole.qweight, whole.scales_f16, whole.qzeros, K, whole.N)
    got = tf.tf_pack_concat(blobs)
    assert got.nbytes == expect.nbytes == tf.tf_packed_size(4, K, whole.N)
    assert np.array_equal(got, expect)


def test_w8_concat_with_group_256():
    K, g = 512, 256
    parts = [wl.make_w8(1, K, n, seed=50 + i, group_size=g) for i, n in enumerate((128, 64, 40))]
    blobs = [tf.tf_pack_w8(p.w_i8, p.scales_f16, K, p.N, g) for p in parts]
    whole = _concat_w8(parts)
    assert np.array_equal(tf.tf_pack_concat(blobs), tf.tf_pack_w8(whole.w_i8, whole.scales_f16, K, whole.N, g))


def test_concat_is_associative():
    K = 256
    parts = [wl.make_w4(1, K, n, seed=60 + i) for i, n in enumerate((64, 128, 64))]
    b = [tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, p.N) for p in parts]
    assert np.array_equal(tf.tf_pack_concat([tf.tf_pack_concat(b[:2]), b[2]]), tf.tf_pack_concat(b))


def test_concat_rejects_what_it_cannot_join():
    K = 256
    a = wl.make_w4(1, K, 64, seed=1)
    b = wl.make_w4(1, K, 72, seed=2)          # does not end on a strip boundary
    c = wl.make_w4(1, 2 * K, 64, seed=3)      # another K
    d = wl.make_w8(1, K, 64, seed=4)          # another width of code
    ba, bb, bc = (tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, p.K, p.N) for p in (a, b, c))
    bd = tf.tf_pack_w8(d.w_i8, d.scales_f16, K, 64)
    tf.tf_pack_concat([ba, bb])               # an unaligned part may come last
    for bad, status in (([bb, ba], 2), ([ba, bc], 2), ([ba, bd], 2), ([], 2)):
        with pytest.raises(tf.TileFuseError) as e:
            tf.tf_pack_concat(bad)
        assert e.value.status == status
    broken = ba.copy()
    broken[0] ^= 0xFF                         # magic
    with pytest.raises(tf.TileFuseError) as e:
        tf.tf_pack_concat([broken, ba])
    assert e.value.status == 4
    small = np.empty(tf.tf_packed_size(4, K, 128) - 1, dtype=np.uint8)
    with pytest.raises(tf.TileFuseError) as e:
        tf.tf_pack_concat([ba, ba], out=small)
    assert e.value.status == 5
    # too wide for the problem statement
    wide = wl.make_w4(1, 128, 16384, seed=5)
    bw = tf.tf_pack_awq(wide.qweight, wide.scales_f16, wide.qzeros, 128, 16384)
    with pytest.raises(tf.TileFuseError) as e:
        tf.tf_pack_concat([bw, bw, bw])
    assert e.value.status == 2


@pytest.mark.parametrize("bits,K,N,g,parts", [(4, 256, 200, 128, 2), (4, 384, 328, 64, 3), (8, 256, 136, 128, 3), (4, 128, 64, 32, 1)])
def test_pack_shard_is_the_packer_on_the_column_slice(bits, K, N, g, parts):
    """tf_pack_shard cuts a column range out of a blob: byte for byte what the packer gives for the sliced inputs,
    and the shards tile the columns without gap or overlap."""
    p = wl.make_w4(1, K, N, seed=77, group_size=g, keep_raw=True) if bits == 4 else wl.make_w8(1, K, N, seed=77, group_size=g)
    full = (tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, N, g) if bits == 4 else tf.tf_pack_w8(p.w_i8, p.scales_f16, K, N, g))
    covered = 0
    for part in range(parts):
        n0, nc = tf.tf_shard_columns(N, part, parts)
        assert n0 == covered and nc > 0 and n0 % 64 == 0
        covered += nc
        shard = tf.tf_pack_shard(full, part, parts)
        if bits == 4:
            q, z = p.raw["q"][:, n0:n0 + nc], p.raw["z"][:, n0:n0 + nc]
            want = tf.tf_pack_awq(wl.awq_pack_words(q), np.ascontiguousarray(p.scales_f16[:, n0:n0 + nc]), wl.awq_pack_words(z), K, nc, g)
        else:
            want = tf.tf_pack_w8(np.ascontiguousarray(p.w_i8[:, n0:n0 + nc]), np.ascontiguousarray(p.scales_f16[:, n0:n0 + nc]), K, nc, g)
        assert np.array_equal(shard, want)
    assert covered == N


def test_pack_shard_errors():
    p = wl.make_w4(1, 128, 64, seed=78)
    full = tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, 128, 64)
    L = tf.lib()
    out = np.zeros(full.nbytes, dtype=np.uint8)
    assert L.tf_pack_shard(full.ctypes.data, 0, 2, out.ctypes.data, out.nbytes) == 2        # more parts than strips
    assert L.tf_pack_shard(full.ctypes.data, 1, 1, out.ctypes.data, out.nbytes) == 2        # part outside 0..parts-1
    assert L.tf_pack_shard(full.ctypes.data, 0, 1, out.ctypes.data, out.nbytes - 1) == 5
    assert L.tf_pack_shard(out.ctypes.data, 0, 1, full.ctypes.data, full.nbytes) == 4       # not a blob
