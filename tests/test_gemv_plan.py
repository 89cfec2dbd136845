"""Host logic of the GEMV launcher: the launch plan (tf_gemv_plan) for a grid of shapes, without a GPU.

The plan decides grid, warps, ring depth and which kernel variant runs; a wrong plan shows up on the GPU as a
launch failure or a hang, so its invariants are pinned here for every shape class, on the SM counts the library may
meet."""
import itertools

import pytest

from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import build as tfbuild

SMEM_HALF, SMEM_WHOLE = 110 * 1024, 220 * 1024


@pytest.fixture(scope="module", autouse=True)
def _built():
    tfbuild.build()


SHAPES = [(128, 8), (128, 64), (512, 200), (4096, 1024), (4096, 4096), (4096, 14336), (14336, 4096), (4096, 32768),
          (32768, 4096), (32768, 32768), (1024, 136), (256, 32768)]


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("sm_count", [148, 132, 80, 16])
def test_plan_invariants(bits, sm_count):
    for (K, N), M in itertools.product(SHAPES, (1, 2, 3, 8, 9, 16)):
        p = tf.tf_gemv_plan(bits, M, K, N, sm_count)
        tiles = (K // 128) * (-(-N // 64))
        assert 1 <= p["grid"] <= 256 and p["grid"] <= max(sm_count, 1) or p["cluster"] > 1
        assert p["threads"] == 32 * (p["consumers"] + 2) and 4 <= p["consumers"] <= 16
        assert p["stages"] >= 2
        assert p["cluster"] in (1, 2, 4, 8)
        assert 1 <= p["nclusters"] <= max(p["grid"], 1)                  # CTAs (or clusters) that take part
        if M > 8:
            assert p["full"] == 1 and p["i8"] == 0 and p["consumers"] <= 8
        if M <= 2:
            assert p["i8"] in (1, 2)                                     # both formats take the integer path at 1 and 2 tokens
            if p["i8"] == 2:                                             # piece table: a warp meets the same k-tiles on every pass
                per_cta = -(-tiles // p["nclusters"])
                assert (K // 128) % p["consumers"] == 0 and per_cta >= K // 128 + p["consumers"]
        else:
            assert p["i8"] == 0 and p["full"] == 1                       # the floating-point path takes the whole SM
        if p["cluster"] == 1 and tiles >= sm_count:
            assert p["grid"] == sm_count                                 # one persistent CTA per SM


def test_plan_of_the_benchmark_shapes_on_a_b200():
    """The shapes of the decode step on 148 SMs: which variant each gets (asserted again on the GPU by the chain tests)."""
    kind = lambda p: "cluster" if p["cluster"] > 1 else ("whole" if p["full"] else "half")
    for (K, N) in ((4096, 4096), (4096, 1024), (4096, 14336), (14336, 4096)):
        assert kind(tf.tf_gemv_plan(4, 1, K, N, 148)) == "half"
        assert kind(tf.tf_gemv_plan(4, 4, K, N, 148)) == "whole"
    # no GPU here: the cluster-occupancy query fails, so 9..16 tokens plan for global mode
    assert kind(tf.tf_gemv_plan(4, 16, 4096, 14336, 148)) == "whole"
    # long ranges of the integer path take the whole SM: 16 consumer warps on 4-bit tiles, 8 on int8 tiles
    p = tf.tf_gemv_plan(4, 1, 4096, 32768, 148)
    assert (p["full"], p["consumers"], p["i8"]) == (1, 16, 2)            # 111 tiles over 32 k-tiles: a warp keeps the pieces it has prepared
    p = tf.tf_gemv_plan(8, 1, 4096, 14336, 148)
    assert (p["full"], p["consumers"], p["i8"]) == (1, 8, 1)             # int8, whole SM: a table would cost a ring stage
    # the decode step's shapes take half an SM; 48 tiles over 32 k-tiles keep their pieces, 24 over 112 and 16 over 32 have none to keep
    assert [tf.tf_gemv_plan(4, 1, K, N, 148)["i8"] for (K, N) in ((4096, 14336), (14336, 4096), (4096, 4096))] == [2, 1, 1]
    for (K, N) in ((4096, 14336), (14336, 4096), (4096, 4096)):
        p = tf.tf_gemv_plan(4, 1, K, N, 148)
        assert (p["full"], p["consumers"]) == (0, 8)
    assert tf.tf_gemv_plan(4, 1, 4096 + 128, 14336, 148)["i8"] == 1      # 33 k-tiles over 8 warps: a warp would meet other k-tiles on its second pass
    p = tf.tf_gemv_plan(4, 1, 4096, 1024, 148)
    assert p["grid"] == 148 and p["nclusters"] == 64                     # 64 CTAs x 8 tiles take part, the grid stays one per SM
    p = tf.tf_gemv_plan(4, 1, 4096, 4096, 148)
    assert p["nclusters"] == 128                                         # 128 CTAs x 16 tiles: ranges line up with the strips


def test_plan_rejects_illegal_arguments():
    L = tf.lib()
    import ctypes
    out = (ctypes.c_int * 8)()
    ptr = ctypes.cast(out, ctypes.c_void_p)
    assert L.tf_gemv_plan(4, 1, 4096, 4096, 148, None) == 1
    assert L.tf_gemv_plan(5, 1, 4096, 4096, 148, ptr) == 2
    assert L.tf_gemv_plan(4, 17, 4096, 4096, 148, ptr) == 2
    assert L.tf_gemv_plan(4, 1, 100, 4096, 148, ptr) == 2
