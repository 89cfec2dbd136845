"""The C-ABI library: loads without a GPU, exports what the header declares, validates arguments."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import build as tfbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    tfbuild.build()


def test_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "tilefuse.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(tf_[a-z0-9_]+)\s*\(", header))
    assert declared == set(tf.EXPORTS)
    L = tf.lib()
    for name in declared:
        assert getattr(L, name) is not None
    assert tf.tf_version() == 100


def test_packed_size():
    assert tf.tf_packed_size(4, 4096, 4096) == 256 + 64 * 32 * 4256
    assert tf.tf_packed_size(8, 4096, 14336) == 256 + 224 * 32 * 8320
    assert tf.tf_packed_size(4, 128, 8) == 256 + 4256              # N padded to one strip
    assert tf.tf_packed_size(4, 256, 72) == 256 + 2 * 2 * 4256
    for bad in [(3, 128, 8, 128), (4, 64, 8, 128), (4, 128, 4, 128), (4, 128, 12, 128),
                (4, 32768 + 128, 8, 128), (4, 128, 32768 + 8, 128), (4, 256, 8, 16), (8, 256, 8, 64), (4, 384, 8, 256)]:
        assert tf.tf_packed_size(*bad) == 0
    assert tf.tf_packed_size(8, 512, 8, 512) > 0                    # per-channel: group_size == K
    assert tf.tf_packed_size(4, 256, 8, 64) == 256 + 2 * 4416 and tf.tf_packed_size(4, 256, 8, 32) == 256 + 2 * 4736


def test_pack_errors_are_codes_not_crashes():
    L = tf.lib()
    out = np.zeros(256 + 4256, dtype=np.uint8)
    qw = np.zeros((128, 1), dtype=np.uint32)
    sc = np.zeros((1, 8), dtype=np.float16)
    qz = np.zeros((1, 1), dtype=np.uint32)
    args = (qw.ctypes.data, sc.ctypes.data, qz.ctypes.data)
    assert L.tf_pack_awq(None, args[1], args[2], 128, 8, 128, out.ctypes.data, out.nbytes) == 1
    assert L.tf_pack_awq(*args, 128, 8, 128, None, out.nbytes) == 1
    assert L.tf_pack_awq(*args, 100, 8, 128, out.ctypes.data, out.nbytes) == 2
    assert L.tf_pack_awq(*args, 128, 8, 128, out.ctypes.data, out.nbytes - 1) == 5
    assert L.tf_pack_awq(*args, 128, 8, 128, out.ctypes.data, out.nbytes) == 0
    assert L.tf_pack_w8(None, args[1], 128, 8, 128, out.ctypes.data, out.nbytes) == 1
    with pytest.raises(tf.TileFuseError):
        tf.tf_pack_awq(qw, sc, qz, 128, 12, 128, out=out)


def test_compute_calls_validate_before_touching_the_gpu():
    """NULL / shape / alignment / workspace errors are reported without any CUDA call."""
    L = tf.lib()
    p = ctypes.c_void_p
    ok = p(0x1000)
    assert L.tf_gemv_w4a16(None, ok, ok, 1, 128, 8, None, 0, None) == 1
    assert L.tf_gemv_w4a16(ok, ok, ok, 17, 128, 8, None, 0, None) == 2
    assert L.tf_gemv_w4a16(ok, ok, ok, 0, 128, 8, None, 0, None) == 2
    assert L.tf_gemv_w8a16(ok, ok, ok, 1, 100, 8, None, 0, None) == 2
    assert L.tf_gemv_w4a16(ok, p(0x1008), ok, 1, 128, 8, None, 0, None) == 3
    assert L.tf_gemm_w4a16(ok, ok, ok, 4097, 128, 8, ok, 1 << 20, None) == 2
    assert L.tf_gemm_w4a16(ok, ok, ok, 16, 128, 8, None, 0, None) == 5
    assert L.tf_unpack_w4(None, ok, ok, ok, 128, 8, 128, None) == 1
    assert L.tf_unpack_w4(ok, ok, ok, ok, 128, 9, 128, None) == 2
    assert L.tf_device_status(None, None) == 1
    raw = L.tf_gemv_awq_raw
    assert raw(None, ok, ok, ok, ok, 1, 128, 8, 128, ok, 1 << 20, None) == 1
    assert raw(ok, ok, ok, ok, ok, 17, 128, 8, 128, ok, 1 << 20, None) == 2
    assert raw(ok, ok, ok, ok, ok, 1, 128, 8, 96, ok, 1 << 20, None) == 2       # group size not 32 / 64 / 128
    assert raw(ok, ok, ok, ok, ok, 1, 160, 8, 64, ok, 1 << 20, None) == 2       # K not a multiple of it
    assert raw(ok, ok, ok, ok, ok, 1, 128, 12, 128, ok, 1 << 20, None) == 2
    assert raw(ok, p(0x1004), ok, ok, ok, 1, 128, 8, 128, ok, 1 << 20, None) == 3
    assert tf.tf_gemv_awq_raw_workspace_size(1, 4096, 4096, 100) == 0
    assert tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, 1, 4096, 4096) >= 4096
    assert tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, 17, 4096, 4096) == 0
    assert L.tf_gemv_w4a16(ok, ok, ok, 1, 128, 8, None, 0, None) == 5
    assert tf.tf_workspace_size(tf.TF_OP_GEMM_W4A16, 2048, 4096, 14336) >= 16
    assert tf.tf_workspace_size(tf.TF_OP_GEMM_W4A16, 5000, 4096, 14336) == 0
    assert tf.tf_workspace_size(99, 1, 4096, 4096) == 0
    for code in range(9):
        assert len(L.tf_status_string(code)) > 0
