"""tf_gemv_w4a16_static: the GEMV for callers that cannot allocate or pass device scratch.

Collected last on purpose (file name), so a run that stops at the first failure has already run everything
else.  The static entry point must give exactly what tf_gemv_w4a16 gives with a caller workspace, on two
calls in a row (the second reuses the library's fixed scratch array with whatever the first left in it).
"""
import numpy as np
import pytest
import torch

from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import workloads as wl
import gpu_util as gu

pytestmark = pytest.mark.gpu


def _both_ways(problem, blob):
    M, K, N = problem.M, problem.K, problem.N
    a = gu.to_device_bf16(problem.a_bf16)
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, M, K, N), dtype=torch.uint8, device="cuda")
    y_ref = torch.full((M, N), -7.0, dtype=torch.bfloat16, device="cuda")
    tf.tf_gemv_w4a16(blob, a, y_ref, M, K, N, ws)
    assert tf.tf_device_status(ws) == 0
    y_new = torch.full((M, N), -9.0, dtype=torch.bfloat16, device="cuda")
    tf.tf_gemv_w4a16_static(blob, a, y_new, M, K, N)
    torch.cuda.synchronize()
    return gu.bits_of(y_ref), gu.bits_of(y_new)


def test_static_scratch_gemv_matches_workspace_gemv_twice():
    # shape with strips cut between CTAs (so counters and partial sums in the scratch are really used)
    p1 = wl.make_w4(4, 4096, 4096, seed=101)
    blob1 = torch.from_numpy(gu.pack(p1)).cuda()
    ref1, new1 = _both_ways(p1, blob1)
    assert np.array_equal(ref1, new1)
    gu.check_against_oracle(p1, new1)
    # second call right away: other activations, other shape, same scratch array
    p2 = wl.make_w4(16, 1024, 1000, seed=102)
    blob2 = torch.from_numpy(gu.pack(p2)).cuda()
    ref2, new2 = _both_ways(p2, blob2)
    assert np.array_equal(ref2, new2)
    gu.check_against_oracle(p2, new2)
    # and the first problem again, to see that nothing stale from the second call leaks in
    ref3, new3 = _both_ways(p1, blob1)
    assert np.array_equal(ref3, ref1) and np.array_equal(new3, ref1)


def test_static_scratch_gemv_rejects_out_of_range():
    L = tf.lib()
    import ctypes
    ok = ctypes.c_void_p(0x1000)
    assert L.tf_gemv_w4a16_static(None, ok, ok, 1, 128, 8, None) == 1          # TF_ERR_NULL
    assert L.tf_gemv_w4a16_static(ok, ok, ok, 17, 128, 8, None) == 2           # M beyond the maximum
    assert L.tf_gemv_w4a16_static(ok, ok, ok, 1, 32768 + 128, 8, None) == 2    # K beyond the maximum
    assert L.tf_gemv_w4a16_static(ok, ok, ok, 1, 128, 32768 + 8, None) == 2    # N beyond the maximum
    assert L.tf_gemv_w4a16_static(ok, ctypes.c_void_p(0x1008), ok, 1, 128, 8, None) == 3


def test_static_scratch_gemv_chain_consumes_previous_output():
    """Two static calls back to back where the second multiplies what the first writes (no host synchronisation in
    between, intermediate pre-filled with NaN on the stream): same bits as the workspace path, within the
    oracle's tolerance."""
    import copy
    M = 4
    p1 = wl.make_w4(M, 4096, 14336, seed=103)
    p2 = wl.make_w4(M, 14336, 4096, seed=104)
    b1, b2 = torch.from_numpy(gu.pack(p1)).cuda(), torch.from_numpy(gu.pack(p2)).cuda()
    a0 = gu.to_device_bf16(p1.a_bf16)
    y1 = torch.empty((M, 14336), dtype=torch.bfloat16, device="cuda")
    y2 = torch.empty((M, 4096), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, M, 4096, 4096), dtype=torch.uint8, device="cuda")
    results = []
    for static in (False, True, True):
        y1.fill_(float("nan"))
        y2.fill_(float("nan"))
        if static:
            tf.tf_gemv_w4a16_static(b1, a0, y1, M, 4096, 14336)
            tf.tf_gemv_w4a16_static(b2, y1, y2, M, 14336, 4096)
        else:
            tf.tf_gemv_w4a16(b1, a0, y1, M, 4096, 14336, ws)
            tf.tf_gemv_w4a16(b2, y1, y2, M, 14336, 4096, ws)
        torch.cuda.synchronize()
        results.append((gu.bits_of(y1), gu.bits_of(y2)))
    assert tf.tf_device_status(ws) == 0
    for o1, o2 in results[1:]:
        assert np.array_equal(o1, results[0][0]) and np.array_equal(o2, results[0][1])
    gu.check_against_oracle(p1, results[1][0])
    q2 = copy.copy(p2)
    q2.a_bf16 = results[1][0]
    gu.check_against_oracle(q2, results[1][1])


def test_static_scratch_status_reports_a_blob_mismatch():
    """A blob that does not match the arguments is detected on the device: y stays untouched and the status reader of
    the static entry point says so (a workspace call reports the same through tf_device_status)."""
    p = wl.make_w4(2, 1024, 512, seed=105)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    a = gu.to_device_bf16(p.a_bf16)
    y = torch.full((2, 256), -5.0, dtype=torch.bfloat16, device="cuda")
    tf.tf_gemv_w4a16_static(blob, a, y, 2, 1024, 256)              # N does not match the blob's header
    assert tf.tf_gemv_w4a16_static_status() == 4                   # TF_ERR_BLOB
    assert bool((y == -5.0).all())
    y2 = torch.empty((2, 512), dtype=torch.bfloat16, device="cuda")
    tf.tf_gemv_w4a16_static(blob, a, y2, 2, 1024, 512)             # the next call clears the word
    assert tf.tf_gemv_w4a16_static_status() == 0
    gu.check_against_oracle(p, gu.bits_of(y2))
