"""The failure path of the kernels, exercised without faulting or hanging anything.

Every device-side wait of the GEMV and GEMM kernels is bounded.  tf_debug_inject shortens the bound to about a
millisecond and makes the packed-weight producer issue no copies ("a flag that nothing sets"), so the waits for
weights run out: the kernel must return by itself with TF_ERR_TIMEOUT in the status word, leave y untouched, free
its tensor memory, and leave the context usable -- the same call made normally right afterwards must pass parity."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TF_ERR_TIMEOUT = 8
LIMIT_KCYCLES = 2000            # about 1 ms at 1.9 GHz

# (kind, bits, M, K, N): the integer GEMV path, the floating-point GEMV path (whole SM), 9..16 tokens in global
# mode and in cluster mode, the int8 GEMV, and the GEMM with a narrow and a full token tile (one of them cut between CTAs)
CASES = [("gemv", 4, 1, 2048, 1024), ("gemv", 4, 5, 2048, 1024), ("gemv", 4, 16, 4096, 14336), ("gemv", 4, 16, 4096, 1024),
         ("gemv", 8, 2, 1024, 512), ("gemm", 4, 24, 1024, 512), ("gemm", 4, 300, 2048, 1096), ("gemm", 8, 64, 512, 256),
         # long integer-path ranges: whole SM with 16 consumer warps and the piece table (4-bit), with 8 warps (int8)
         ("gemv", 4, 1, 4096, 32768), ("gemv", 8, 2, 4096, 14336)]


@pytest.fixture(autouse=True)
def _always_restore_normal_operation():
    yield
    tf.tf_debug_inject(0, False)


@pytest.mark.parametrize("kind,bits,M,K,N", CASES)
def test_bounded_wait_runs_out_and_the_library_recovers(kind, bits, M, K, N):
    p = wl.make_w4(M, K, N, seed=3000 + M) if bits == 4 else wl.make_w8(M, K, N, seed=3000 + M)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    a = gu.to_device_bf16(p.a_bf16)
    y = torch.full((M, N), -3.0, dtype=torch.bfloat16, device="cuda")
    op = {("gemv", 4): tf.TF_OP_GEMV_W4A16, ("gemv", 8): tf.TF_OP_GEMV_W8A16,
          ("gemm", 4): tf.TF_OP_GEMM_W4A16, ("gemm", 8): tf.TF_OP_GEMM_W8A16}[(kind, bits)]
    ws = torch.zeros(tf.tf_workspace_size(op, M, K, N), dtype=torch.uint8, device="cuda")
    fn = getattr(tf, f"tf_{kind}_w{bits}a16")

    tf.tf_debug_inject(LIMIT_KCYCLES, True)
    fn(blob, a, y, M, K, N, ws)                                   # returns at once; the kernel gives up by itself
    assert tf.tf_device_status(ws) == TF_ERR_TIMEOUT             # synchronises: so the kernel did return
    detail = int(ws[4:8].view(torch.int32).item())
    assert detail != 0                                            # which wait gave up
    assert bool((y == -3.0).all()), "y was written although no weights ever arrived"
    tf.tf_debug_inject(0, False)

    ws.zero_()                                                    # the status word is sticky until the caller clears it
    for _ in range(2):                                            # tensor memory was freed, barriers and rings start afresh
        fn(blob, a, y, M, K, N, ws)
    assert tf.tf_device_status(ws) == 0
    gu.check_against_oracle(p, gu.bits_of(y))


def test_short_limit_alone_changes_nothing():
    """With the producer at work a millisecond is ample: the shortened limit by itself must not trip any wait."""
    p = wl.make_w4(4, 4096, 4096, seed=3100)
    blob = torch.from_numpy(gu.pack(p)).cuda()
    a = gu.to_device_bf16(p.a_bf16)
    y = torch.empty((4, 4096), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, 4, 4096, 4096), dtype=torch.uint8, device="cuda")
    tf.tf_debug_inject(LIMIT_KCYCLES, False)
    tf.tf_gemv_w4a16(blob, a, y, 4, 4096, 4096, ws)
    assert tf.tf_device_status(ws) == 0
    gu.check_against_oracle(p, gu.bits_of(y))


def test_debug_inject_rejects_out_of_range():
    assert tf.lib().tf_debug_inject(1 << 24, 0) == 2
