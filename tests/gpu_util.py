"""Helpers for the GPU parity tests: move a Problem to the device, call the C ABI, compare."""
import numpy as np
import torch

from oracle import tilefuse_oracle as orc
from paper_2606_11357_b200 import binding as tf
from helpers import bf16_bits_to_f64, error_ratio

CANARY = 0x7FC1            # a bf16 NaN pattern no kernel produces from finite inputs


def pack(problem) -> np.ndarray:
    if problem.bits == 4:
        return tf.tf_pack_awq(problem.qweight, problem.scales_f16, problem.qzeros, problem.K, problem.N,
                              problem.group_size)
    return tf.tf_pack_w8(problem.w_i8, problem.scales_f16, problem.K, problem.N, problem.group_size)


def to_device_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def run(problem, kind: str, blob_dev=None, a_bits=None):
    """Call tf_{kind}_w{bits}a16 through the binding with guard bands around y; returns y bits [M, N]."""
    M, K, N = problem.M, problem.K, problem.N
    if blob_dev is None:
        blob_dev = torch.from_numpy(pack(problem)).cuda()
    a = to_device_bf16(problem.a_bf16 if a_bits is None else a_bits)
    M = a.shape[0]
    guard = 512
    ybuf = torch.full((guard + M * N + guard,), CANARY, dtype=torch.int16, device="cuda")
    # keep the payload 16-byte aligned inside the guarded buffer
    y = ybuf[guard:guard + M * N].view(torch.bfloat16).view(M, N)
    op = {("gemv", 4): tf.TF_OP_GEMV_W4A16, ("gemv", 8): tf.TF_OP_GEMV_W8A16,
          ("gemm", 4): tf.TF_OP_GEMM_W4A16, ("gemm", 8): tf.TF_OP_GEMM_W8A16}[(kind, problem.bits)]
    ws_bytes = max(tf.tf_workspace_size(op, M, K, N), 256)
    ws = torch.zeros(ws_bytes + 1024, dtype=torch.uint8, device="cuda")
    ws[ws_bytes:] = 0xA5
    fn = getattr(tf, f"tf_{kind}_w{problem.bits}a16")
    fn(blob_dev, a, y, M, K, N, ws[:ws_bytes])
    status = tf.tf_device_status(ws)
    assert status == 0, f"device status {status}"
    torch.cuda.synchronize()
    raw = ybuf.cpu().numpy().view(np.uint16)
    assert np.all(raw[:guard] == CANARY) and np.all(raw[guard + M * N:] == CANARY), "write outside y"
    assert bool((ws[ws_bytes:] == 0xA5).all()), "write outside the workspace"
    return raw[guard:guard + M * N].reshape(M, N).copy()


def check_against_oracle(problem, y_bits, columns=None):
    """Element-by-element acceptance |y - y_ref| <= 4e-3 * B + 1e-5; returns the max ratio."""
    y_ref, bound = orc.solve(problem, columns=columns)
    y = bf16_bits_to_f64(y_bits if columns is None else y_bits[:, columns])
    assert np.all(np.isfinite(y)), "non-finite output (a canary or NaN reached y)"
    ratio = error_ratio(y, y_ref, bound)
    assert ratio <= 1.0, f"{problem.name}: max |err|/tol = {ratio:.3f}"
    return ratio
