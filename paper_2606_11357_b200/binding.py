"""Thin ctypes binding over libtilefuse.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/tilefuse.h).  Host
arrays are numpy, device buffers are torch CUDA tensors (torch is used for device memory and
streams, nothing else).  There is no fallback: if the library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libtilefuse.so")
_lib = None

TF_OK = 0
TF_OP_GEMV_W4A16, TF_OP_GEMV_W8A16, TF_OP_GEMM_W4A16, TF_OP_GEMM_W8A16 = 0, 1, 2, 3
STATUS_NAMES = {0: "TF_OK", 1: "TF_ERR_NULL", 2: "TF_ERR_SHAPE", 3: "TF_ERR_ALIGN", 4: "TF_ERR_BLOB",
                5: "TF_ERR_WORKSPACE", 6: "TF_ERR_ARCH", 7: "TF_ERR_CUDA", 8: "TF_ERR_TIMEOUT"}

EXPORTS = ("tf_packed_size", "tf_pack_awq", "tf_pack_w8", "tf_pack_concat", "tf_unpack_w4", "tf_unpack_w8",
           "tf_gemv_w4a16", "tf_gemv_w8a16", "tf_gemm_w4a16", "tf_gemm_w8a16",
           "tf_workspace_size", "tf_device_status", "tf_status_string", "tf_version", "tf_gemv_w4a16_static",
           "tf_dequant_bf16", "tf_gemv_awq_raw", "tf_gemv_awq_raw_workspace_size", "tf_gemv_plan", "tf_debug_inject", "tf_gemv_w4a16_static_status",
           "tf_gemv_w4a16_grouped", "tf_gemm_w4a16_grouped", "tf_shard_columns", "tf_pack_shard",
           "tf_pack_awq_device", "tf_gemm_awq_raw", "tf_gemm_awq_raw_workspace_size")


class TileFuseError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        msg = lib().tf_status_string(status).decode() if _lib is not None else ""
        super().__init__(f"{call} -> {STATUS_NAMES.get(status, status)}: {msg}")


def lib() -> ctypes.CDLL:
    """Load the C-ABI library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2606_11357_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(_LIB_PATH)
        c_int, c_size, vp = ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p
        L.tf_packed_size.restype, L.tf_packed_size.argtypes = c_size, [c_int] * 4
        L.tf_pack_awq.restype, L.tf_pack_awq.argtypes = c_int, [vp, vp, vp, c_int, c_int, c_int, vp, c_size]
        L.tf_pack_w8.restype, L.tf_pack_w8.argtypes = c_int, [vp, vp, c_int, c_int, c_int, vp, c_size]
        L.tf_pack_concat.restype, L.tf_pack_concat.argtypes = c_int, [vp, c_int, vp, c_size]
        L.tf_shard_columns.restype, L.tf_shard_columns.argtypes = c_int, [c_int, c_int, c_int, vp, vp]
        L.tf_pack_shard.restype, L.tf_pack_shard.argtypes = c_int, [vp, c_int, c_int, vp, c_size]
        L.tf_unpack_w4.restype, L.tf_unpack_w4.argtypes = c_int, [vp, vp, vp, vp, c_int, c_int, c_int, vp]
        L.tf_unpack_w8.restype, L.tf_unpack_w8.argtypes = c_int, [vp, vp, vp, c_int, c_int, c_int, vp]
        for name in ("tf_gemv_w4a16", "tf_gemv_w8a16", "tf_gemm_w4a16", "tf_gemm_w8a16"):
            fn = getattr(L, name)
            fn.restype, fn.argtypes = c_int, [vp, vp, vp, c_int, c_int, c_int, vp, c_size, vp]
        for name in ("tf_gemv_w4a16_grouped", "tf_gemm_w4a16_grouped"):
            fn = getattr(L, name)
            fn.restype, fn.argtypes = c_int, [vp, vp, vp, c_int, c_int, c_int, c_int, vp, c_size, vp]
        L.tf_gemv_w4a16_static.restype = c_int
        L.tf_gemv_w4a16_static.argtypes = [vp, vp, vp, c_int, c_int, c_int, vp]
        L.tf_workspace_size.restype, L.tf_workspace_size.argtypes = c_size, [c_int] * 4
        L.tf_gemv_plan.restype, L.tf_gemv_plan.argtypes = c_int, [c_int] * 5 + [vp]
        L.tf_debug_inject.restype, L.tf_debug_inject.argtypes = c_int, [ctypes.c_uint, c_int]
        L.tf_gemv_w4a16_static_status.restype, L.tf_gemv_w4a16_static_status.argtypes = c_int, [vp]
        L.tf_dequant_bf16.restype, L.tf_dequant_bf16.argtypes = c_int, [vp, vp, c_int, c_int, c_int, vp]
        L.tf_gemv_awq_raw.restype = c_int
        L.tf_gemv_awq_raw.argtypes = [vp, vp, vp, vp, vp, c_int, c_int, c_int, c_int, vp, c_size, vp]
        L.tf_gemv_awq_raw_workspace_size.restype, L.tf_gemv_awq_raw_workspace_size.argtypes = c_size, [c_int] * 4
        L.tf_gemm_awq_raw.restype = c_int
        L.tf_gemm_awq_raw.argtypes = [vp, vp, vp, vp, vp, c_int, c_int, c_int, c_int, vp, c_size, vp]
        L.tf_gemm_awq_raw_workspace_size.restype, L.tf_gemm_awq_raw_workspace_size.argtypes = c_size, [c_int] * 4
        L.tf_pack_awq_device.restype = c_int
        L.tf_pack_awq_device.argtypes = [vp, vp, vp, c_int, c_int, c_int, vp, c_size, vp]
        L.tf_device_status.restype, L.tf_device_status.argtypes = c_int, [vp, vp]
        L.tf_status_string.restype, L.tf_status_string.argtypes = ctypes.c_char_p, [c_int]
        L.tf_version.restype, L.tf_version.argtypes = c_int, []
        _lib = L
    return _lib


def _check(call: str, status: int) -> None:
    if status != TF_OK:
        raise TileFuseError(call, status)


def _host(arr: np.ndarray, dtype) -> np.ndarray:
    out = np.ascontiguousarray(arr)
    if out.dtype != np.dtype(dtype):
        raise TypeError(f"expected {np.dtype(dtype)}, got {out.dtype}")
    return out


def _dev(t):
    """Raw device address of a torch CUDA tensor (or None)."""
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device buffers must be contiguous CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


# ---------------------------------------------------------------------------- host calls
def tf_version() -> int:
    return lib().tf_version()


def tf_packed_size(bits: int, K: int, N: int, group_size: int = 128) -> int:
    return lib().tf_packed_size(bits, K, N, group_size)


def tf_pack_awq(qweight, scales_f16, qzeros, K: int, N: int, group_size: int = 128, out=None) -> np.ndarray:
    """AWQ arrays (numpy, host) -> packed blob (numpy uint8, host)."""
    qweight, qzeros = _host(qweight, np.uint32), _host(qzeros, np.uint32)
    scales = _host(scales_f16, np.float16)
    size = tf_packed_size(4, K, N, group_size)
    if out is None:
        out = np.empty(size, dtype=np.uint8)
    _check("tf_pack_awq", lib().tf_pack_awq(qweight.ctypes.data, scales.ctypes.data, qzeros.ctypes.data,
                                            K, N, group_size, out.ctypes.data, out.nbytes))
    return out


def tf_pack_w8(w_i8, scales_f16, K: int, N: int, group_size: int = 128, out=None) -> np.ndarray:
    w, scales = _host(w_i8, np.int8), _host(scales_f16, np.float16)
    size = tf_packed_size(8, K, N, group_size)
    if out is None:
        out = np.empty(size, dtype=np.uint8)
    _check("tf_pack_w8", lib().tf_pack_w8(w.ctypes.data, scales.ctypes.data, K, N, group_size,
                                          out.ctypes.data, out.nbytes))
    return out


def tf_pack_concat(parts, out=None) -> np.ndarray:
    """parts: packed blobs (uint8 numpy arrays) with the same bits, K and group size -> blob of [W_0 | W_1 | ...]."""
    parts = [_host(p, np.uint8) for p in parts]
    if out is None:
        payload = sum(int(p.nbytes) - 256 for p in parts)
        out = np.empty(256 + max(payload, 0), dtype=np.uint8)
    ptrs = (ctypes.c_void_p * max(len(parts), 1))(*[p.ctypes.data for p in parts])
    _check("tf_pack_concat", lib().tf_pack_concat(ctypes.cast(ptrs, ctypes.c_void_p), len(parts), out.ctypes.data, out.nbytes))
    return out


def tf_shard_columns(N: int, part: int, parts: int):
    """(n_begin, n_count) of column shard `part` of `parts` (whole strips of 64 columns)."""
    b, c = ctypes.c_int(0), ctypes.c_int(0)
    _check("tf_shard_columns", lib().tf_shard_columns(N, part, parts, ctypes.byref(b), ctypes.byref(c)))
    return b.value, c.value


def tf_pack_shard(packed, part: int, parts: int, out=None) -> np.ndarray:
    """The blob of column shard `part` of `parts`, cut out of the blob of the whole matrix (host arrays)."""
    packed = _host(packed, np.uint8)
    hdr = np.frombuffer(packed[:48].tobytes(), dtype=np.uint32)
    bits, K, N, g = int(hdr[2]), int(hdr[3]), int(hdr[4]), int(hdr[5])
    _, count = tf_shard_columns(N, part, parts)
    if out is None:
        out = np.empty(tf_packed_size(bits, K, count, g), dtype=np.uint8)
    _check("tf_pack_shard", lib().tf_pack_shard(packed.ctypes.data, part, parts, out.ctypes.data, out.nbytes))
    return out


def tf_gemv_plan(bits: int, M: int, K: int, N: int, sm_count: int = 0) -> dict:
    """Launch geometry the GEMV would choose (sm_count <= 0: the current device)."""
    out = (ctypes.c_int * 8)()
    _check("tf_gemv_plan", lib().tf_gemv_plan(bits, M, K, N, sm_count, ctypes.cast(out, ctypes.c_void_p)))
    names = ("grid", "threads", "consumers", "stages", "full", "i8", "cluster", "nclusters")
    return dict(zip(names, (int(v) for v in out)))


def tf_workspace_size(op: int, M: int, K: int, N: int) -> int:
    return lib().tf_workspace_size(op, M, K, N)


# -------------------------------------------------------------------------- device calls
def tf_unpack_w4(packed, q, z, s_f16, K: int, N: int, group_size: int = 128, stream=None) -> None:
    """packed: uint8 CUDA tensor; q uint8 [K,N], z uint8 [K/g,N], s_f16 float16 [K/g,N] (any may be None)."""
    _check("tf_unpack_w4", lib().tf_unpack_w4(_dev(packed), _dev(q), _dev(z), _dev(s_f16), K, N, group_size,
                                              _stream(stream)))


def tf_dequant_bf16(packed, w_bf16, bits: int, K: int, N: int, stream=None) -> None:
    """packed: uint8 CUDA tensor; w_bf16: bfloat16 CUDA tensor [K, N] that receives the dequantized matrix."""
    _check("tf_dequant_bf16", lib().tf_dequant_bf16(_dev(packed), _dev(w_bf16), bits, K, N, _stream(stream)))


def tf_gemv_awq_raw_workspace_size(M: int, K: int, N: int, group_size: int = 128) -> int:
    return int(lib().tf_gemv_awq_raw_workspace_size(M, K, N, group_size))


def tf_gemv_awq_raw(qweight, scales_f16, qzeros, a, y, M: int, K: int, N: int, group_size: int, workspace,
                    stream=None) -> None:
    """The fused GEMV on the AWQ arrays themselves (CUDA tensors: int32 [K, N/8], int16/float16 [K/g, N],
    int32 [K/g, N/8]); a, y as for tf_gemv_w4a16; workspace: uint8 CUDA tensor."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("tf_gemv_awq_raw", lib().tf_gemv_awq_raw(_dev(qweight), _dev(scales_f16), _dev(qzeros), _dev(a), _dev(y),
                                                    M, K, N, group_size, _dev(workspace), ws_bytes, _stream(stream)))


def tf_pack_awq_device(qweight, scales_f16, qzeros, K: int, N: int, group_size: int, out, stream=None) -> None:
    """The AWQ arrays (CUDA tensors) -> the packed blob (uint8 CUDA tensor of at least tf_packed_size bytes)."""
    _check("tf_pack_awq_device", lib().tf_pack_awq_device(_dev(qweight), _dev(scales_f16), _dev(qzeros), K, N, group_size,
                                                          _dev(out), out.numel() * out.element_size(), _stream(stream)))


def tf_gemm_awq_raw_workspace_size(M: int, K: int, N: int, group_size: int = 128) -> int:
    return int(lib().tf_gemm_awq_raw_workspace_size(M, K, N, group_size))


def tf_gemm_awq_raw(qweight, scales_f16, qzeros, a, y, M: int, K: int, N: int, group_size: int, workspace, stream=None) -> None:
    """The fused GEMM on the AWQ arrays themselves (re-tiled into the workspace on every call, then multiplied)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("tf_gemm_awq_raw", lib().tf_gemm_awq_raw(_dev(qweight), _dev(scales_f16), _dev(qzeros), _dev(a), _dev(y),
                                                    M, K, N, group_size, _dev(workspace), ws_bytes, _stream(stream)))


def tf_unpack_w8(packed, q, s_f16, K: int, N: int, group_size: int = 128, stream=None) -> None:
    _check("tf_unpack_w8", lib().tf_unpack_w8(_dev(packed), _dev(q), _dev(s_f16), K, N, group_size,
                                              _stream(stream)))


def _linear(name, packed, a, y, M, K, N, workspace, stream):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(name, getattr(lib(), name)(_dev(packed), _dev(a), _dev(y), M, K, N, _dev(workspace), ws_bytes,
                                      _stream(stream)))


def tf_gemv_w4a16(packed, a, y, M, K, N, workspace, stream=None) -> None:
    """a: bfloat16 [M,K], y: bfloat16 [M,N] CUDA tensors; asynchronous on the stream."""
    _linear("tf_gemv_w4a16", packed, a, y, M, K, N, workspace, stream)


def _linear_grouped(name, packed, a, y, M, K, N, group_size, workspace, stream):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(name, getattr(lib(), name)(_dev(packed), _dev(a), _dev(y), M, K, N, group_size, _dev(workspace), ws_bytes,
                                      _stream(stream)))


def tf_gemv_w4a16_grouped(packed, a, y, M, K, N, group_size, workspace, stream=None) -> None:
    """tf_gemv_w4a16 for a blob packed with `group_size` (32, 64 or a multiple of 128)."""
    _linear_grouped("tf_gemv_w4a16_grouped", packed, a, y, M, K, N, group_size, workspace, stream)


def tf_gemm_w4a16_grouped(packed, a, y, M, K, N, group_size, workspace, stream=None) -> None:
    _linear_grouped("tf_gemm_w4a16_grouped", packed, a, y, M, K, N, group_size, workspace, stream)


def tf_gemv_w4a16_static(packed, a, y, M, K, N, stream=None) -> None:
    """tf_gemv_w4a16 for callers that cannot provide a workspace: scratch is a fixed array inside the library.
    Calls share that array, so do not let two of them overlap on the GPU."""
    _check("tf_gemv_w4a16_static", lib().tf_gemv_w4a16_static(_dev(packed), _dev(a), _dev(y), M, K, N, _stream(stream)))


def tf_gemv_w4a16_static_status(stream=None) -> int:
    return lib().tf_gemv_w4a16_static_status(_stream(stream))


def tf_debug_inject(wait_limit_kcycles: int = 0, drop_weight_copies: bool = False) -> None:
    """Failure-path test hook: shorten the device-side wait limit and/or make the weight producer issue nothing,
    for every launch that follows; tf_debug_inject() restores normal operation."""
    _check("tf_debug_inject", lib().tf_debug_inject(wait_limit_kcycles, 1 if drop_weight_copies else 0))


def tf_gemv_w8a16(packed, a, y, M, K, N, workspace, stream=None) -> None:
    _linear("tf_gemv_w8a16", packed, a, y, M, K, N, workspace, stream)


def tf_gemm_w4a16(packed, a, y, M, K, N, workspace, stream=None) -> None:
    _linear("tf_gemm_w4a16", packed, a, y, M, K, N, workspace, stream)


def tf_gemm_w8a16(packed, a, y, M, K, N, workspace, stream=None) -> None:
    _linear("tf_gemm_w8a16", packed, a, y, M, K, N, workspace, stream)


def tf_device_status(workspace, stream=None) -> int:
    return lib().tf_device_status(_dev(workspace), _stream(stream))
