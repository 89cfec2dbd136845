"""Shared helpers for the tests: tolerance rule, tiny independent encoders, golden readers."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

# Acceptance rule for every output element (written here once, used by every parity test):
#     |y - y_ref| <= 4e-3 * sum_k |a_k * w_k| + 1e-5
REL_TOL = 4e-3
ABS_TOL = 1e-5


def tolerance(bound):
    return REL_TOL * np.asarray(bound, dtype=np.float64) + ABS_TOL


def error_ratio(y, y_ref, bound):
    """max over elements of |y - y_ref| / tolerance; parity holds iff <= 1."""
    return float(np.max(np.abs(np.asarray(y, np.float64) - y_ref) / tolerance(bound)))


def bf16_bits_to_f64(bits):
    """Test-side bf16 decoder (kept separate from the oracle's and the library's)."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) * np.uint32(65536)
    return b.view(np.float32).astype(np.float64)


def loop_pack_awq(codes):
    """Scalar-loop AWQ encoder written from the format rule; independent of workloads/oracle."""
    order = [0, 2, 4, 6, 1, 3, 5, 7]
    rows, cols = len(codes), len(codes[0])
    out = np.zeros((rows, cols // 8), dtype=np.uint32)
    for r in range(rows):
        for j in range(cols // 8):
            word = 0
            for i in range(8):
                word |= int(codes[r][8 * j + order[i]]) << (4 * i)
            out[r, j] = word
    return out


def read_golden_words():
    cases = []
    with open(os.path.join(GOLDEN, "awq_words.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if not line:
                continue
            parts = line.split()
            cases.append(([int(p) for p in parts[:8]], int(parts[8], 16)))
    return cases


def read_golden_dequant():
    cases = []
    with open(os.path.join(GOLDEN, "dequant_cases.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if not line:
                continue
            kind, q, z, s, a, w, aw = line.split()
            cases.append((kind, int(q), int(z), float(s), float(a), float(w), float(aw)))
    return cases


# ----------------------------------------------------------------------------------------------
# Host-side reader of the packed blob, written from the layout description in include/tilefuse.h
# and csrc/layout.h (test-only; the library's own decoders are the GPU kernels).
# ----------------------------------------------------------------------------------------------
HEADER_BYTES, TILE_K, TILE_N = 256, 128, 64
W4_TILE, W8_TILE = 4256, 8320


def read_header(blob):
    h = np.frombuffer(blob[:48].tobytes(), dtype=np.uint32)
    names = ["magic", "version", "bits", "K", "N", "group_size", "n_padded", "strips", "ktiles", "tile_bytes"]
    out = {n: int(h[i]) for i, n in enumerate(names)}
    tail = np.frombuffer(blob[40:56].tobytes(), dtype=np.uint64)
    out["tiles_offset"], out["total_bytes"] = int(tail[0]), int(tail[1])
    return out


def read_blob(blob, bits, K, N, group_size=128):
    """Decode a blob on the host -> (q [K, Np], z [rows, Np] or None, s_bits [rows, Np]): one metadata row per tile
    (group sizes that are multiples of 128) or per group (4-bit group sizes 64 and 32: G = 128 / group_size rows per
    tile, stored as G scale blocks followed by G zero blocks)."""
    strips, ktiles = (N + TILE_N - 1) // TILE_N, K // TILE_K
    G = 1 if group_size >= TILE_K else TILE_K // group_size
    wbytes = 4096 if bits == 4 else 8192
    tile_bytes = (4096 + 160 * G) if bits == 4 else W8_TILE
    tiles = blob[HEADER_BYTES:HEADER_BYTES + strips * ktiles * tile_bytes].reshape(strips, ktiles, tile_bytes)
    Np = strips * TILE_N
    q = np.zeros((K, Np), dtype=np.int16)
    kb, lane, w = np.meshgrid(np.arange(8), np.arange(32), np.arange(4), indexing="ij")
    g, t = lane >> 2, lane & 3
    if bits == 4:
        words = np.ascontiguousarray(tiles[:, :, :wbytes]).view(np.uint32).reshape(strips, ktiles, 8, 32, 4)
        for p in range(8):
            reg, el = p & 3, p >> 2
            dk = 16 * kb + 4 * t + 2 * (reg >> 1) + el
            dn = 16 * w + g + 8 * (reg & 1)
            vals = ((words >> np.uint32(4 * p)) & np.uint32(0xF)).astype(np.int16)
            for S in range(strips):
                for T in range(ktiles):
                    q[T * TILE_K + dk, S * TILE_N + dn] = vals[S, T]
    else:
        raw = np.ascontiguousarray(tiles[:, :, :wbytes]).view(np.int8).reshape(strips, ktiles, 8, 2, 32, 4, 4)
        for r in range(2):
            for b in range(4):
                reg, el = 2 * r + (b >> 1), b & 1
                dk = 16 * kb + 4 * t + 2 * (reg >> 1) + el
                dn = 16 * w + g + 8 * (reg & 1)
                for S in range(strips):
                    for T in range(ktiles):
                        q[T * TILE_K + dk, S * TILE_N + dn] = raw[S, T, kb, w >> 1, lane, 2 * (w & 1) + r, b]
    s = np.zeros((ktiles * G, Np), dtype=np.uint16)
    z = np.zeros((ktiles * G, Np), dtype=np.int16) if bits == 4 else None
    gg, ww, hh = np.meshgrid(np.arange(8), np.arange(4), np.arange(2), indexing="ij")
    ncol = 16 * ww + gg + 8 * hh
    for gr in range(G):
        sc = np.ascontiguousarray(tiles[:, :, wbytes + 128 * gr:wbytes + 128 * (gr + 1)]).view(np.uint16).reshape(strips, ktiles, 8, 4, 2)
        if bits == 4:
            z0 = wbytes + 128 * G + 32 * gr
            zw = np.ascontiguousarray(tiles[:, :, z0:z0 + 32]).view(np.uint32).reshape(strips, ktiles, 8)
        for S in range(strips):
            for T in range(ktiles):
                s[T * G + gr, S * TILE_N + ncol] = sc[S, T]
                if bits == 4:
                    for i in range(8):
                        z[T * G + gr, S * TILE_N + 16 * (i & 3) + np.arange(8) + 8 * (i >> 2)] = \
                            (zw[S, T] >> np.uint32(4 * i)) & np.uint32(0xF)
    return q, z, s
