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
