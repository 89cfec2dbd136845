"""Chains of dependent GEMVs on one stream (Section 4.6: operators are dispatched in sequence, each consuming
the output of the one before it).

Every kernel of the library lets its successor on the stream start early (programmatic dependent launch) and a
half-SM GEMV becomes resident beside its predecessor.  The successor may fetch weights at once but must not read
activations before the predecessor has completed.  These tests make the window as wide as it gets -- a long
first call, a second call whose activations ARE the first call's output, intermediates pre-filled with NaN on the
same stream -- for every launch plan of the GEMV, and check every result against the oracle applied to the bits
the previous call actually produced."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from paper_2606_11357_b200 import binding as tf
from paper_2606_11357_b200 import workloads as wl

pytestmark = pytest.mark.gpu

_WEIGHTS = {}


def weights(K, N, seed):
    """(problem with M = 16 activations, device blob), cached per shape: the 30 MB matrices take a moment to draw."""
    key = (K, N, seed)
    if key not in _WEIGHTS:
        p = wl.make_w4(16, K, N, seed=seed)
        _WEIGHTS[key] = (p, torch.from_numpy(gu.pack(p)).cuda())
    return _WEIGHTS[key]


def with_activations(problem, a_bits):
    """The same weights as `problem` with other activations (a shallow copy: the oracle reads, never writes)."""
    import copy
    q = copy.copy(problem)
    q.a_bf16 = a_bits
    q.M = a_bits.shape[0]
    return q


def plan_kind(M, K, N):
    p = tf.tf_gemv_plan(4, M, K, N)
    return "cluster" if p["cluster"] > 1 else ("whole" if p["full"] else "half")


# dims = layer widths d0 -> d1 -> d2 (-> d3); `plans` = the launch plan each call of the chain must take, so that
# a change of the planning heuristics cannot silently move a case to another code path
CHAINS = [
    ((4096, 14336, 4096), 1, ("half", "half")),
    ((4096, 14336, 4096), 2, ("half", "half")),
    ((4096, 14336, 4096), 4, ("whole", "whole")),
    ((4096, 14336, 4096), 8, ("whole", "whole")),
    ((4096, 4096, 1024), 1, ("half", "half")),
    ((4096, 4096, 1024), 8, ("whole", "whole")),
    ((4096, 14336, 4096, 1024), 1, ("half", "half", "half")),
    ((4096, 14336, 4096, 1024), 4, ("whole", "whole", "whole")),
    ((4096, 14336, 4096), 16, ("whole", "whole")),
    ((4096, 4096, 1024), 16, ("cluster", "cluster")),
    ((4096, 32768, 1024), 2, ("whole", "half")),            # a long integer-path range: whole SM, 16 warps, piece table
    ((1024, 32768, 1024), 2, ("half", "half")),            # two tokens with the piece table, then without
    ((384, 14336, 4096), 1, ("half", "half")),
]


@pytest.mark.parametrize("dims,M,plans", CHAINS, ids=[f"{'x'.join(map(str, d))}-M{m}" for d, m, _ in CHAINS])
def test_gemv_chain_consumes_previous_output(dims, M, plans):
    layers = [weights(dims[i], dims[i + 1], seed=2000 + i) for i in range(len(dims) - 1)]
    assert tuple(plan_kind(M, dims[i], dims[i + 1]) for i in range(len(layers))) == plans
    a0_bits = layers[0][0].a_bf16[:M].copy()
    a0 = gu.to_device_bf16(a0_bits)
    ys = [torch.empty((M, dims[i + 1]), dtype=torch.bfloat16, device="cuda") for i in range(len(layers))]
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, M, 4096, 4096), dtype=torch.uint8, device="cuda")
    for rep in range(4):                                   # an early read shows up intermittently
        for y in ys:
            y.fill_(float("nan"))                          # on the stream, right before the chain
        x = a0
        for (p, blob), y in zip(layers, ys):
            tf.tf_gemv_w4a16(blob, x, y, M, p.K, p.N, ws)
            x = y
        assert tf.tf_device_status(ws) == 0
        torch.cuda.synchronize()
        outs = [gu.bits_of(y) for y in ys]
        if rep == 0:
            first = outs
            x_bits = a0_bits
            for (p, _), out in zip(layers, outs):
                gu.check_against_oracle(with_activations(p, x_bits), out)
                x_bits = out
        else:                                              # deterministic: later repetitions must give the same bits
            for o, f in zip(outs, first):
                assert np.array_equal(o, f)


def test_gemm_then_half_sm_gemv_chain():
    """A whole-SM kernel (the GEMM) followed by two half-SM GEMVs that each consume the previous result."""
    M = 2
    (p1, b1), (p2, b2), (p3, b3) = weights(4096, 4096, 2100), weights(4096, 14336, 2101), weights(14336, 4096, 2102)
    a0_bits = p1.a_bf16[:M].copy()
    a0 = gu.to_device_bf16(a0_bits)
    y1 = torch.empty((M, 4096), dtype=torch.bfloat16, device="cuda")
    y2 = torch.empty((M, 14336), dtype=torch.bfloat16, device="cuda")
    y3 = torch.empty((M, 4096), dtype=torch.bfloat16, device="cuda")
    need = max(tf.tf_workspace_size(tf.TF_OP_GEMM_W4A16, M, 4096, 4096), tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, M, 4096, 4096))
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    for rep in range(3):
        for y in (y1, y2, y3):
            y.fill_(float("nan"))
        tf.tf_gemm_w4a16(b1, a0, y1, M, 4096, 4096, ws)
        tf.tf_gemv_w4a16(b2, y1, y2, M, 4096, 14336, ws)
        tf.tf_gemv_w4a16(b3, y2, y3, M, 14336, 4096, ws)
        assert tf.tf_device_status(ws) == 0
        torch.cuda.synchronize()
        o1, o2, o3 = gu.bits_of(y1), gu.bits_of(y2), gu.bits_of(y3)
        gu.check_against_oracle(with_activations(p1, a0_bits), o1)
        gu.check_against_oracle(with_activations(p2, o1), o2)
        gu.check_against_oracle(with_activations(p3, o2), o3)


def test_w8_integer_path_chain():
    """The W8A16 integer path (1 and 2 tokens) reads its activations in the consumer warps too."""
    M = 2
    p1 = wl.make_w8(M, 4096, 14336, seed=2200)
    p2 = wl.make_w8(M, 14336, 4096, seed=2201)
    assert tf.tf_gemv_plan(8, M, 4096, 14336)["i8"] == 1 and tf.tf_gemv_plan(8, M, 14336, 4096)["i8"] == 1
    b1, b2 = torch.from_numpy(gu.pack(p1)).cuda(), torch.from_numpy(gu.pack(p2)).cuda()
    a0 = gu.to_device_bf16(p1.a_bf16)
    y1 = torch.empty((M, 14336), dtype=torch.bfloat16, device="cuda")
    y2 = torch.empty((M, 4096), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMV_W8A16, M, 4096, 4096), dtype=torch.uint8, device="cuda")
    for rep in range(3):
        y1.fill_(float("nan"))
        y2.fill_(float("nan"))
        tf.tf_gemv_w8a16(b1, a0, y1, M, 4096, 14336, ws)
        tf.tf_gemv_w8a16(b2, y1, y2, M, 14336, 4096, ws)
        assert tf.tf_device_status(ws) == 0
        torch.cuda.synchronize()
        o1, o2 = gu.bits_of(y1), gu.bits_of(y2)
        gu.check_against_oracle(p1, o1)
        gu.check_against_oracle(with_activations(p2, o1), o2)
