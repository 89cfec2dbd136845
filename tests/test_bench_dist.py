"""The multi-rank plumbing of bench.py on CPU: two gloo ranks, max / sum over ranks, byte accounting."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, w = bench.init_dist("gloo")
    assert (r, w) == (rank, world)
    bench.barrier()
    mx = bench.max_over_ranks(10.0 + rank)
    sm = bench.sum_over_ranks(1.5 * (rank + 1))
    out[rank] = (mx, sm)
    dist.destroy_process_group()


def test_two_ranks_gloo():
    world, port = 2, 29731
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1] == (11.0, 4.5)


def _gather_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    bench.init_dist("gloo")
    from paper_2606_11357_b200 import binding as tf
    N, M = 200, 3                                           # four strips, the last one ragged: shards of 128 and 72 columns
    counts = [tf.tf_shard_columns(N, r, world)[1] for r in range(world)]
    begin = tf.tf_shard_columns(N, rank, world)[0]
    full = torch.arange(M * N, dtype=torch.float32).reshape(M, N)
    y = bench.gather_columns(full[:, begin:begin + counts[rank]].contiguous(), counts)
    out[rank] = (counts, bool(torch.equal(y, full)))
    dist.destroy_process_group()


def test_column_shards_gather_back_on_two_gloo_ranks():
    """The one exchange of the column-parallel arrangement: ragged column shards all-gathered into the full result."""
    world, port = 2, 29733
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_gather_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1] == ([128, 72], True)


def test_single_process_passthrough():
    assert bench.max_over_ranks(3.25) == 3.25 and bench.sum_over_ranks(2.0) == 2.0


def test_algorithmic_bytes():
    # weights + fp16 scales + 4-bit zeros + activations + output, each once
    assert bench.gemv_algorithmic_bytes(4, 1, 4096, 4096) == 8732672
    assert bench.gemv_algorithmic_bytes(4, 1, 4096, 14336) == 30543872
    assert bench.gemv_algorithmic_bytes(8, 1, 4096, 14336) == 59674624
    assert bench.gemv_algorithmic_bytes(4, 1, 4096, 32768) == 69804032


def test_peaks_fallback_and_reference_arm(monkeypatch, capsys):
    peaks, kind = bench.load_peaks()
    assert kind in ("measured", "fallback") and peaks["hbm_gbs"] > 1000
    monkeypatch.setenv("RANK", "1")
    assert bench.main(["--impl", "reference", "--steps", "1", "--warmup", "0"]) == 0   # non-zero ranks do no work
    assert capsys.readouterr().out == ""
