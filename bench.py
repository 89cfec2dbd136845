#!/usr/bin/env python
"""Benchmark of the fused W4A16 linear layer on B200 (one process per GPU).

A *step* is one decode pass over the four Llama-3-8B-shaped linear layers (K x N = 4096x4096,
4096x1024, 4096x14336, 14336x4096) at M = 1, 4 and 16 tokens: twelve tf_gemv_w4a16 calls, each on
its own device copy of the packed weights.  Two full sets of copies alternate between steps, so the
weights of a call (432 MB in total) have been pushed out of the 126 MB L2 before they are read again.

  value      algorithmic GB/s of the whole step, inputs resident in HBM, launches replayed from a
             CUDA graph, timed with CUDA events on the launching stream (max over ranks).
  e2e        the same step through the C-ABI calls, issued one by one inside the timed loop, with
             HOST activations: pinned host -> device copy of A and device -> host copy of Y inside
             the timed region (`graph_replay_value`: the same with the calls replayed from a graph).
  gemm       the prefill GEMM (M=2048, K=4096, N=14336, 1 % outlier channels) in TFLOP/s.
  configs    the other benchmark configurations (0: GEMV 1x4096x4096; 3: W8A16 GEMM 1024x4096x4096
             and GEMV 1x4096x14336; 4: GEMM 512x32768x4096 and GEMV 1x4096x32768), each in us and
             GB/s or TFLOP/s with its fraction of the measured peak.
  roofline   achieved / measured-peak for the GEMV step (HBM bound); gemm.roofline likewise (tensor).
  cpu_baseline  the fp64 CPU oracle timed on this machine's host cores on a bounded sample.

`--impl reference` times the CPU oracle instead (rank 0 only).  Multi-GPU runs (`torchrun`) give
every rank the same step on its own GPU (independent problems, no data-path collective): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GEMV_MS = (1, 4, 16)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# ------------------------------------------------------------------------------------------ helpers
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            data = json.load(fh)
        return {k: float(data[k]) for k in FALLBACK_PEAKS if k in data}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def load_traffic():
    """DRAM bytes per launch from the committed ncu summaries (profiles/traffic.json), if present."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh)
    return {}


def gemv_algorithmic_bytes(bits, M, K, N, group=128):
    """What the method itself must move, each byte once: weights, scales, zeros, A and Y."""
    b = K * N * bits // 8 + (K // group) * N * 2 + M * K * 2 + M * N * 2
    if bits == 4:
        b += (K // group) * N // 2
    return b


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init_dist(backend):
    import torch.distributed as dist
    rank, _, world = dist_env()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def lines(self) -> int:
        if self.proc is None or self.path is None:
            return 1 << 30                        # no sampler: nothing to wait for
        try:
            with open(self.path) as fh:
                return sum(1 for _ in fh)
        except OSError:
            return 1 << 30

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()                      # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = []
        with open(self.path) as fh:
            for line in fh:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) == 7:
                    try:
                        rows.append((float(parts[0]), float(parts[1]), float(parts[2]), parts[3:]))
                    except ValueError:
                        pass
        os.unlink(self.path)
        if not rows:
            return out
        busy = [r for r in rows if r[2] > 250.0] or rows          # samples under load if any
        out["sm_mhz"] = float(np.median([r[0] for r in busy]))
        out["sm_max_mhz"] = float(rows[0][1])
        out["samples"] = len(busy)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for i, name in enumerate(names):
            if any(r[3][i].lower().startswith("active") for r in busy):
                out["reasons"].append(name)
        return out


# ------------------------------------------------------------------------------- CPU oracle timing
_ORACLE_PROBLEMS = None


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return int(os.cpu_count() or 1)


def time_oracle_sample(repeats: int = 3):
    """The oracle as it stands on the step itself: the four layer shapes at M = 1, 4, 16, `repeats` passes (about ten
    seconds of CPU work; most of it is the fp64 dequantization of the weights, which does not depend on M)."""
    from oracle import tilefuse_oracle as orc
    from paper_2606_11357_b200 import workloads as wl
    global _ORACLE_PROBLEMS
    if _ORACLE_PROBLEMS is None:
        _ORACLE_PROBLEMS = [wl.config1(M, K, N) for (K, N) in wl.LLAMA3_8B_SHAPES for M in GEMV_MS]
    probs = _ORACLE_PROBLEMS
    np.zeros(1) @ np.zeros(1)                      # make sure the BLAS threads exist before counting them
    nbytes = sum(gemv_algorithmic_bytes(4, p.M, p.K, p.N) for p in probs)
    t0 = time.perf_counter()
    for _ in range(repeats):
        for p in probs:
            orc.solve(p)
    dt = (time.perf_counter() - t0) / repeats
    return {"value": nbytes / dt / 1e9, "unit": "GB/s", "cores": oracle_threads(), "kind": "oracle",
            "sample": f"the oracle as it stands (numpy: vectorised fp64 unpack and dequantization, one library fp64 matmul per call, BLAS threads as "
                      f"counted in `cores`), the whole step (four Llama-3-8B layer shapes at M = 1, 4, 16), {repeats} passes "
                      f"({dt:.2f} s per pass, {nbytes / 1e6:.1f} MB algorithmic per pass)"}, dt, nbytes


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    for _ in range(min(args.warmup, 1)):
        time_oracle_sample(repeats=1)
    total_t, total_b = 0.0, 0
    steps = max(1, min(args.steps, 5))             # each step is a bounded sample; keep the run to minutes
    for _ in range(steps):
        _, dt, nb = time_oracle_sample(repeats=1)
        total_t += dt
        total_b += nb
    value = total_b / total_t / 1e9
    line = {
        "impl": "reference", "metric": "W4A16 GEMV GB/s", "value": value, "unit": "GB/s", "n_gpus": world,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": total_t / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "cfg1 decode GEMV sweep: Llama-3-8B layer shapes at M = 1, 4, 16 (each step: the oracle on the whole step, once)",
                   "l2": "n/a (CPU)"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": oracle_threads(), "kind": "oracle",
                         "sample": "the oracle as it stands (numpy fp64, one library matmul per call): the whole step (four layer shapes at M = 1, 4, 16) once per timed step"},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# --------------------------------------------------------------------------------------- GPU bench
def run_gpu(args):
    import torch
    from paper_2606_11357_b200 import binding as tf
    from paper_2606_11357_b200 import workloads as wl

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank % torch.cuda.device_count())
    dev = torch.device("cuda", torch.cuda.current_device())
    init_dist("nccl")
    tf.lib()                                        # fail loudly if the extension is missing
    peaks, peak_kind = load_peaks()
    traffic = load_traffic()

    # ---- inputs: seeded, synthetic, resident in HBM ----------------------------------------------------
    stream = torch.cuda.Stream()
    ws_bytes = tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, 16, 4096, 4096)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    calls = []                                       # (set, M, K, N, blob, a, y, a_host, y_host)
    step_bytes = 0
    # The activations (and the results) of one step live side by side in one device buffer and one pinned host buffer
    # per weight set, so that the end-to-end loop moves each direction with a single copy per step.
    a_elems = sum(M * K for (K, N) in wl.LLAMA3_8B_SHAPES for M in GEMV_MS)
    y_elems = sum(M * N for (K, N) in wl.LLAMA3_8B_SHAPES for M in GEMV_MS)
    a_host_all = [torch.empty(a_elems, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    y_host_all = [torch.empty(y_elems, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    a_dev_all = [torch.empty(a_elems, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    y_dev_all = [torch.empty(y_elems, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    a_off, y_off = [0, 0], [0, 0]
    awq_host = {}                                    # the AWQ arrays as given, for the layout arm of the ablation
    for (K, N) in wl.LLAMA3_8B_SHAPES:
        prob = wl.config1(16, K, N)
        awq_host[(K, N)] = (prob.qweight, prob.scales_f16, prob.qzeros)
        blob_host = tf.tf_pack_awq(prob.qweight, prob.scales_f16, prob.qzeros, K, N)
        a_all = torch.from_numpy(prob.a_bf16.view(np.int16).copy()).view(torch.bfloat16)
        for M in GEMV_MS:
            step_bytes += gemv_algorithmic_bytes(4, M, K, N)
            for s in range(2):
                blob = torch.from_numpy(blob_host).to(dev)
                a_host = a_host_all[s][a_off[s]:a_off[s] + M * K].view(M, K)
                a_host.copy_(a_all[:M])
                a = a_dev_all[s][a_off[s]:a_off[s] + M * K].view(M, K)
                a.copy_(a_host)
                y = y_dev_all[s][y_off[s]:y_off[s] + M * N].view(M, N)
                y_host = y_host_all[s][y_off[s]:y_off[s] + M * N].view(M, N)
                a_off[s] += M * K
                y_off[s] += M * N
                calls.append((s, M, K, N, blob, a, y, a_host, y_host))
    # one decode step per batch size: for each M, the four layer shapes in turn (as a model runs them)
    sets = [[c for M in GEMV_MS for c in calls if c[0] == s and c[1] == M] for s in range(2)]
    launches_per_step = len(sets[0])

    def enqueue_step(s):
        for (_, M, K, N, blob, a, y, _, _) in sets[s]:
            tf.tf_gemv_w4a16(blob, a, y, M, K, N, ws, stream=stream)

    torch.cuda.synchronize()                         # inputs were created on the default stream
    with torch.cuda.stream(stream):
        for s in range(2):
            enqueue_step(s)
    stream.synchronize()
    if tf.tf_device_status(ws, stream=stream) != 0:
        raise SystemExit("device status word reports an error after the first step")

    # the clock sampler needs a moment to come up: start it before the graph is captured
    sampler = ClockSampler(torch.cuda.current_device())
    if rank == 0:
        sampler.start()
    # two steps (one per weight set) per graph replay
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            enqueue_step(0)
            enqueue_step(1)

    replays_warm = max(2, (args.warmup + 1) // 2)
    replays = max(1, (args.steps + 1) // 2)
    steps_timed = 2 * replays
    with torch.cuda.stream(stream):
        for _ in range(replays_warm):
            graph.replay()
    stream.synchronize()
    barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    lines_before = sampler.lines() if rank == 0 else 0
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(replays):
            graph.replay()
        e1.record(stream)
    stream.synchronize()
    torch.cuda.synchronize()
    barrier()
    ms_local = e0.elapsed_time(e1)
    ms_total = max_over_ranks(ms_local, dev)
    # A short timed region can end before the sampler has taken a sample under load: keep the same load running
    # (the same graph, untimed) until it has a few, for at most two seconds.
    extended = False
    if rank == 0:
        t_wait = time.time()
        while sampler.lines() < lines_before + 3 and time.time() - t_wait < 2.0:
            extended = True
            with torch.cuda.stream(stream):
                for _ in range(200):
                    graph.replay()
            stream.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None and extended:
        clocks["note"] = "timed region shorter than the sampling period: sampled while the same graph kept replaying right after it"

    ms_per_step = ms_total / steps_timed
    value = world * step_bytes / (ms_per_step * 1e-3) / 1e9

    # ---- end to end: host activations in, host result out, call by call ----------------------------------
    e2e_steps = max(2, min(steps_timed, 200))
    h2d = a_elems * 2
    d2h = y_elems * 2

    # Three streams: the copy-in of step i+1 and the copy-out of step i-1 run beside the GEMVs of step i (the two
    # weight sets have their own activation and result buffers, so consecutive steps never share one).  Every step
    # still gets its inputs from pinned host memory and delivers its results there inside the timed region.
    # The 12 calls of a step are captured once per weight set (as a decoder would capture its layer) and replayed.
    step_graph = []
    for s in range(2):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g, stream=stream):
                enqueue_step(s)
        step_graph.append(g)
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]          # inputs of the set are on the device
    ev_comp = [torch.cuda.Event() for _ in range(2)]        # the set's GEMVs are done
    ev_out = [torch.cuda.Event() for _ in range(2)]         # the set's results are on the host

    def e2e_step(s, first, use_graph):
        with torch.cuda.stream(s_in):
            if not first:
                s_in.wait_event(ev_comp[s])                 # the step that last read these activations
            a_dev_all[s].copy_(a_host_all[s], non_blocking=True)
            ev_in[s].record(s_in)
        with torch.cuda.stream(stream):
            stream.wait_event(ev_in[s])
            if not first:
                stream.wait_event(ev_out[s])                # the results of that step have left the device
            if use_graph:
                step_graph[s].replay()
            else:
                enqueue_step(s)                             # twelve tf_gemv_w4a16 calls through the C ABI, one by one
            ev_comp[s].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[s])
            y_host_all[s].copy_(y_dev_all[s], non_blocking=True)
            ev_out[s].record(s_out)

    def e2e_run(use_graph):
        e2e_step(0, True, use_graph)
        e2e_step(1, True, use_graph)
        torch.cuda.synchronize()
        barrier()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            e2e_step(i & 1, False, use_graph)
        torch.cuda.synchronize()
        dt = max_over_ranks(time.perf_counter() - t0, dev)
        return world * step_bytes * e2e_steps / dt / 1e9

    e2e_value = e2e_run(False)                   # the calls a user makes, issued inside the timed loop
    e2e_graph_value = e2e_run(True)              # the same step captured once per weight set and replayed

    # ---- per-shape breakdown (graph of 2 launches on alternating copies; context for the step number) ---
    per_shape = []
    if rank == 0:
        for (K, N) in wl.LLAMA3_8B_SHAPES:
            for M in GEMV_MS:
                pair = [c for c in calls if (c[1], c[2], c[3]) == (M, K, N)]
                extra = []
                nbytes = gemv_algorithmic_bytes(4, M, K, N)
                need = int(300e6 // nbytes) + 2                      # rotate over > 2x L2 worth of copies
                while len(pair) + len(extra) < need:
                    extra.append(pair[0][4].clone())
                torch.cuda.synchronize()
                blobs = [p[4] for p in pair] + extra
                g = torch.cuda.CUDAGraph()
                a, y = pair[0][5], pair[0][6]
                with torch.cuda.stream(stream):
                    with torch.cuda.graph(g, stream=stream):
                        for b in blobs:
                            tf.tf_gemv_w4a16(b, a, y, M, K, N, ws, stream=stream)
                    g.replay()
                    stream.synchronize()
                    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    s0.record(stream)
                    for _ in range(5):
                        g.replay()
                    s1.record(stream)
                    stream.synchronize()
                us = s0.elapsed_time(s1) * 1e3 / (5 * len(blobs))
                per_shape.append({"M": M, "K": K, "N": N, "us": round(us, 3), "GBps": round(nbytes / us / 1e3, 1),
                                  "frac_of_peak": round(nbytes / us / 1e3 / peaks["hbm_gbs"], 4)})
                del g, extra, blobs

    # ---- one decoder layer at M = 1: seven GEMVs, or four after joining QKV and gate + up at pack time -------
    decode_layer = None
    if rank == 0:
        def blob_of(K, N):
            return next(c[4] for c in calls if (c[1], c[2], c[3]) == (1, K, N))
        def act_of(K):
            return next(c[5] for c in calls if c[1] == 1 and c[2] == K)
        (Kh, Nh), (_, Nkv), (_, Nff), (Kff, _) = wl.LLAMA3_8B_SHAPES
        bq, bkv, bff, bdown = blob_of(Kh, Nh), blob_of(Kh, Nkv), blob_of(Kh, Nff), blob_of(Kff, Nh)
        host = lambda t: t.cpu().numpy()
        bqkv = torch.from_numpy(tf.tf_pack_concat([host(bq), host(bkv), host(bkv)])).to(dev)
        bgu = torch.from_numpy(tf.tf_pack_concat([host(bff), host(bff)])).to(dev)
        a_h, a_ff = act_of(Kh), act_of(Kff)
        y_big = torch.empty((1, 2 * Nff), dtype=torch.bfloat16, device=dev)
        layers = {"unfused": [(bq, a_h, Kh, Nh), (bkv, a_h, Kh, Nkv), (bkv, a_h, Kh, Nkv), (bq, a_h, Kh, Nh),
                              (bff, a_h, Kh, Nff), (bff, a_h, Kh, Nff), (bdown, a_ff, Kff, Nh)],
                  "fused": [(bqkv, a_h, Kh, Nh + 2 * Nkv), (bq, a_h, Kh, Nh), (bgu, a_h, Kh, 2 * Nff), (bdown, a_ff, Kff, Nh)]}
        decode_layer = {"M": 1, "note": "Llama-3-8B decoder layer, W4A16, CUDA graph of 3 layers on separate weight copies"}
        for name, ops in layers.items():
            copies = [[(b.clone(), a, K, N) for (b, a, K, N) in ops] for _ in range(3)]     # 3 x 113 MB > L2
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(stream):
                for (b, a, K, N) in copies[0]:
                    tf.tf_gemv_w4a16(b, a, y_big[:, :N], 1, K, N, ws, stream=stream)
                stream.synchronize()
                with torch.cuda.graph(g, stream=stream):
                    for layer in copies:
                        for (b, a, K, N) in layer:
                            tf.tf_gemv_w4a16(b, a, y_big[:, :N], 1, K, N, ws, stream=stream)
                g.replay()
                stream.synchronize()
                s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s0.record(stream)
                for _ in range(10):
                    g.replay()
                s1.record(stream)
                stream.synchronize()
            decode_layer[name] = {"launches": len(ops), "us_per_layer": round(s0.elapsed_time(s1) * 1e3 / 30, 2)}
            del g, copies
        iso = {(r["K"], r["N"]): r["us"] for r in per_shape if r["M"] == 1}
        decode_layer["sum_of_isolated_us"] = round(2 * iso[(Kh, Nh)] + 2 * iso[(Kh, Nkv)] + 2 * iso[(Kh, Nff)] + iso[(Kff, Nh)], 2)
        assert tf.tf_device_status(ws) == 0
        del bqkv, bgu

    # ---- prefill GEMM (config 2) ---------------------------------------------------------------------------
    gemm = None
    if rank == 0 and not args.skip_gemm:
        p2 = wl.config2()
        blob = torch.from_numpy(tf.tf_pack_awq(p2.qweight, p2.scales_f16, p2.qzeros, p2.K, p2.N)).to(dev)
        a = torch.from_numpy(p2.a_bf16.view(np.int16).copy()).to(dev).view(torch.bfloat16)
        y = torch.empty((p2.M, p2.N), dtype=torch.bfloat16, device=dev)
        gws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMM_W4A16, p2.M, p2.K, p2.N), dtype=torch.uint8, device=dev)
        iters = 20
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            for _ in range(5):
                tf.tf_gemm_w4a16(blob, a, y, p2.M, p2.K, p2.N, gws, stream=stream)
            stream.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(stream)
            for _ in range(iters):
                tf.tf_gemm_w4a16(blob, a, y, p2.M, p2.K, p2.N, gws, stream=stream)
            g1.record(stream)
            stream.synchronize()
        if tf.tf_device_status(gws, stream=stream) != 0:
            raise SystemExit("GEMM device status word reports an error")
        us = g0.elapsed_time(g1) * 1e3 / iters
        flops = 2.0 * p2.M * p2.K * p2.N
        tfl = flops / us / 1e6
        gemm = {"metric": "W4A16 GEMM TFLOP/s", "value": tfl, "unit": "TFLOP/s", "us_per_launch": us,
                "workload": f"cfg2 prefill GEMM M={p2.M} K={p2.K} N={p2.N}, 1% outlier channels x20",
                "dtype": "bf16", "gpu_launches": iters,
                "roofline": {"bound": "tensor", "achieved": tfl, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                             "frac": tfl / peaks["bf16_tflops"], "peak_kind": f"{peak_kind} (burst, cuBLAS bf16)",
                             "traffic": traffic.get("gemm_w4_cfg2_dram_bytes_per_launch")}}

    # ---- the other configurations: 0 (GEMV 1x4096x4096), 3 (W8A16 GEMM and GEMV), 4 (32K stress GEMM and GEMV) -----
    configs = None
    if rank == 0 and not args.skip_gemm:
        def gemv_case(label, prob, bits):
            """us per call over rotating weight copies (more than twice the L2 in rotation), replayed from a graph."""
            M, K, N = prob.M, prob.K, prob.N
            host = (tf.tf_pack_awq(prob.qweight, prob.scales_f16, prob.qzeros, K, N) if bits == 4
                    else tf.tf_pack_w8(prob.w_i8, prob.scales_f16, K, N))
            nbytes = gemv_algorithmic_bytes(bits, M, K, N)
            first = torch.from_numpy(host).to(dev)
            blobs = [first] + [first.clone() for _ in range(int(300e6 // nbytes) + 1)]
            a = torch.from_numpy(prob.a_bf16.view(np.int16).copy()).to(dev).view(torch.bfloat16)
            y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            fn = tf.tf_gemv_w4a16 if bits == 4 else tf.tf_gemv_w8a16
            g = torch.cuda.CUDAGraph()
            torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                fn(blobs[0], a, y, M, K, N, ws, stream=stream)
                stream.synchronize()
                with torch.cuda.graph(g, stream=stream):
                    for b in blobs:
                        fn(b, a, y, M, K, N, ws, stream=stream)
                g.replay()
                stream.synchronize()
                s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s0.record(stream)
                for _ in range(5):
                    g.replay()
                s1.record(stream)
                stream.synchronize()
            us = s0.elapsed_time(s1) * 1e3 / (5 * len(blobs))
            gbs = nbytes / us / 1e3
            return {"config": label, "call": f"tf_gemv_w{bits}a16", "M": M, "K": K, "N": N, "us": round(us, 3),
                    "GBps": round(gbs, 1), "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 4),
                    "frac_of_8TBps": round(gbs / 8000.0, 4), "l2": f"{len(blobs)} weight copies in rotation"}

        def gemm_case(label, prob, bits):
            M, K, N = prob.M, prob.K, prob.N
            host = (tf.tf_pack_awq(prob.qweight, prob.scales_f16, prob.qzeros, K, N) if bits == 4
                    else tf.tf_pack_w8(prob.w_i8, prob.scales_f16, K, N))
            blob = torch.from_numpy(host).to(dev)
            a = torch.from_numpy(prob.a_bf16.view(np.int16).copy()).to(dev).view(torch.bfloat16)
            y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            op = tf.TF_OP_GEMM_W4A16 if bits == 4 else tf.TF_OP_GEMM_W8A16
            gws = torch.zeros(tf.tf_workspace_size(op, M, K, N), dtype=torch.uint8, device=dev)
            fn = tf.tf_gemm_w4a16 if bits == 4 else tf.tf_gemm_w8a16
            torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                for _ in range(5):
                    fn(blob, a, y, M, K, N, gws, stream=stream)
                stream.synchronize()
                s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s0.record(stream)
                for _ in range(20):
                    fn(blob, a, y, M, K, N, gws, stream=stream)
                s1.record(stream)
                stream.synchronize()
            if tf.tf_device_status(gws, stream=stream) != 0:
                raise SystemExit("GEMM device status word reports an error")
            us = s0.elapsed_time(s1) * 1e3 / 20
            tfl = 2.0 * M * K * N / us / 1e6
            return {"config": label, "call": f"tf_gemm_w{bits}a16", "M": M, "K": K, "N": N, "us": round(us, 2),
                    "TFLOPs": round(tfl, 1), "frac_of_bf16_burst_peak": round(tfl / peaks["bf16_tflops"], 4),
                    "frac_of_2250_nominal": round(tfl / 2250.0, 4)}

        configs = [gemv_case("cfg0", wl.config0(), 4),
                   gemm_case("cfg3", wl.config3_gemm(), 8), gemv_case("cfg3", wl.config3_gemv(), 8),
                   gemm_case("cfg4", wl.config4_gemm(), 4), gemv_case("cfg4", wl.config4_gemv(), 4)]
        assert tf.tf_device_status(ws) == 0

    # ---- library kernels on the same sizes, as context (not part of the path, not a target) ----------------
    ceilings = None
    if rank == 0 and not args.skip_gemm:
        ceilings = {}
        with torch.cuda.stream(stream):
            # bf16 x bf16 library GEMM on the config-2 shape (weights already full precision in HBM)
            w_full = torch.randn((p2.K, p2.N), device=dev).to(torch.bfloat16)
            for _ in range(3):
                torch.matmul(a, w_full)
            stream.synchronize()
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(stream)
            for _ in range(10):
                torch.matmul(a, w_full)
            c1.record(stream)
            stream.synchronize()
            ceilings["matmul_bf16_cfg2_tflops"] = round(2.0 * p2.M * p2.K * p2.N / (c0.elapsed_time(c1) * 1e3 / 10) / 1e6, 1)
            del w_full
            # a read-only pass (library reduction) over 512 MB: what a kernel that only reads can reach
            src = torch.empty(128 * 1024 * 1024, dtype=torch.float32, device=dev)
            src.zero_()
            for _ in range(2):
                src.sum()
            stream.synchronize()
            c0.record(stream)
            for _ in range(5):
                src.sum()
            c1.record(stream)
            stream.synchronize()
            ceilings["read_only_pass_gbs"] = round(src.numel() * 4 / (c0.elapsed_time(c1) * 1e3 / 5) / 1e3, 1)
            del src
            # a device-to-device copy of as many bytes as each GEMV shape reads, back to back in a graph over rotating
            # sources: what a dependent chain of trivial kernels of that size takes (it moves twice the bytes)
            chain = {}
            for nbytes in sorted({gemv_algorithmic_bytes(4, 1, K, N) for (K, N) in wl.LLAMA3_8B_SHAPES}):
                copies = max(4, int(300e6 // nbytes) + 1)
                srcs = [torch.empty(nbytes // 4, dtype=torch.float32, device=dev).zero_() for _ in range(copies)]
                dst = torch.empty(nbytes // 4, dtype=torch.float32, device=dev)
                g = torch.cuda.CUDAGraph()
                dst.copy_(srcs[0])
                stream.synchronize()
                with torch.cuda.graph(g, stream=stream):
                    for t in srcs:
                        dst.copy_(t)
                g.replay()
                stream.synchronize()
                c0.record(stream)
                for _ in range(5):
                    g.replay()
                c1.record(stream)
                stream.synchronize()
                chain[str(nbytes)] = round(c0.elapsed_time(c1) * 1e3 / (5 * copies), 2)
                del g, srcs, dst
            ceilings["copy_us_per_call_at_gemv_bytes"] = chain
        ceilings["note"] = "torch library kernels, same process, context only"

    # ---- ablation (Section 5.5 analogue): fused kernels against full-precision weights kept in memory, and against
    # dequantizing into memory before every multiplication ------------------------------------------------------
    ablation = None
    if rank == 0 and not args.skip_gemm:
        def timed(fn, n):
            fn()
            stream.synchronize()
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(stream)
            for _ in range(n):
                fn()
            c1.record(stream)
            stream.synchronize()
            return c0.elapsed_time(c1) * 1e3 / n
        ablation = {"note": "us per call; bf16 = torch.matmul on weights held in bf16; unfused = tf_dequant_bf16 into memory, then torch.matmul"}
        with torch.cuda.stream(stream):
            for name, M, K, N, fused in (("gemv_1x4096x14336", 1, 4096, 14336, tf.tf_gemv_w4a16),
                                         ("gemm_2048x4096x14336", 2048, 4096, 14336, tf.tf_gemm_w4a16)):
                pa = wl.make_w4(M, K, N, seed=7)
                blobs = [torch.from_numpy(tf.tf_pack_awq(pa.qweight, pa.scales_f16, pa.qzeros, K, N)).to(dev) for _ in range(1)]
                blobs += [blobs[0].clone() for _ in range(5)]                       # 6 x 29 MB: beyond L2 in rotation
                a = torch.from_numpy(pa.a_bf16.view(np.int16).copy()).to(dev).view(torch.bfloat16)
                y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                op = tf.TF_OP_GEMV_W4A16 if M <= 16 else tf.TF_OP_GEMM_W4A16
                aws = torch.zeros(tf.tf_workspace_size(op, M, K, N), dtype=torch.uint8, device=dev)
                w_full = [torch.empty((K, N), dtype=torch.bfloat16, device=dev) for _ in range(2)]     # 2 x 117 MB
                tf.tf_dequant_bf16(blobs[0], w_full[0], 4, K, N, stream=stream)
                w_full[1].copy_(w_full[0])
                it = {"i": 0}
                def run_fused():
                    it["i"] += 1
                    fused(blobs[it["i"] % 6], a, y, M, K, N, aws, stream=stream)
                def run_bf16():
                    it["i"] += 1
                    torch.matmul(a, w_full[it["i"] & 1], out=y)
                def run_unfused():
                    it["i"] += 1
                    tf.tf_dequant_bf16(blobs[it["i"] % 6], w_full[it["i"] & 1], 4, K, N, stream=stream)
                    torch.matmul(a, w_full[it["i"] & 1], out=y)
                n = 30 if M <= 16 else 10
                ablation[name] = {"fused_w4_us": round(timed(run_fused, n), 2), "bf16_us": round(timed(run_bf16, n), 2),
                                  "unfused_w4_us": round(timed(run_unfused, n), 2)}
                assert tf.tf_device_status(aws) == 0
                del blobs, w_full, a, y, aws

    # ---- layout arm of the ablation: the same fused GEMV on the AWQ arrays as given (no offline pre-tiling) ----
    if rank == 0 and ablation is not None:
        layout = {"note": "us per call, graph replay over 6 rotating weight copies (the 2 MB and 9 MB shapes stay in L2 "
                          "for both arms); pretiled = tf_gemv_w4a16 on the packed blob, raw = tf_gemv_awq_raw on "
                          "qweight / scales / qzeros"}
        def replay_us(enqueue, copies):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(stream):
                enqueue(0)
                stream.synchronize()
                with torch.cuda.graph(g, stream=stream):
                    for c in range(copies):
                        enqueue(c)
                g.replay()
                stream.synchronize()
                c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                c0.record(stream)
                for _ in range(5):
                    g.replay()
                c1.record(stream)
                stream.synchronize()
            return c0.elapsed_time(c1) * 1e3 / (5 * copies)
        for (K, N) in wl.LLAMA3_8B_SHAPES:
            qw, sc, qz = awq_host[(K, N)]
            raw = [(torch.from_numpy(qw.view(np.int32)).to(dev), torch.from_numpy(sc.view(np.int16)).to(dev),
                    torch.from_numpy(qz.view(np.int32)).to(dev))]
            raw += [tuple(t.clone() for t in raw[0]) for _ in range(5)]
            tiled = [next(c[4] for c in calls if (c[2], c[3]) == (K, N))]
            tiled += [tiled[0].clone() for _ in range(5)]
            for M in GEMV_MS:
                a = next(c[5] for c in calls if (c[1], c[2], c[3]) == (M, K, N))
                y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                rws = torch.empty(tf.tf_gemv_awq_raw_workspace_size(M, K, N, 128), dtype=torch.uint8, device=dev)
                t_tiled = replay_us(lambda c: tf.tf_gemv_w4a16(tiled[c], a, y, M, K, N, ws, stream=stream), 6)
                t_raw = replay_us(lambda c: tf.tf_gemv_awq_raw(*raw[c], a, y, M, K, N, 128, rws, stream=stream), 6)
                layout[f"{M}x{K}x{N}"] = {"pretiled_us": round(t_tiled, 2), "raw_us": round(t_raw, 2)}
            del raw, tiled
        assert tf.tf_device_status(ws) == 0
        # the GEMM arm: the pre-tiled GEMM on the offline blob against the same GEMM with the AWQ arrays re-tiled on
        # the fly into scratch on every call (tf_gemm_awq_raw): the difference is what the offline pre-tiling removes
        p2 = wl.config2()
        qw = torch.from_numpy(p2.qweight.view(np.int32)).to(dev)
        sc = torch.from_numpy(p2.scales_f16.view(np.int16)).to(dev)
        qz = torch.from_numpy(p2.qzeros.view(np.int32)).to(dev)
        blob = torch.from_numpy(tf.tf_pack_awq(p2.qweight, p2.scales_f16, p2.qzeros, p2.K, p2.N)).to(dev)
        a2 = torch.from_numpy(p2.a_bf16.view(np.int16).copy()).to(dev).view(torch.bfloat16)
        y2 = torch.empty((p2.M, p2.N), dtype=torch.bfloat16, device=dev)
        rws = torch.zeros(tf.tf_gemm_awq_raw_workspace_size(p2.M, p2.K, p2.N, 128), dtype=torch.uint8, device=dev)
        with torch.cuda.stream(stream):
            t_pre = timed(lambda: tf.tf_gemm_w4a16(blob, a2, y2, p2.M, p2.K, p2.N, rws, stream=stream), 10)
            t_raw = timed(lambda: tf.tf_gemm_awq_raw(qw, sc, qz, a2, y2, p2.M, p2.K, p2.N, 128, rws, stream=stream), 10)
        assert tf.tf_device_status(rws) == 0
        layout[f"gemm_{p2.M}x{p2.K}x{p2.N}"] = {"pretiled_us": round(t_pre, 2), "raw_us": round(t_raw, 2),
                                                "note": "raw = tf_pack_awq_device into scratch + the pre-tiled GEMM, per call"}
        del qw, sc, qz, blob, a2, y2, rws
        ablation["layout"] = layout

    if rank != 0:
        return 0
    cpu_baseline = None
    if not args.skip_cpu:
        cpu_baseline, _, _ = time_oracle_sample()
    achieved = step_bytes / (ms_local / steps_timed * 1e-3) / 1e9
    line = {
        "metric": "W4A16 GEMV GB/s", "value": value, "unit": "GB/s", "n_gpus": world, "steps": steps_timed,
        "warmup": 2 * replays_warm, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "cfg1 decode GEMV sweep: Llama-3-8B layer shapes 4096x4096, 4096x1024, 4096x14336, "
                               "14336x4096 for M=1, then M=4, then M=16 (12 tf_gemv_w4a16 calls per step)",
                   "l2": "inputs larger than L2: two alternating sets of 12 weight copies, 432 MB in rotation",
                   "bytes_per_step": step_bytes, "launch": "CUDA graph replay of two steps"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps,
                "how": "per step one pinned-host -> device copy of the 12 activation blocks, 12 tf_gemv_w4a16 calls issued one by "
                       "one through the C ABI inside the timed loop (no graph), one device -> pinned-host copy of the 12 results; "
                       "copies and GEMVs of neighbouring steps overlap on three streams (two buffer sets); wall clock over all steps",
                "graph_replay_value": e2e_graph_value,
                "graph_replay_how": "the same loop with the 12 calls of a step captured once per weight set and replayed"},
        "gpu_launches": launches_per_step * steps_timed,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"{peak_kind} (copy bandwidth)",
                     "traffic": traffic.get("gemv_w4_step_dram_bytes"),
                     "kernel": "gemv_stream_kernel (all 12 launches of the step)"},
        "cpu_baseline": cpu_baseline,
        "configs": configs,
        "per_shape": per_shape,
        "decode_layer": decode_layer,
        "ablation": ablation,
        "gemm": gemm,
        "ceilings": ceilings,
    }
    print(json.dumps(line), flush=True)
    return 0


def run_gemm_sweep(args):
    """Shape stability of the prefill GEMM (the paper's kernel evaluation, Section 5.1: M swept in steps of 256 over
    two shapes with K and N swapped), preceded by the token counts between the decode and the prefill range, which
    take the same entry point with token tiles of 32 / 64 / 128.  Prints one JSON object with us and TFLOP/s per
    (shape, M)."""
    import torch
    from paper_2606_11357_b200 import binding as tf
    from paper_2606_11357_b200 import workloads as wl
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    rows = []
    for (K, N) in ((4096, 14336), (14336, 4096)):
        p = wl.make_w4(1, K, N, seed=11)
        blob = torch.from_numpy(tf.tf_pack_awq(p.qweight, p.scales_f16, p.qzeros, K, N)).to(dev)
        for M in (17, 32, 64, 128, 192) + tuple(range(256, 4097, 256)):       # below 256: the narrower token tiles
            a = torch.randn((M, K), device=dev).to(torch.bfloat16)
            y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMM_W4A16, M, K, N), dtype=torch.uint8, device=dev)
            for _ in range(3):
                tf.tf_gemm_w4a16(blob, a, y, M, K, N, ws)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n = 10
            e0.record()
            for _ in range(n):
                tf.tf_gemm_w4a16(blob, a, y, M, K, N, ws)
            e1.record()
            torch.cuda.synchronize()
            assert tf.tf_device_status(ws) == 0
            us = e0.elapsed_time(e1) * 1e3 / n
            rows.append({"K": K, "N": N, "M": M, "us": round(us, 1), "tflops": round(2.0 * M * K * N / us / 1e6, 1)})
            del a, y, ws
    print(json.dumps({"gemm_sweep_w4a16": rows}), flush=True)
    return 0


def gather_columns(y_local, counts):
    """All-gather of column shards: rank r holds y_local [M, counts[r]]; returns y [M, sum(counts)] on every rank.
    The only exchange of the column-parallel arrangement (Section 4.4: distinct output columns per worker, shared
    activations, no partial sums between workers).  NCCL on GPUs, gloo in the CPU test."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return y_local
    world, M, width = dist.get_world_size(), y_local.shape[0], max(counts)
    padded = torch.zeros((M, width), dtype=y_local.dtype, device=y_local.device)
    padded[:, :y_local.shape[1]] = y_local
    out = [torch.empty((M, width), dtype=y_local.dtype, device=y_local.device) for _ in range(world)]
    dist.all_gather(out, padded)
    return torch.cat([out[r][:, :counts[r]] for r in range(world)], dim=1)


def run_column_parallel(args):
    """One decode pass over the four layer shapes with every matrix sharded by columns over the ranks (Section 4.4):
    each rank packs its shard out of the full blob (tf_pack_shard), multiplies the full activations into it
    (tf_gemv_w4a16 with N = its column count) and the results are all-gathered.  Strong scaling: the total work is
    fixed.  Prints one JSON line.  On one GPU the shard is the whole matrix and the gather is the identity."""
    import torch
    from paper_2606_11357_b200 import binding as tf
    from paper_2606_11357_b200 import workloads as wl
    rank, local_rank, world = dist_env()
    torch.cuda.set_device(local_rank % torch.cuda.device_count())
    dev = torch.device("cuda", torch.cuda.current_device())
    init_dist("nccl")
    M = args.profile_m or 1
    stream = torch.cuda.current_stream()
    ws = torch.zeros(tf.tf_workspace_size(tf.TF_OP_GEMV_W4A16, 16, 4096, 4096), dtype=torch.uint8, device=dev)
    layers, total_bytes = [], 0
    for (K, N) in wl.LLAMA3_8B_SHAPES:
        prob = wl.config1(M, K, N)
        full = tf.tf_pack_awq(prob.qweight, prob.scales_f16, prob.qzeros, K, N)
        counts = [tf.tf_shard_columns(N, r, world)[1] for r in range(world)]
        shard = torch.from_numpy(tf.tf_pack_shard(full, rank, world)).to(dev)
        copies = [shard] + [shard.clone() for _ in range(int(300e6 // max(shard.numel(), 1)) + 1)]   # beyond L2 in rotation
        a = torch.from_numpy(prob.a_bf16.view(np.int16).copy()).to(dev).view(torch.bfloat16)
        y_local = torch.empty((M, counts[rank]), dtype=torch.bfloat16, device=dev)
        layers.append((K, N, counts, copies, a, y_local))
        total_bytes += gemv_algorithmic_bytes(4, M, K, N)
    it = {"i": 0}

    def step():
        it["i"] += 1
        outs = []
        for (K, N, counts, copies, a, y_local) in layers:
            tf.tf_gemv_w4a16(copies[it["i"] % len(copies)], a, y_local, M, K, counts[rank], ws)
            outs.append(gather_columns(y_local, counts))
        return outs

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps = min(args.steps, 2000)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), dev) / steps
    if tf.tf_device_status(ws) != 0:
        raise SystemExit("device status word reports an error")
    if rank == 0:
        print(json.dumps({"mode": "column_parallel", "metric": "W4A16 GEMV GB/s", "value": total_bytes / (ms * 1e-3) / 1e9,
                          "unit": "GB/s", "n_gpus": world, "steps": steps, "ms_per_step": ms, "scaling": "strong",
                          "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                          "config": {"workload": f"Llama-3-8B layer shapes at M = {M}, every matrix sharded by columns over the ranks, "
                                                 "results all-gathered; calls issued one by one",
                                     "columns_per_rank": {f"{K}x{N}": counts for (K, N, counts, _, _, _) in layers}}}), flush=True)
    return 0


def run_profile_case(args):
    """A handful of launches of one kernel on one seeded case, for `ncu` captures (prints no bench line)."""
    import torch
    from paper_2606_11357_b200 import binding as tf
    from paper_2606_11357_b200 import workloads as wl
    torch.cuda.set_device(0)
    kind, bits = args.profile_case.split("_")
    big = bits.endswith("big")
    bits = int(bits[1])
    shape = tuple(int(v) for v in args.profile_shape.lower().split("x")) if args.profile_shape else None
    if kind == "gemv" and big:
        prob = wl.config4_gemv()
    elif kind == "gemv":
        K, N = shape or (4096, 14336)
        prob = (wl.config1(args.profile_m or 1, K, N) if bits == 4 else wl.config3_gemv())
    elif big:
        prob = wl.config4_gemm()
    else:
        prob = (wl.config2(args.profile_m or 2048) if bits == 4 else wl.config3_gemm())
    M, K, N = prob.M, prob.K, prob.N
    host = (tf.tf_pack_awq(prob.qweight, prob.scales_f16, prob.qzeros, K, N) if bits == 4
            else tf.tf_pack_w8(prob.w_i8, prob.scales_f16, K, N))
    copies = [torch.from_numpy(host).cuda() for _ in range(max(1, args.steps))]
    a = torch.from_numpy(prob.a_bf16.view(np.int16).copy()).cuda().view(torch.bfloat16)
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    op = {("gemv", 4): 0, ("gemv", 8): 1, ("gemm", 4): 2, ("gemm", 8): 3}[(kind, bits)]
    ws = torch.zeros(tf.tf_workspace_size(op, M, K, N), dtype=torch.uint8, device="cuda")
    fn = getattr(tf, f"tf_{kind}_w{bits}a16")
    for blob in copies:
        fn(blob, a, y, M, K, N, ws)
    torch.cuda.synchronize()
    status = tf.tf_device_status(ws)
    print(json.dumps({"profile_case": args.profile_case, "M": M, "K": K, "N": N, "launches": len(copies),
                      "device_status": status}), flush=True)
    return 0 if status == 0 else 1


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--skip-gemm", action="store_true", help="leave out the prefill GEMM section")
    ap.add_argument("--skip-cpu", action="store_true", help="leave out the CPU-oracle baseline")
    ap.add_argument("--profile-case", choices=["gemv_w4", "gemv_w4big", "gemv_w8", "gemm_w4", "gemm_w4big", "gemm_w8"], default=None,
                    help="run --steps launches of one kernel on one case and exit (for ncu captures)")
    ap.add_argument("--profile-m", type=int, default=0, help="token count for --profile-case")
    ap.add_argument("--profile-shape", default="", help="KxN of a config-1 layer shape for --profile-case gemv_w4 (default 4096x14336)")
    ap.add_argument("--column-parallel", action="store_true",
                    help="decode pass with every matrix sharded by columns over the ranks and the results all-gathered (--profile-m tokens)")
    ap.add_argument("--gemm-sweep", action="store_true", help="time the W4A16 GEMM for M = 256..4096 on two K/N-swapped shapes")
    args = ap.parse_args(argv)
    if args.gemm_sweep:
        return run_gemm_sweep(args)
    if args.column_parallel:
        return run_column_parallel(args)
    if args.profile_case:
        return run_profile_case(args)
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
