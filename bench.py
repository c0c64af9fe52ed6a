#!/usr/bin/env python
"""Benchmark of the ILRe token-recall path on B200.

A "step" is one whole recall (query packing, row statistics, scores, pooling, top-K_m
selection, allocation) on the L = 1M benchmark configuration: key cache [1048576, 8, 128]
bf16 (2 GiB), q_len = 256, budget 4096, window sizes {1,7,15,31,63}.  The headline value is
key-cache GB/s = bytes of K / time of one recall, with the inputs resident in HBM; `e2e` is
the same metric through the host entry point (host buffers, copies inside the timed region).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config NAME]

With N > 1 (under torchrun) every rank runs an independent replica of the same recall on its
own GPU (the path has no exchange step); the value is the sum over ranks divided by the
slowest rank's time; the same line then carries, under `sharded_recall`, ONE recall with the
keys split by position over the ranks (its two all-gathers included).  `--impl reference`
times the CPU oracle on a bounded sample.

Beside the headline the line carries `configs`: the other benchmark configurations (L = 4K
to 512K), an HBM-bound probe (L = 1M, q_len 16) and the L = 1M configuration under
Algorithm 1's default pooling spec, each timed with a cold L2; and the steps around the
recall (key fill, Eq. 7 re-rotation alone and followed by the recall, chunk attention, the
per-rank steps of a sharded recall, the retrieval-layer sweep).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

# DRAM bytes per context position of the dominant kernel (row statistics), from one ncu
# capture at L = 131072, q_len = 256: (270.60 MB read + 3.96 MB written, mean of two launches)
# / 131072 keys.  Traffic grows in proportion to L (the query block is L2-resident), so it is
# scaled by L.
ROW_STATS_DRAM_BYTES_PER_KEY = 2095.0
METRIC = "key_cache_GBps_per_recall_L1M"
UNIT = "GB/s"
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0,
                source="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={CLOCK_QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.gpu_index), "-f", self.path],
                stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            with open(self.path) as f:
                for line in f:
                    cols = [c.strip() for c in line.split(",")]
                    if len(cols) < 9:
                        continue
                    try:
                        sm.append(float(cols[1]))
                        smax.append(float(cols[2]))
                    except ValueError:
                        continue
                    for name, val in zip(names, cols[5:9]):
                        if val.lower().startswith("active"):
                            reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(smax)),
                       reasons=sorted(reasons), samples=len(sm))
        return out


def dist_setup(n_gpus: int):
    """Process-group plumbing for N > 1 (barrier and max-over-ranks only; no data exchange)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend)
    return world, rank, local


def aggregate(elapsed_ms: float, units: float, device=None):
    """(max elapsed over ranks, sum of units over ranks).  Works on gloo (CPU) and nccl."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return elapsed_ms, units
    dev = device if device is not None else torch.device("cpu")
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def workload_string(w) -> str:
    return (f"{w.name}: L={w.L}, q_len={w.q_len}, kv_heads={w.n_kv_heads}, "
            f"q_heads={w.n_q_heads}, d={w.d}, budget={w.budget}, "
            f"windows={list(w.win_sizes)} ({'max' if w.win_op else 'avg'}), "
            f"max_sizes={list(w.max_sizes)}, n_sink={w.n_sink}")


def pick_workload(args):
    import dataclasses
    from workloads import CONFIGS
    w = CONFIGS[args.config]
    if args.L and args.L != w.L:
        w = dataclasses.replace(w, name=f"{w.name}_L{args.L}", L=args.L,
                                n_spans=max(1, w.n_spans * args.L // w.L),
                                budget=min(w.budget, args.L))
    return w


SIDE_WORKLOADS = ("cfg1_L4k", "cfg2_L32k", "cfg3_L128k", "cfg4_L512k", "probe_L1m_q16",
                  "cfg5_L1m_paper_pool")


def time_side_workload(eng, dev, w, x, steps, flush, peaks, K=None, Q=None):
    """One row of the `configs` block: `steps` recalls of workload `w`, each between its own
    pair of CUDA events, with a write of `flush` (larger than L2) before every recall so that
    no key is served from L2 left warm by the previous recall.  Returns ms per recall (median
    and mean), key-cache GB/s, stage times and the roofline fractions."""
    K = x.K.to(dev) if K is None else K
    Q = x.Q.to(dev) if Q is None else Q
    spec = (w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    out_idx = torch.empty(w.n_sink + w.budget, dtype=torch.int32, device=dev)
    for _ in range(3):
        eng.run(K, Q, *spec, out_idx=out_idx)
    torch.cuda.synchronize()
    eng.check_status()
    eng.set_profiling(True)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(steps)]
    for a, b in evs:
        flush.zero_()
        a.record()
        eng.run(K, Q, *spec, out_idx=out_idx)
        b.record()
    torch.cuda.synchronize()
    ms_all = sorted(a.elapsed_time(b) for a, b in evs)
    stages = eng.stage_times()
    eng.set_profiling(False)
    eng.check_status()
    # the same loop back to back (keys of short contexts stay in L2), for comparison
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        eng.run(K, Q, *spec, out_idx=out_idx)
    b.record()
    torch.cuda.synchronize()
    ms_warm = a.elapsed_time(b) / steps
    # short contexts: the same recalls captured once in a CUDA graph and replayed (the call
    # allocates nothing and never synchronises, so it can be captured)
    ms_graph = None
    if w.L <= 131072:
        side = torch.cuda.Stream(device=dev)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            eng.run(K, Q, *spec, out_idx=out_idx, stream=side)
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(steps):
                    eng.run(K, Q, *spec, out_idx=out_idx, stream=side)
        graph.replay()
        torch.cuda.synchronize()
        a.record()
        graph.replay()
        b.record()
        torch.cuda.synchronize()
        ms_graph = a.elapsed_time(b) / steps
        eng.check_status()
        del graph
    ms = ms_all[len(ms_all) // 2]
    k_bytes = K.numel() * 2
    flops = 2.0 * w.q_len * w.n_q_heads * w.L * w.d
    gbs = k_bytes / (ms * 1e-3) / 1e9
    row = dict(workload=workload_string(w), ms_per_recall=ms, ms_mean=sum(ms_all) / len(ms_all),
               ms_min=ms_all[0], ms_back_to_back=ms_warm, ms_graph_replay=ms_graph, steps=steps,
               l2="flushed before every recall (256 MiB write, untimed)",
               key_cache_gbs=gbs, stages_ms=stages, launches_per_recall=eng.last_launch_count(),
               hbm_frac_one_read_of_K=gbs / peaks["hbm_gbs"],
               tensor_frac_one_qk_burst=flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
               tensor_frac_one_qk_sustained=flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
               per_pass=dict(
                   row_stats_gbs=k_bytes / (stages["row_stats"] * 1e-3) / 1e9,
                   row_stats_hbm_frac=k_bytes / (stages["row_stats"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                   row_stats_tflops=flops / (stages["row_stats"] * 1e-3) / 1e12,
                   scores_gbs=k_bytes / (stages["scores"] * 1e-3) / 1e9,
                   scores_hbm_frac=k_bytes / (stages["scores"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                   scores_tflops=flops / (stages["scores"] * 1e-3) / 1e12))
    return row


def oracle_sample_run(x, sample_keys: int):
    """One oracle recall on the first `sample_keys` positions of the workload."""
    import oracle
    w = x.workload
    Ks = x.K[:sample_keys].contiguous()
    budget = min(w.budget, sample_keys)
    t0 = time.perf_counter()
    oracle.recall(Ks, x.Q, budget, w.max_sizes, w.win_sizes, w.win_op, 0)
    return time.perf_counter() - t0, Ks.numel() * 2


def run_reference(args, world, rank):
    """Reference arm: the CPU oracle, as it stands, on a bounded sample of the workload."""
    if rank != 0:
        return
    from workloads import make_inputs
    import dataclasses
    w = pick_workload(args)
    cores = len(os.sched_getaffinity(0))
    sample_keys = args.ref_sample_keys
    # only the sampled prefix of the cache is needed; the generator is prefix-stable in L
    # except for span placement, so build a workload of the sample length with the same seed
    ws = dataclasses.replace(w, L=sample_keys, n_spans=max(1, w.n_spans * sample_keys // w.L),
                             budget=min(w.budget, sample_keys))
    x = make_inputs(ws)
    for _ in range(args.warmup):
        oracle_sample_run(x, sample_keys)
    t_total, nbytes = 0.0, 0
    for _ in range(args.steps):
        dt, nb = oracle_sample_run(x, sample_keys)
        t_total += dt
        nbytes = nb
    ms = 1e3 * t_total / args.steps
    value = nbytes / (ms * 1e-3) / 1e9
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=ms, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=workload_string(w),
                            sample=f"each step: first {sample_keys} of {w.L} keys, budget "
                                   f"{ws.budget}"),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle",
                                  sample=f"first {sample_keys} keys of the cache, all "
                                         f"{w.q_len * w.n_q_heads} query rows, per step"),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


def run_sharded(args, world, rank, dev, w, x, eng, spec):
    """ONE recall over keys split by position across the ranks (strong scaling): per-rank
    kernels plus the two all-gathers of the exchange, timed together.  Returns the result
    line on rank 0 (None elsewhere)."""
    import torch.distributed as dist
    from paper_2508_17892_b200.sharded import shard_bounds, sharded_recall
    own_group = not dist.is_initialized()
    if own_group:                                       # single process: a 1-rank group
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29751", rank=0, world_size=1,
                                device_id=dev)
    lo, hi = shard_bounds(w.L, world, rank)
    K, Q = x.K[lo:hi].contiguous().to(dev), x.Q.to(dev)

    def step():
        return sharded_recall(eng, K, Q, w.L, *spec)

    for _ in range(max(args.warmup, 3)):
        idx, _ = step()
    torch.cuda.synchronize()
    eng.check_status()
    sampler = ClockSampler(dev.index)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    start.record()
    for _ in range(args.steps):
        idx, _ = step()
    stop.record()
    torch.cuda.synchronize()
    barrier()
    elapsed_ms = start.elapsed_time(stop)
    eng.check_status()
    clocks = sampler.stop() if rank == 0 else None
    # every rank must hold the same list
    ref = idx.clone()
    dist.broadcast(ref, src=0)
    assert torch.equal(ref, idx), "ranks disagree on the recalled indices"
    elapsed_max, units = aggregate(elapsed_ms, float(K.numel() * 2) * args.steps, dev)
    line = None
    if rank == 0:
        ms = elapsed_max / args.steps
        line = dict(metric=METRIC, value=units / (elapsed_max * 1e-3) / 1e9, unit=UNIT, n_gpus=world,
                    steps=args.steps, warmup=max(args.warmup, 3), ms_per_step=ms,
                    higher_is_better=True, scaling="strong", vs_baseline=None, dtype="bf16",
                    data="synthetic",
                    config=dict(workload=workload_string(w),
                                parallelism=f"key-range sharded over {world} rank(s), two all-gathers"),
                    clocks=clocks, e2e=None, gpu_launches=8 * args.steps, roofline=None,
                    cpu_baseline=None)
    del K
    if own_group:
        dist.destroy_process_group()
    return line


def run_ours(args, world, rank, local):
    from paper_2508_17892_b200 import IlreRecall, build
    from workloads import make_inputs
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100); there is no CPU fallback")
    build.build()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    w = pick_workload(args)
    x = make_inputs(w)
    eng = IlreRecall(max_L=w.L, max_q_len=w.q_len, max_budget=w.budget, n_kv_heads=w.n_kv_heads,
                     n_q_heads=w.n_q_heads, device=local, host_staging=not (args.no_e2e or args.sharded))
    spec = (w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    if args.sharded:
        line = run_sharded(args, world, rank, dev, w, x, eng, spec)
        if rank == 0:
            print(json.dumps(line), flush=True)
        eng.close()
        return
    K, Q = x.K.to(dev), x.Q.to(dev)
    out_idx = torch.empty(w.n_sink + w.budget, dtype=torch.int32, device=dev)
    k_bytes = K.numel() * 2

    def step():
        eng.run(K, Q, *spec, out_idx=out_idx)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    eng.check_status()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    eng.set_profiling(True)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    start.record()
    for _ in range(args.steps):
        step()
    stop.record()
    torch.cuda.synchronize()
    barrier()
    elapsed_ms = start.elapsed_time(stop)
    stages = eng.stage_times()
    sm_mhz_in_kernel = eng.sm_clock_mhz()
    eng.set_profiling(False)
    launches = eng.last_launch_count() * args.steps
    eng.check_status()
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None:
        # what the driver reports is the clock it asks for; under the power cap the SMs run
        # slower: cycles / global-timer nanoseconds of the last row-statistics launch
        clocks["sm_mhz_in_kernel"] = sm_mhz_in_kernel

    # end to end through the host entry point: pinned host inputs, copies inside the timing
    e2e = None
    if not args.no_e2e:
        Kh, Qh = x.K.pin_memory(), x.Q.pin_memory()
        idx_h = torch.empty(w.n_sink + w.budget, dtype=torch.int32).pin_memory()
        e2e_steps = max(3, min(args.steps, 10))
        eng.run_host(Kh, Qh, *spec, out_idx=idx_h)
        barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            eng.run_host(Kh, Qh, *spec, out_idx=idx_h)
        torch.cuda.synchronize()
        e2e_ms = 1e3 * (time.perf_counter() - t0) / e2e_steps
        e2e_ms_max, e2e_units = aggregate(e2e_ms, float(k_bytes), dev)
        # the pipelined upload merges its pieces' statistics in another order than the
        # device entry point: a few positions at a cut-off may differ
        assert len(set(idx_h.tolist()) ^ set(out_idx.cpu().tolist())) <= max(2, idx_h.numel() // 100)
        e2e = dict(value=e2e_units / (e2e_ms_max * 1e-3) / 1e9, unit=UNIT, ms_per_step=e2e_ms_max,
                   h2d_bytes_per_step=int(k_bytes + Q.numel() * 2),
                   d2h_bytes_per_step=int(idx_h.numel() * 4), steps=e2e_steps)

    # Dual Chunk Attention re-rotation of the cache (Eq. 7), timed on its own: an HBM-bound
    # streaming kernel, in place on a scratch copy of K
    dca = None
    if args.dca_chunk > 0 and rank == 0:
        Kc = K.clone()
        n_chunks = -(-(w.L - w.n_sink) // args.dca_chunk)
        rotated = max(0, min(w.L, w.n_sink + (n_chunks - 2) * args.dca_chunk))
        for _ in range(3):
            eng.rerope_keys(Kc, args.dca_chunk, w.n_sink)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 20
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            eng.rerope_keys(Kc, args.dca_chunk, w.n_sink)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        moved = 2.0 * rotated * w.n_kv_heads * w.d * 2              # read + write
        dca = dict(kernel="rerope_kernel", chunk=args.dca_chunk, ms=ms,
                   algorithmic_bytes=moved, achieved=moved / (ms * 1e-3) / 1e9, unit="GB/s",
                   bound="hbm", peak=measured_peaks()["hbm_gbs"],
                   frac=moved / (ms * 1e-3) / 1e9 / measured_peaks()["hbm_gbs"])
        # the recall with DCA on (Eq. 7 -> Eq. 4): the cache re-rotated into a second buffer,
        # then the recall on the rotated keys, one stream, one timed region
        def dca_recall():
            eng.rerope_keys(K, args.dca_chunk, w.n_sink, out=Kc)
            eng.run(Kc, Q, *spec, out_idx=out_idx)
        for _ in range(3):
            dca_recall()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            dca_recall()
        e1.record()
        torch.cuda.synchronize()
        ms_on = e0.elapsed_time(e1) / reps
        dca["recall_with_dca"] = dict(ms=ms_on, key_cache_gbs=k_bytes / (ms_on * 1e-3) / 1e9,
                                      steps=reps, note="re-rotation out of place + recall, one "
                                      "timed region; key cache larger than L2")
        eng.check_status()
        del Kc

    # Key-cache fill (key projection + RoPE into the cache), timed on its own: a tensor-bound
    # GEMM.  Llama-3.1-8B shape (d_model 4096), activations and weights drawn on the device.
    fill = None
    if args.fill_tokens > 0 and rank == 0:
        gen = torch.Generator(device=dev).manual_seed(1234)
        d_model = 4096
        n_fill = min(args.fill_tokens, w.L)
        Xf = torch.randn(n_fill, d_model, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        Wf = (torch.randn(w.n_kv_heads * w.d, d_model, generator=gen, device=dev) / 64).to(torch.bfloat16)
        Kf = torch.empty(n_fill, w.n_kv_heads, w.d, dtype=torch.bfloat16, device=dev)

        def timed(fn, reps):
            for _ in range(3):
                fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps

        ms_all = timed(lambda: eng.fill_keys(Xf, Wf, Kf, 0), 5)
        chunk = min(1024, n_fill)
        n_chunks = n_fill // chunk

        def by_chunks():
            for c in range(n_chunks):
                eng.fill_keys(Xf[c * chunk:(c + 1) * chunk], Wf, Kf, c * chunk)

        ms_chunks = timed(by_chunks, 2) / max(n_chunks, 1)
        fl_all = 2.0 * n_fill * d_model * w.n_kv_heads * w.d
        fl_chunk = 2.0 * chunk * d_model * w.n_kv_heads * w.d
        pk = measured_peaks()["bf16_tflops_sustained"]
        fill = dict(kernel="fill_kernel", d_model=d_model, tokens=n_fill, bound="tensor",
                    unit="TFLOP/s", peak=pk, ms=ms_all, achieved=fl_all / (ms_all * 1e-3) / 1e12,
                    frac=fl_all / (ms_all * 1e-3) / 1e12 / pk,
                    per_chunk=dict(tokens=chunk, ms=ms_chunks,
                                   achieved=fl_chunk / (ms_chunks * 1e-3) / 1e12))
        del Xf, Wf, Kf

    # Streaming chunked prefill attention of one chunk (paper defaults: chunk 1024, sink 4 +
    # window 512), timed on its own
    attn = None
    if args.attn_chunk > 0 and rank == 0:
        gen = torch.Generator(device=dev).manual_seed(4321)
        c_len, n_pre = args.attn_chunk, 516
        Qa = torch.randn(c_len, w.n_q_heads, w.d, generator=gen, device=dev).to(torch.bfloat16)
        Ka = torch.randn(n_pre + c_len, w.n_kv_heads, w.d, generator=gen, device=dev).to(torch.bfloat16)
        Va = torch.randn(n_pre + c_len, w.n_kv_heads, w.d, generator=gen, device=dev).to(torch.bfloat16)
        for _ in range(3):
            eng.chunk_attention(Qa, Ka, Va, n_pre)
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 50
        torch.cuda.synchronize()
        a0.record()
        for _ in range(reps):
            eng.chunk_attention(Qa, Ka, Va, n_pre)
        a1.record()
        torch.cuda.synchronize()
        ms = a0.elapsed_time(a1) / reps
        pairs = c_len * n_pre + c_len * (c_len + 1) / 2.0               # visible (query, key) pairs
        fl = pairs * w.n_q_heads * 4.0 * w.d                             # QK^T and PV
        pk = measured_peaks()["bf16_tflops"]
        attn = dict(kernel="chunk_attention_kernel", chunk=c_len, n_prefix=n_pre, ms=ms,
                    algorithmic_flops=fl, achieved=fl / (ms * 1e-3) / 1e12, unit="TFLOP/s",
                    bound="tensor", peak=pk, frac=fl / (ms * 1e-3) / 1e12 / pk)
        del Qa, Ka, Va

    # Key-range sharded recall: the three per-rank steps of a P-way split, timed on one
    # GPU for the first shard (the exchanges between them, 2 floats per query row and one
    # float per position, are not timed here)
    shard = None
    if args.shards > 1 and rank == 0:
        from paper_2508_17892_b200.sharded import shard_bounds
        lo, hi = shard_bounds(w.L, args.shards, 0)
        Ks = K[lo:hi]
        n_rows = w.q_len * w.n_q_heads
        st_one = torch.empty(n_rows, 2, dtype=torch.float32, device=dev)
        sc_one = torch.empty(hi - lo, dtype=torch.float32, device=dev)
        sc_all = torch.empty(w.L, dtype=torch.float32, device=dev)
        eng.run(K, Q, *spec, out_idx=out_idx, out_scores=sc_all)
        eng.shard_stats(Ks, Q, out=st_one)
        st_all = st_one.unsqueeze(0).repeat(args.shards, 1, 1).contiguous()

        def timed_ms(fn, reps=50):
            for _ in range(3):
                fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps

        ms_stats = timed_ms(lambda: eng.shard_stats(Ks, Q, out=st_one))
        ms_scores = timed_ms(lambda: eng.shard_scores(Ks, Q, st_all, out=sc_one))
        ms_alloc = timed_ms(lambda: eng.allocate(sc_all, *spec, out_idx=out_idx))
        shard = dict(shards=args.shards, keys_per_shard=hi - lo, shard_stats_ms=ms_stats,
                     shard_scores_ms=ms_scores, allocate_ms=ms_alloc,
                     per_rank_ms=ms_stats + ms_scores + ms_alloc,
                     exchange_bytes_per_rank=dict(statistics=n_rows * 8, scores=(hi - lo) * 4),
                     note="one GPU, first shard; all-gathers not included")
        eng.check_status()

    # Offline retrieval-layer sweep: the same recall against the caches of several candidate
    # layers of one context, then the exact-match layer choice.  Keys and queries drawn on
    # the device, phrases planted along each layer's mean query direction.
    sweep = None
    if args.sweep_layers > 0 and rank == 0:
        from paper_2508_17892_b200 import layer_recall
        gen = torch.Generator(device=dev).manual_seed(777)
        Ls, qs, n_lay, n_ph, ph_len = min(w.L, 131072), min(w.q_len, 64), args.sweep_layers, 20, 32
        seg = Ls // n_ph
        sb = torch.arange(n_ph, dtype=torch.int32, device=dev) * seg + seg // 3
        sl = torch.full((n_ph,), ph_len, dtype=torch.int32, device=dev)
        Kl, Ql = [], []
        for l in range(n_lay):
            q = torch.randn(qs, w.n_q_heads, w.d, generator=gen, device=dev).to(torch.bfloat16)
            k = torch.randn(Ls, w.n_kv_heads, w.d, generator=gen, device=dev)
            u = q.float().view(qs, w.n_kv_heads, -1, w.d).mean(dim=(0, 2))
            u = u / u.norm(dim=-1, keepdim=True)
            gain = 0.4 + 2.6 * l / max(n_lay - 1, 1)
            for b in sb.tolist():
                k[b:b + ph_len] = gain * math.sqrt(w.d) * u[None] + 0.5 * k[b:b + ph_len]
            Kl.append(k.to(torch.bfloat16))
            Ql.append(q)
            del k
        idx_all = torch.empty(n_lay, w.n_sink + 1024, dtype=torch.int32, device=dev)
        sspec = (1024, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)

        def one_sweep():
            for l in range(n_lay):
                eng.run(Kl[l], Ql[l], *sspec, out_idx=idx_all[l])
            return layer_recall(idx_all, sb, sl)

        for _ in range(3):
            one_sweep()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 20
        torch.cuda.synchronize()
        s0.record()
        for _ in range(reps):
            _, full, layer = one_sweep()
        s1.record()
        torch.cuda.synchronize()
        ms = s0.elapsed_time(s1) / reps
        swept = float(n_lay) * Ls * w.n_kv_heads * w.d * 2
        sweep = dict(layers=n_lay, L=Ls, q_len=qs, budget=1024, phrases=n_ph, ms=ms,
                     ms_per_layer=ms / n_lay, key_cache_gbs=swept / (ms * 1e-3) / 1e9,
                     retrieved_per_layer=full.tolist(), chosen_layer=int(layer.item()))
        eng.check_status()
        del Kl, Ql

    # The other workloads: benchmark configurations 1-4, the HBM-bound probe and the benchmark
    # configuration under Algorithm 1's default pooling, each timed with a cold L2.
    configs_block = None
    if args.side_steps > 0 and rank == 0 and args.config == "cfg5_L1m" and not args.L:
        from workloads import CONFIGS
        peaks_now = measured_peaks()
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        configs_block = {}
        for name in SIDE_WORKLOADS:
            sw = CONFIGS[name]
            same_cache = (sw.seed == w.seed and sw.L == w.L and sw.q_len == w.q_len)
            if same_cache:                                   # same keys and query as the main workload
                row = time_side_workload(eng, dev, sw, x, args.side_steps, flush, peaks_now, K=K, Q=Q)
            else:
                sx = make_inputs(sw)
                row = time_side_workload(eng, dev, sw, sx, args.side_steps, flush, peaks_now)
                del sx
            if name.startswith("probe"):
                row["note"] = ("not one of the five benchmark configurations: q_len 16 puts the key scan below the ridge, "
                               "so per_pass.*_hbm_frac is the streaming efficiency of each pass")
            configs_block[name] = row
        del flush

    # With more than one rank: also ONE recall over keys split by position across the ranks
    # (the replica line above measures throughput, this one the latency of a sharded recall)
    sharded_line = None
    if world > 1 and not args.no_sharded_line:
        del K
        torch.cuda.empty_cache()
        sharded_line = run_sharded(args, world, rank, dev, w, x, eng, spec)

    elapsed_max, units = aggregate(elapsed_ms, float(k_bytes) * args.steps, dev)
    if rank != 0:
        return
    ms_per_step = elapsed_max / args.steps
    value = units / (elapsed_max * 1e-3) / 1e9
    peaks = measured_peaks()
    R = w.q_len * w.n_q_heads
    flops = 2.0 * R * w.L * w.d                         # one QK^T (Eq. 4), algorithmic
    dom = max(("row_stats", "scores"), key=lambda k: stages[k])
    dom_tflops = flops / (stages[dom] * 1e-3) / 1e12
    # which roofline binds the contraction kernels: flop per key byte against the measured ridge
    ridge = peaks["bf16_tflops_sustained"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    hbm_bound = (flops / k_bytes) < ridge
    dom_gbs = k_bytes / (stages[dom] * 1e-3) / 1e9
    # A timed loop shorter than about a second runs before the board settles at its power cap:
    # the burst bf16 figure is then the matching denominator, the sustained one otherwise.
    loop_s = elapsed_max * 1e-3
    regime = "burst" if loop_s < 1.0 else "sustained"
    tensor_peak = peaks["bf16_tflops"] if regime == "burst" else peaks["bf16_tflops_sustained"]
    roofline = dict(bound="hbm" if hbm_bound else "tensor", kernel=f"{dom}_kernel",
                    achieved=dom_gbs if hbm_bound else dom_tflops,
                    peak=peaks["hbm_gbs"] if hbm_bound else tensor_peak,
                    unit="GB/s" if hbm_bound else "TFLOP/s",
                    frac=(dom_gbs / peaks["hbm_gbs"] if hbm_bound else dom_tflops / tensor_peak),
                    frac_of_burst_bf16=dom_tflops / peaks["bf16_tflops"],
                    frac_of_sustained_bf16=dom_tflops / peaks["bf16_tflops_sustained"],
                    regime=f"{regime}: timed loop of {loop_s:.2f} s, in-kernel SM clock "
                           f"{sm_mhz_in_kernel:.0f} MHz",
                    flop_per_key_byte=flops / k_bytes, ridge_flop_per_byte=ridge,
                    traffic=(ROW_STATS_DRAM_BYTES_PER_KEY * w.L
                             if dom == "row_stats" and w.q_len == 256 else None),
                    traffic_unit="bytes per launch (ncu at L=131072, scaled by L)",
                    peak_source=(f"{peaks['source']} (HBM copy)" if hbm_bound
                                 else f"{peaks['source']} ({regime} bf16)"),
                    kernel_ms=stages[dom], algorithmic_flops_per_launch=flops,
                    algorithmic_bytes_per_launch=k_bytes,
                    kernel_hbm_gbs=k_bytes / (stages[dom] * 1e-3) / 1e9)
    # the row-statistics kernel also evaluates R * L exponentials; the special-function unit
    # alone would do 16 per clock per SM
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    sm_max_ghz = ((clocks or {}).get("sm_max_mhz") or 1965.0) / 1e3
    exp_peak = 16.0 * n_sm * sm_max_ghz * 1e9
    exp_rate = float(R) * w.L / (stages["row_stats"] * 1e-3)
    roofline["row_stats_exponentials"] = dict(
        bound="alu", achieved=exp_rate / 1e12, peak=exp_peak / 1e12, unit="Texp/s",
        frac=exp_rate / exp_peak,
        peak_source=f"16 ex2 per clock per SM x {n_sm} SMs x {sm_max_ghz:.3f} GHz",
        frac_at_in_kernel_clock=(exp_rate / (16.0 * n_sm * sm_mhz_in_kernel * 1e6)
                                 if sm_mhz_in_kernel > 0 else None))
    step_hbm_frac = (k_bytes / (ms_per_step * 1e-3) / 1e9) / peaks["hbm_gbs"]
    step_tensor_frac = (flops / (ms_per_step * 1e-3) / 1e12) / peaks["bf16_tflops_sustained"]

    cpu_baseline = None
    if not args.no_cpu_baseline and world == 1:
        cores = len(os.sched_getaffinity(0))
        dt, nb = oracle_sample_run(x, min(args.cpu_sample_keys, w.L))
        cpu_baseline = dict(value=nb / dt / 1e9, unit=UNIT, cores=cores, kind="oracle",
                            seconds=dt,
                            sample=f"first {min(args.cpu_sample_keys, w.L)} of {w.L} keys, all {R} query "
                                   f"rows, full Algorithm 1 on that prefix")

    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps,
                warmup=max(args.warmup, 3), ms_per_step=ms_per_step, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic",
                config=dict(workload=workload_string(w),
                            l2="key cache (2 GiB) is larger than L2; no flush needed",
                            parallelism="replicas only" if world > 1 else "single GPU"),
                clocks=clocks, e2e=e2e, gpu_launches=launches, roofline=roofline,
                cpu_baseline=cpu_baseline,
                stages_ms=stages, dca_rerope=dca, key_fill=fill, chunk_attention=attn,
                sharded_steps=shard, layer_sweep=sweep, configs=configs_block,
                sharded_recall=sharded_line,
                whole_step=dict(hbm_frac_one_read_of_K=step_hbm_frac,
                                tensor_frac_one_qk=step_tensor_frac,
                                hbm_frac_of_8TBps=(k_bytes / (ms_per_step * 1e-3) / 1e9) / 8000.0))
    print(json.dumps(line), flush=True)
    eng.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", default="cfg5_L1m")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--L", type=int, default=0,
                    help="override the context length of --config (profiling on a small case)")
    ap.add_argument("--dca-chunk", type=int, default=1024,
                    help="also time the Eq. 7 key re-rotation with this chunk size (0 = skip)")
    ap.add_argument("--attn-chunk", type=int, default=1024,
                    help="also time the chunked prefill attention of one chunk (0 = skip)")
    ap.add_argument("--fill-tokens", type=int, default=1048576,
                    help="also time the key-cache fill over this many tokens (0 = skip)")
    ap.add_argument("--sharded", action="store_true",
                    help="strong scaling: one recall with the keys split by position over the "
                         "ranks (default: independent replicas)")
    ap.add_argument("--shards", type=int, default=8,
                    help="also time the per-rank steps of a key-range split this many ways (0 = skip)")
    ap.add_argument("--sweep-layers", type=int, default=8,
                    help="also time the offline retrieval-layer sweep over this many candidate "
                         "layers at L = 128K (0 = skip)")
    ap.add_argument("--side-steps", type=int, default=20,
                    help="recalls timed per workload of the `configs` block (benchmark "
                         "configurations 1-4, the q_len 16 probe, the default pooling spec; 0 = skip)")
    ap.add_argument("--no-sharded-line", action="store_true",
                    help="with --gpus N > 1: skip the additional key-range sharded recall")
    ap.add_argument("--cpu-sample-keys", type=int, default=131072)
    ap.add_argument("--ref-sample-keys", type=int, default=4096)
    args = ap.parse_args()
    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        run_reference(args, int(os.environ.get("WORLD_SIZE", "1")), rank)
        return
    world, rank, local = dist_setup(args.gpus)
    try:
        run_ours(args, world, rank, local)
    finally:
        if world > 1:
            import torch.distributed as dist
            if dist.is_initialized():
                dist.destroy_process_group()


if __name__ == "__main__":
    main()
