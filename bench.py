#!/usr/bin/env python
"""Benchmark of the ShadowSync hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--workload medium] [--impl reference]

One "step" is one pass of the whole hot path over one batch per replica: every one of the R replicas
runs embedding forward, MLP forward, MLP backward + dense Adagrad and embedding backward + row-wise
Adagrad on its own high-priority stream, while the shadow loop keeps enqueuing the synchronisation
kernel (S-EASGD / S-MA / S-BMUF as the workload says) on the lowest-priority stream.
`value` = training examples per second with the shadow sync on, inputs resident in HBM.
With N > 1 (launched under torchrun) every rank runs the same job on its own GPU: the path does not
shard across GPUs, so these are independent replicas of the job and the values add (weak scaling).

The K-step region is repeated (sync off and sync on alternating) until at least a second has been timed, and the
median region gives `value`; the spread is reported beside it.  The same line carries, as legs, the other
single-GPU workloads (`workloads.medium_bmuf`, `workloads.large`) and the sync-kernel sweep running concurrently with
this training (`sync.concurrent_sweep`).

`--impl reference` times the CPU oracle (oracle/, test infrastructure) on a bounded sample of the same
workload on the host cores; it is deliberately slow and is a reported baseline, not a target.
`--plain` runs a few un-captured replica steps (every kernel its own launch) for profilers.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "training examples/sec at 1 B200 with shadow sync on; sync HBM GB/s vs peak"
UNIT = "examples/s"
RING = 8            # pre-generated batches per replica, cycled through

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from one ncu capture of the kernel, valid
# for the named workload and for exactly the sources whose hashes are listed: once one of them changes the figure is
# reported as null until the counters are taken again.
NCU_TRAFFIC = {
    "embbag_fwd_kernel": {"workload": "medium", "bytes_per_launch": 60735488, "launches_captured": 1,
        "sources": {"embbag.cu": "01f2a02f35307de16d0a5d128e477c12fd20889ec1001c7ea1e48540166ef266"}},
    "gemm_tc_kernel": {"workload": "medium", "bytes_per_launch": 13713152, "launches_captured": 2,
        "tensor_pipe_active_pct": {"forward flow": 22.0, "backward flow": 26.0},   # of peak, on the SMs it runs on
        "sources": {"gemm_tc.cu": "324cae2590c1e98d6b70ac25e93c69b0a80f94fce0502b293775aef07ef70fcf", "gemm.cuh": "4d6c8c9e6e5d6074538581dc140b390c97ecf03d2981f64d8c6141a64a63af34", "mlp.cu": "b822041d4f8cd57822dcb356f9b6c1cc6c848a25a244fe4ae0e58143ebfa5b2a", "mlp_plan.cuh": "5f73399683bba8691505ec8d1e6cbb83fe39a5e25044ee8f2a9823f698f03d9a"}},
    "window_apply_kernel": {"workload": "medium", "bytes_per_launch": 123957760, "launches_captured": 1,
        "sources": {"embbag.cu": "01f2a02f35307de16d0a5d128e477c12fd20889ec1001c7ea1e48540166ef266"}},
    "combine_rows_kernel": {"workload": "medium", "bytes_per_launch": 12092672, "launches_captured": 1,
        "sources": {"embbag.cu": "01f2a02f35307de16d0a5d128e477c12fd20889ec1001c7ea1e48540166ef266"}},
}


def ncu_traffic(kernel, workload, field="bytes_per_launch"):
    """Bytes per launch (or another field) from the stored ncu capture, or None when it does not cover this
    kernel, this workload or the current sources."""
    import hashlib
    e = NCU_TRAFFIC.get(kernel)
    if e is None or e["workload"] != workload:
        return None
    csrc = os.path.join(os.path.dirname(os.path.abspath(__file__)), "paper_2003_03477_b200", "csrc")
    for name, want in e["sources"].items():
        try:
            with open(os.path.join(csrc, name), "rb") as f:
                if hashlib.sha256(f.read()).hexdigest() != want:
                    return None
        except OSError:
            return None
    return e.get(field)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"], bf16_tflops_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index, self.proc, self.lines = gpu_index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu_index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm),
                "sm_mhz_min": min(sm) if sm else None, "sm_mhz_highest_seen": max(sm) if sm else None,
                "sampled": "nvidia-smi every 100 ms across all repeated timed regions"}


# ----------------------------------------------------------------------------------------------
def build_job(cfg, device, workers=1, ring=RING):
    """Tables, replicas and a ring of device-resident batches for one GPU."""
    import torch
    from paper_2003_03477_b200 import binding as ss, synth, trainer
    tables = trainer.device_tables(cfg, device)
    spec = ss.MlpSpec(cfg.bottom, cfg.top, cfg.bf16)
    w0 = torch.from_numpy(trainer.pack_params(spec, synth.initial_weights(cfg))).to(device)
    host = [[synth.make_batch(cfg, r, t) for t in range(ring)] for r in range(cfg.R)]
    max_L = max(b.L for bs in host for b in bs)
    model = trainer.Model(cfg.T, cfg.N, cfg.D, cfg.B, cfg.bottom, cfg.top, cfg.bf16, cfg.R, w0, tables, cfg.lr, cfg.eps,
                          max_L=max_L, device=device, workers=workers)
    dev = [[trainer.DeviceBatch(b.indices, b.offsets, b.dense, b.labels, device) for b in bs] for bs in host]
    return model, host, dev, max_L


def capture_graphs(model, dev):
    """One CUDA graph per (replica, ring slot): the four calls of a replica step."""
    import torch
    graphs = []
    for r, rep in enumerate(model.replicas):
        row = []
        for slot, b in enumerate(dev[r]):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=rep.stream):
                model.step(r, b, stream=rep.stream)
            row.append(g)
        graphs.append(row)
    return graphs


STEPS_AHEAD = 16   # set from --steps-ahead


def run_steps(model, graphs, first_step, n_steps, paced=None):
    """Replays the replicas' step graphs.  The host keeps at most STEPS_AHEAD steps of a replica queued on the device
    (it waits for the event of step t - STEPS_AHEAD before it enqueues step t; 0 = no bound).  An unbounded queue
    changes nothing for training but makes the shadow thread's launches wait behind thousands of queued graph
    launches: measured 76 sync rounds/s (a pass every 25 steps) unbounded, 312/s (every 6 steps) with 16, 1416/s
    (every 1.3 steps, training -1 %) with 4.
    paced = (every, fn): the paced form of the background sync (one pass after each round of `every` local steps):
    fn() enqueues a pass on the low-priority sync stream, with no dependency on the training streams.
    Returns the number of paced passes enqueued."""
    import torch
    ring = len(graphs[0])
    evs = [[] for _ in model.replicas]
    passes = 0
    for t in range(first_step, first_step + n_steps):
        for r, rep in enumerate(model.replicas):
            if STEPS_AHEAD and len(evs[r]) >= STEPS_AHEAD:
                evs[r].pop(0).synchronize()
            with torch.cuda.stream(rep.stream):
                graphs[r][t % ring].replay()
                if STEPS_AHEAD:
                    e = torch.cuda.Event()
                    e.record(rep.stream)
                    evs[r].append(e)
        if paced and (t - first_step + 1) % paced[0] == 0:
            paced[1]()
            passes += 1
    return passes


def timed_region(model, graphs, first_step, n_steps, paced=None):
    """Device time of n_steps steps over all replica streams (ms), and the paced sync passes enqueued in it."""
    import torch
    main = torch.cuda.current_stream()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record(main)
    for rep in model.replicas:
        rep.stream.wait_event(start)
    passes = run_steps(model, graphs, first_step, n_steps, paced)
    for rep in model.replicas:
        e = torch.cuda.Event()
        e.record(rep.stream)
        main.wait_event(e)
    stop.record(main)
    stop.synchronize()
    return start.elapsed_time(stop), passes


def reduce_over_ranks(ms_list, examples, device):
    """Max over ranks of each timed region (ms) and the sum over ranks of the examples processed.
    Each rank runs an independent copy of the job (the path does not shard across GPUs)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(ms_list), examples
    t = torch.tensor(list(ms_list), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([examples], dtype=torch.int64, device=device)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return [float(x) for x in t], int(n[0])


def region_stats(ms):
    """Median, extremes and count of repeated timed regions."""
    return {"median_ms": statistics.median(ms), "min_ms": min(ms), "max_ms": max(ms), "repeats": len(ms)}


def repeats_for(region_ms, min_total_s, min_reps, max_reps):
    """How often the K-step region is repeated so that at least min_total_s are timed (clocks settle, and a sync
    loss of a fraction of a per cent is above the spread)."""
    need = int(np.ceil(min_total_s * 1e3 / max(region_ms, 1e-3)))
    return max(min_reps, min(max_reps, need))


def sync_args(cfg):
    return dict(rule=cfg.sync, alpha=cfg.alpha, eta=cfg.eta, mu=cfg.mu)


def time_kernel_call(fn, stream, reps):
    """Average device time (ms) of a library call that is exactly one kernel, from CUDA events on its stream."""
    import torch
    evs = []
    for i in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn(i)
        b.record(stream)
        evs.append((a, b))
    stream.synchronize()
    return sum(a.elapsed_time(b) for a, b in evs) / reps


class Barrier:
    def __init__(self, world):
        self.world = world

    def __call__(self):
        import torch
        import torch.distributed as dist
        torch.cuda.synchronize()
        if self.world > 1:
            dist.barrier()
            torch.cuda.synchronize()


def measure_training(model, graphs, cfg, K, W, barrier, device, args, sampler=None):
    """Sync-off and sync-on regions of exactly K steps each, alternating, repeated until args.min_seconds have been
    timed per arm (at least args.min_repeats times).  Background sync: the native shadow thread, paused (drained)
    during the off regions so that the pass count of an on region is the number of passes that completed in it; for a
    workload with a paced sync (one pass after each round of k local steps) the host enqueues that pass on the
    low-priority sync stream instead.  Returns a dict of lists (max over ranks per region) and totals."""
    import torch
    from paper_2003_03477_b200 import trainer
    paced = (cfg.sync_every, lambda: model.sync(**sync_args(cfg))) if cfg.sync_every else None
    loop = None
    if paced is None:
        loop = trainer.ShadowLoop(model, max_in_flight=args.sync_in_flight, pause_s=args.sync_pause, **sync_args(cfg)).start()
        loop.pause()
    run_steps(model, graphs, 0, W)
    barrier()
    # one probe region sizes the repeat count (every rank takes the same count: the max over ranks decides)
    probe, _ = timed_region(model, graphs, W, K)
    (probe,), _ = reduce_over_ranks([probe], 0, device)
    reps = repeats_for(probe, args.min_seconds, args.min_repeats, 400)
    ms_on, ms_off, rounds = [], [], []
    if sampler is not None:
        sampler.start()
    for i in range(reps):
        barrier()
        t_off, _ = timed_region(model, graphs, W + i * K, K)
        barrier()
        if loop is not None:
            r0 = loop.rounds
            loop.resume()
            t_on, _ = timed_region(model, graphs, W + i * K, K)
            r1 = loop.pause()
            rounds.append(r1 - r0)
        else:
            t_on, n_pass = timed_region(model, graphs, W + i * K, K, paced)
            model.sync_stream.synchronize()
            rounds.append(n_pass)
        ms_on.append(t_on)
        ms_off.append(t_off)
    clocks = sampler.stop() if sampler is not None else None
    barrier()
    if loop is not None:
        loop.stop()
    torch.cuda.synchronize()
    both, examples = reduce_over_ranks(ms_on + ms_off, cfg.R * cfg.B * K, device)
    return {"ms_on": both[:reps], "ms_off": both[reps:], "rounds": rounds, "examples_per_region": examples,
            "clocks": clocks, "paced": paced is not None}


def summarise_training(m, K):
    """examples/s from the median region of each arm, the spread, the sync loss and the sync rate."""
    on, off = region_stats(m["ms_on"]), region_stats(m["ms_off"])
    ex = m["examples_per_region"]
    value, value_off = ex / (on["median_ms"] * 1e-3), ex / (off["median_ms"] * 1e-3)
    total_rounds, total_s = sum(m["rounds"]), sum(m["ms_on"]) * 1e-3
    # loss from the medians, and the median of the per-pair losses (regions alternate, so a pair shares its clocks)
    pair = [100.0 * (1.0 - b / a) for a, b in zip(m["ms_on"], m["ms_off"])]
    return value, on, {
        "rounds_per_s": total_rounds / total_s if total_s > 0 else None,
        "avg_sync_gap_steps": (K * len(m["ms_on"]) / total_rounds) if total_rounds else None,
        "passes_counted": total_rounds, "counting": "passes completed inside the sync-on regions (the shadow thread is "
        "paused and drained outside them)" if not m["paced"] else "one pass enqueued on the sync stream per round of local steps",
        "examples_per_s_sync_off": value_off,
        "throughput_loss_pct": 100.0 * (1.0 - value / value_off),
        "throughput_loss_pct_median_of_pairs": statistics.median(pair),
        "regions_sync_on": on, "regions_sync_off": off,
        "examples_per_s_sync_on_best_region": ex / (on["min_ms"] * 1e-3),
    }


def workload_text(cfg):
    return (f"{cfg.name}: R={cfg.R} T={cfg.T} N={cfg.N} D={cfg.D} B={cfg.B} "
            f"bottom={'-'.join(map(str, cfg.bottom))} top={'-'.join(map(str, cfg.top))} "
            f"sync={cfg.sync} alpha={cfg.alpha} "
            + (f"one background pass per {cfg.sync_every} local steps" if cfg.sync_every else "background, continuous"))


def bench_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2003_03477_b200 import binding as ss, synth, trainer

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    cfg = synth.CONFIGS[args.workload]
    if args.replicas:
        cfg = synth.scaled(cfg, R=args.replicas)
    K, W = args.steps, max(args.warmup, 3)
    peaks = measured_peaks()
    barrier = Barrier(world)

    ss.ss_mlp_set_flow_ctas(args.flow_ctas if args.flow_ctas else -1)
    model, host, dev, max_L = build_job(cfg, device, workers=max(1, args.workers))
    # un-captured warm-up: first-use set-up inside the library (function attributes, symbol addresses)
    for r in range(cfg.R):
        model.step(r, dev[r][0])
    model.sync(**sync_args(cfg))
    torch.cuda.synchronize()
    graphs = capture_graphs(model, dev)

    m = measure_training(model, graphs, cfg, K, W, barrier, device, args, sampler=ClockSampler(local))
    value, on, sync_info = summarise_training(m, K)
    clocks = m["clocks"]
    # ---- foreground variant (the paper's FR-* baselines): the sync pass inside the training loop every k steps
    ms_fg = None
    if args.foreground > 0:
        def fg_region(n_steps):
            for t0 in range(0, n_steps, args.foreground):
                run_steps(model, graphs, W + t0, min(args.foreground, n_steps - t0))
                model.foreground_sync(**sync_args(cfg))
        fg_region(W)
        barrier()
        main = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(main)
        for rep in model.replicas:
            rep.stream.wait_event(e0)
        fg_region(K)
        for rep in model.replicas:
            e = torch.cuda.Event()
            e.record(rep.stream)
            main.wait_event(e)
        e1.record(main)
        e1.synchronize()
        ms_fg = e0.elapsed_time(e1)
    # ---- intra-trainer Hogwild: m workers per replica, each on its own batches, sharing the replica's parameters
    ms_hw = None
    if args.workers > 1:
        mw = args.workers
        for r in range(cfg.R):
            for k in range(1, mw):
                model.step(r, dev[r][k % RING], worker=k)
        torch.cuda.synchronize()
        wg = []
        for r in range(cfg.R):
            per_worker = []
            for k in range(mw):
                wk, row = model.workers[r][k], []
                for slot in range(RING):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=wk.stream):
                        model.step(r, dev[r][(slot + 3 * k) % RING], stream=wk.stream, worker=k)
                    row.append(g)
                per_worker.append(row)
            wg.append(per_worker)

        def hw_steps(first, n):
            for t in range(first, first + n):
                for r in range(cfg.R):
                    for k in range(mw):
                        with torch.cuda.stream(model.workers[r][k].stream):
                            wg[r][k][t % RING].replay()
        hw_steps(0, W)
        barrier()
        main = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(main)
        for ws_ in model.workers:
            for wk in ws_:
                wk.stream.wait_event(e0)
        hw_steps(W, K)
        for ws_ in model.workers:
            for wk in ws_:
                e = torch.cuda.Event()
                e.record(wk.stream)
                main.wait_event(e)
        e1.record(main)
        e1.synchronize()
        ms_hw = e0.elapsed_time(e1)
    status = model.status()

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": on["median_ms"] / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.bf16 else "f32", "data": "synthetic",
        "config": {"workload": workload_text(cfg),
                   "l2": f"inputs larger than L2: tables {cfg.T * cfg.N * cfg.D * 4 / 1e9:.1f} GB gathered by skewed "
                         f"indices, {RING} rotating batches per replica",
                   "multi_gpu": "replicas only (no cross-GPU exchange on this path)",
                   "steps_ahead": STEPS_AHEAD,
                   "timing": f"CUDA events around exactly {K} steps, barrier + synchronise on both sides, max over "
                             f"ranks; the region is repeated {on['repeats']} times (sync off / on alternating) and "
                             f"value is examples / median region"},
        "clocks": clocks,
        "status_word": status,
    }
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- extra measurements on rank 0 ---------------------------------------------------------
    out["sync"] = sync_info

    if ms_fg is not None:
        out["sync"]["foreground"] = {"every_k_steps": args.foreground, "examples_per_s": cfg.R * cfg.B * K / (ms_fg * 1e-3),
                                     "note": "same kernels enqueued on the training streams (FR-* of the paper)"}
    if ms_hw is not None:
        out["hogwild"] = {"workers_per_replica": args.workers, "sync": "off",
                          "examples_per_s": cfg.R * args.workers * cfg.B * K / (ms_hw * 1e-3)}
    kernels, per_step = profile_pass(model, dev, cfg)
    out["kernels"] = kernels
    out["gpu_launches"] = int(round(per_step * cfg.R * K)) + int(round(sum(m["rounds"]) / len(m["rounds"])))
    out["gpu_launches_note"] = "kernel launches of this library inside one timed K-step region (sync on)"
    out["roofline"] = roofline(kernels, model, host, cfg, peaks)
    # the same kernel with one replica training alone (no other replica's kernels competing for the SMs)
    k1, _ = profile_pass(model, dev, cfg, replicas=[0])
    alone = roofline({out["roofline"]["kernel"]: k1[out["roofline"]["kernel"]]}, model, host, cfg, peaks) \
        if out["roofline"]["kernel"] in k1 else None
    if alone:
        out["roofline"]["one_replica_alone"] = {k: alone[k] for k in ("achieved", "frac", "us_per_launch")}

    # the sync kernel alone on vectors far larger than L2 (HBM-bound) -- the "sync HBM GB/s vs peak" half of the metric
    s = model.replicas[0].stream

    def time_sync(n, R):
        ws = [torch.randn(n, device=device) * 0.02 for _ in range(R)]
        c = torch.zeros(n, device=device)
        d = torch.zeros(n, device=device)
        fn = {"easgd": lambda i: ss.ss_sync_easgd(ws, c, n, cfg.alpha, 0, None, s),
              "ma": lambda i: ss.ss_sync_ma(ws, c, n, cfg.alpha, 0, None, s),
              "bmuf": lambda i: ss.ss_sync_bmuf(ws, c, d, n, cfg.alpha, cfg.eta, cfg.mu, 0, None, s)}[cfg.sync]
        with torch.cuda.stream(s):
            time_kernel_call(fn, s, 3)
            ms = time_kernel_call(fn, s, 20)
        gbs = SYNC_VECTORS[cfg.sync](R) * 4 * n / (ms * 1e-3) / 1e9
        return {"n": n, "R": R, "us": ms * 1e3, "GB/s": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"]}
    out["sync"]["kernel_alone_64M"] = time_sync(1 << 26, cfg.R)
    torch.cuda.synchronize()
    if cfg.bf16:
        out["gemm_alone"] = gemm_alone(s, peaks)
    if cfg.D <= 128:
        out["embedding_alone"] = embedding_alone(model, host, dev, cfg, peaks)
        torch.cuda.synchronize()

    # ---- the sync-kernel sweep running concurrently with this training ---------------------------
    if not args.quick and not args.no_sweep:
        out["sync"]["concurrent_sweep"] = concurrent_sweep(model, graphs, cfg, K, W, args, peaks,
                                                           value_off=sync_info["examples_per_s_sync_off"])
    # ---- end to end through the public API with host buffers ------------------------------------
    if not args.quick:
        out["e2e"] = bench_e2e(model, host, dev, graphs, cfg, K, W, args)
        out["cpu_baseline"] = cpu_baseline(cfg, budget_s=args.cpu_budget)
    # ---- the other single-GPU workloads, as legs of the same line ---------------------------------
    if not args.quick and not args.no_legs and world == 1 and args.workload == "medium" and not args.replicas:
        del graphs, dev, host, model
        torch.cuda.empty_cache()
        out["workloads"] = {}
        for name in ("medium_bmuf", "large"):
            out["workloads"][name] = bench_leg(synth.CONFIGS[name], K, W, device, args, peaks)
            torch.cuda.empty_cache()
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


SYNC_VECTORS = {"easgd": lambda R: 2 * R + 2, "ma": lambda R: 2 * R + 1, "bmuf": lambda R: 2 * R + 4}


def bench_leg(cfg, K, W, device, args, peaks):
    """Another workload measured the same way (K-step regions, sync off / on alternating, median), reported as a leg:
    examples/s, sync loss, sync gap and the roofline entry of its dominant kernel."""
    import torch
    ring = 4 if cfg.R * cfg.B >= 32768 else RING           # fewer pre-generated batches where one is ~850 k lookups
    model, host, dev, max_L = build_job(cfg, device, ring=ring)
    for r in range(cfg.R):
        model.step(r, dev[r][0])
    model.sync(**sync_args(cfg))
    torch.cuda.synchronize()
    graphs = capture_graphs(model, dev)
    m = measure_training(model, graphs, cfg, K, W, Barrier(1), device, args)
    value, on, info = summarise_training(m, K)
    kernels, per_step = profile_pass(model, dev, cfg, steps=3)
    leg = {"value": value, "unit": UNIT, "ms_per_step": on["median_ms"] / K, "config": {"workload": workload_text(cfg)},
           "sync": info, "roofline": roofline(kernels, model, host, cfg, peaks),
           "kernel_launches_per_replica_step": per_step, "status_word": model.status()}
    del graphs, dev, host, model
    return leg


def concurrent_sweep(model, graphs, cfg, K, W, args, peaks, value_off):
    """The sync-kernel sweep run concurrently with this workload's training: the shadow thread loops a sync pass
    over R vectors of n floats each (separate buffers, N(0, 0.02^2)) on the lowest-priority stream while the
    replicas train; per point the training throughput, its loss against the sync-off figure and the sync traffic
    the passes got under that contention (algorithmic bytes of the completed passes / time)."""
    import torch
    from paper_2003_03477_b200 import binding as ss
    device = model.center.device
    rows = []
    Rs = (2, 4, 8, 16) if args.sweep_all_r else (cfg.R,)
    gen = torch.Generator(device=device).manual_seed(20030347)
    for n in (1 << 20, 1 << 23, 1 << 26, 1 << 28):
        for R in Rs:
            if (R + 2) * n * 4 > 40e9:
                continue
            ws = [torch.randn(n, device=device, generator=gen) * 0.02 for _ in range(R)]
            c = ws[0].clone()
            d = torch.zeros(n, device=device)
            for rule, alpha, eta, mu in (("easgd", 0.1, 1.0, 0.0), ("ma", 0.1, 1.0, 0.0), ("bmuf", 0.1, 1.0, 0.9)):
                h = ss.ss_shadow_start(rule, ws, c, d, n, alpha, eta, mu, 0, None, model.sync_stream, args.sync_in_flight, 0)
                ss.ss_shadow_pause(h, True)
                run_steps(model, graphs, 0, W)
                torch.cuda.synchronize()
                reps = 0
                t_ms = 0.0
                r0 = ss.ss_shadow_rounds(h)
                ss.ss_shadow_pause(h, False)
                while t_ms < 1e3 * args.sweep_seconds or reps < 2:
                    ms, _ = timed_region(model, graphs, W + reps * K, K)
                    t_ms += ms
                    reps += 1
                ss.ss_shadow_pause(h, True)
                passes = ss.ss_shadow_rounds(h) - r0
                ss.ss_shadow_stop(h)
                ex = cfg.R * cfg.B * K * reps / (t_ms * 1e-3)
                gbs = SYNC_VECTORS[rule](R) * 4 * n * passes / (t_ms * 1e-3) / 1e9
                rows.append({"rule": rule, "R": R, "n": n, "train_examples_per_s": ex,
                             "train_loss_pct": 100.0 * (1.0 - ex / value_off), "sync_passes_per_s": passes / (t_ms * 1e-3),
                             "sync_GB/s": gbs, "sync_frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
                             "timed_s": t_ms * 1e-3})
            del ws, c, d
            torch.cuda.empty_cache()
    return {"training": workload_text(cfg), "rows": rows,
            "note": "sync vectors are separate buffers; passes counted as completed (thread paused and drained at both "
                    "ends); train_loss_pct is against examples_per_s_sync_off of the same run"}


def gemm_alone(stream, peaks):
    """The tensor-core GEMM kernel on its own (ss_gemm_bf16, bf16 in, fp32 out), timed with events around a
    captured graph of back-to-back launches: two products large enough to fill the machine (256 x 256 tiles on CTA
    pairs: 4096^3 is 256 such tiles on 74 pairs, i.e. 3.5 rounds; 8192 x 8192 x 4096 is 13.8 rounds), and the largest
    product of the medium model's step, against the measured burst bf16 peak."""
    import torch
    from paper_2003_03477_b200 import binding as ss
    res = []
    for M, N, K, reps in ((4096, 4096, 4096, 10), (8192, 8192, 4096, 5), (2048, 1728, 512, 20)):
        a = torch.randn(M, K, device="cuda").to(torch.bfloat16)
        b = torch.randn(N, K, device="cuda").to(torch.bfloat16)
        c = torch.empty(M, N, device="cuda")
        ss.ss_gemm_bf16(a, 0, K, b, 0, K, c, N, M, N, K, 0, stream)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(reps):
                ss.ss_gemm_bf16(a, 0, K, b, 0, K, c, N, M, N, K, 0, stream)
        with torch.cuda.stream(stream):
            g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.replay()
            e1.record(stream)
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / reps
        tf = 2.0 * M * N * K / us / 1e6
        res.append({"M": M, "N": N, "K": K, "us": us, "TFLOP/s": tf, "frac_of_bf16_peak": tf / peaks["bf16_tflops"]})
    return res


def embedding_alone(model, host, dev, cfg, peaks):
    """The embedding kernels on their own: the forward gather, and the reduction half of the backward (fused
    window kernel + combine kernel, which also update the rows), each timed with events around a captured graph
    of `reps` launches with an L2 flush (a 256 MiB fill) before every launch; the time of a graph of the flushes
    alone is subtracted.  Algorithmic bytes as in roofline(); fractions are of the measured copy peak."""
    import torch
    from paper_2003_03477_b200 import binding as ss
    rep, sp = model.replicas[0], model.spec
    s = rep.stream
    T, N, D, B = model.T, model.N, model.D, model.B
    b, hb = dev[0][0], host[0][0]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=b.indices.device)
    reps = 8
    with torch.cuda.stream(s):
        # the workspace holds the sort of this batch; the gradient is whatever the last step left (any values do)
        ss.ss_embbag_bwd_sort(T, N, D, b.indices, b.offsets, B, b.L, rep.emb_ws, None, None, None, rep.num_unique,
                              model.d_status, s)
    torch.cuda.synchronize()
    U = float(rep.num_unique.item())

    def fwd():
        ss.ss_embbag_fwd(model.tables, T, N, D, b.indices, b.offsets, B, rep.concat_f32, sp.W, rep.concat_bf16, sp.W, D,
                         model.d_status, s)

    def apply():
        ss.ss_embbag_bwd_apply(model.tables, model.row_state, T, N, D, B, b.L, rep.grad_pooled, T * D, 0, model.lr,
                               model.eps, rep.emb_ws, model.d_status, s)

    def graph_ms(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for _ in range(reps):
                flush.fill_(1)
                if fn is not None:
                    fn()
        best = None
        with torch.cuda.stream(s):
            g.replay()
            for _ in range(3):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(s)
                g.replay()
                e1.record(s)
                e1.synchronize()
                ms = e0.elapsed_time(e1)
                best = ms if best is None else min(best, ms)
        return best

    base = graph_ms(None)
    out = {}
    obytes = T * B * D * (2 if cfg.bf16 else 4)
    for name, fn, nbytes, compulsory, kernels in (
            ("embbag_fwd", fwd, hb.L * (4 * D + 4) + 4 * (T * B + 1) + obytes,
             U * 4 * D + 4 * hb.L + 4 * (T * B + 1) + obytes, ("embbag_fwd_kernel",)),
            ("embbag_bwd_apply", apply, hb.L * (4 * D + 16) + U * (2 * 4 * D + 8),
             U * (2 * 4 * D + 8) + T * B * 4 * D + 16 * hb.L, ("window_apply_kernel", "combine_rows_kernel"))):
        us = (graph_ms(fn) - base) * 1e3 / reps
        gbs = nbytes / (us * 1e-6) / 1e9
        cgbs = compulsory / (us * 1e-6) / 1e9
        dram = [ncu_traffic(k, cfg.name) for k in kernels]
        dram = sum(dram) if all(d is not None for d in dram) else None
        out[name] = {"us": us, "algorithmic_bytes": nbytes, "GB/s": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
                     "compulsory_bytes": compulsory, "compulsory_GB/s": cgbs,
                     "compulsory_frac_of_hbm_peak": cgbs / peaks["hbm_gbs"],
                     "dram_bytes_ncu": dram,
                     "dram_GB/s_ncu_bytes_over_this_time": (dram / (us * 1e-6) / 1e9) if dram else None}
    out["note"] = ("L2 flushed before every launch.  algorithmic_bytes counts every lookup's row (forward) or gradient row "
                   "(backward) once per lookup, which is what the kernels move between L2 and the SMs: Zipf-hot rows and the "
                   "gathered gradient rows are served from L2 within a launch, so this is an effective figure and is the one "
                   "the 0.70 target is read against; compulsory_bytes counts each distinct row, the gradient matrix and the "
                   "index / sort metadata once (what must cross DRAM); dram_bytes_ncu is dram__bytes_read + write of one ncu "
                   "capture (null when the kernels changed since).  embbag_bwd_apply = window kernel + combine kernel")
    return out


def profile_pass(model, dev, cfg, steps=6, replicas=None):
    """Per-kernel device times from the library's event timers over a short region in which all replicas
    train concurrently (plain launches: timing events cannot be read back from a captured graph).
    Returns ({kernel: {launches_per_replica_step, us_per_launch, share}}, launches per replica step)."""
    import torch
    from paper_2003_03477_b200 import binding as ss
    reps = list(range(cfg.R)) if replicas is None else list(replicas)
    ring = len(dev[0])
    for t in range(2):
        for r in reps:
            model.step(r, dev[r][t % ring])
    torch.cuda.synchronize()
    ss.ss_profile(True)
    for t in range(steps):
        for r in reps:
            model.step(r, dev[r][t % ring])
    recs = ss.ss_profile_collect()
    ss.ss_profile(False)
    agg = {}
    for name, ms in recs:
        a = agg.setdefault(name, [0, 0.0])
        a[0] += 1
        a[1] += ms * 1e3
    total = sum(a[1] for a in agg.values()) or 1.0
    n_rs = steps * len(reps)
    table = {k: {"launches_per_replica_step": c / n_rs, "us_per_launch": t / c, "share": t / total}
             for k, (c, t) in sorted(agg.items(), key=lambda kv: -kv[1][1])}
    return table, len(recs) / n_rs


def roofline(kernels, model, host, cfg, peaks):
    """Roofline entry of the kernel with the largest share of the step's kernel time.

    Algorithmic work per launch: embedding forward L(4D+4) + 4(TB+1) + TB*D*{2,4} bytes; fused window kernel
    L(4D+16) + U(2*4D+8) (gather plus row read-modify-write); unfused window reduction L(4D+16) + U*4D; row update
    U(3*4D+12); tensor-core GEMMs: the step's 2MNK summed over its GEMM launches.
    L and U are the means over the batches of replica 0 (U read back from the device)."""
    T, D, B = cfg.T, cfg.D, cfg.B
    L = float(np.mean([b.L for b in host[0]]))
    U = float(model.replicas[0].num_unique.item())
    dims = model.spec.layer_dims
    nl = len(dims)
    gemm_flops = 0.0
    for l, (fin, fout) in enumerate(dims):
        if l == nl - 1 or fin < 16:
            continue                      # single-logit and 13-input layers run on SIMT kernels
        gemm_flops += 6.0 * B * fin * fout   # forward, weight gradient, input gradient: 2*B*in*out each
    work = {
        "embbag_fwd_kernel": ("hbm", L * (4 * D + 4) + 4 * (T * B + 1) + T * B * D * (2 if cfg.bf16 else 4), 1),
        "window_apply_kernel": ("hbm", L * (4 * D + 16) + U * (2 * 4 * D + 8), 1),
        "window_reduce_kernel": ("hbm", L * (4 * D + 16) + U * 4 * D, 1),
        "apply_rows_kernel": ("hbm", U * (3 * 4 * D + 12), 1),
        "gemm_tc_kernel": ("tensor", gemm_flops, None),
    }
    name = next((k for k in kernels if k in work), None)
    if name is None:
        return {"kernel": next(iter(kernels), None), "bound": "alu", "achieved": None, "peak": None, "unit": None,
                "frac": None, "traffic": None}
    bound, amount, per = work[name]
    k = kernels[name]
    n_launch = k["launches_per_replica_step"]
    us_total = k["us_per_launch"] * n_launch          # per replica step
    if bound == "hbm":
        achieved = amount / (us_total / n_launch * 1e-6) / 1e9
        peak, unit = peaks["hbm_gbs"], "GB/s"
    else:
        achieved = amount / (us_total * 1e-6) / 1e12
        peak, unit = peaks["bf16_tflops_sustained"], "TFLOP/s"
    extra = {}
    if name == "gemm_tc_kernel":
        # the launch deliberately takes only some of the SMs (the other replicas' kernels run on the rest), so the
        # fraction of the whole device's peak understates the kernel: give the share of the SMs it holds as well
        import torch
        from paper_2003_03477_b200 import binding as ss
        sms = torch.cuda.get_device_properties(model.center.device).multi_processor_count
        ctas = min(ss.ss_mlp_set_flow_ctas(-1), sms)
        extra = {"ctas_per_launch": ctas, "sms": sms, "frac_of_the_peak_of_the_sms_it_takes": achieved / peak * sms / ctas,
                 "tensor_pipe_active_pct_ncu": ncu_traffic(name, cfg.name, "tensor_pipe_active_pct")}
    return {"kernel": name, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
            **extra, "traffic": ncu_traffic(name, cfg.name), "traffic_unit": "bytes per launch (ncu, DRAM read + write)",
            "peak_source": peaks["source"], "launches_per_replica_step": n_launch,
            "us_per_launch": k["us_per_launch"], "share_of_kernel_time": k["share"],
            "work_per_replica_step": amount,
            "timing": "CUDA events around every launch on its stream, all replicas training concurrently"}


def bench_e2e(model, host, dev, graphs, cfg, K, W, args):
    """Same metric with the step's inputs in pinned host memory: every step copies its batch host->device
    into the ring slot's device buffers (on a copy stream, so the copy of a later step overlaps the kernels of an
    earlier one), replays that slot's captured step once the copy has landed and reads the loss back.  Host wall
    clock around exactly K steps (ending with a synchronise of every replica stream), the region repeated until
    half of args.min_seconds has been timed; the median region gives the value."""
    import torch
    from paper_2003_03477_b200 import trainer
    pinned = [[trainer.DeviceBatch.pack_host(b.indices, b.offsets, b.dense, b.labels) for b in bs] for bs in host]
    loss_host = [torch.zeros(1).pin_memory() for _ in range(cfg.R)]
    h2d = d2h = 0
    ring = len(dev[0])
    paced = cfg.sync_every

    # A copy stream per replica prefetches: the copies of step t go out as soon as the step that used the ring slot
    # before (t - ring) has finished, not behind step t - 1, so they overlap this replica's own kernels.
    copy_streams = [torch.cuda.Stream(device=rep.stream.device) for rep in model.replicas]
    slot_free = [[None] * ring for _ in range(cfg.R)]          # recorded after the step that read the slot
    slot_ready = [[torch.cuda.Event() for _ in range(ring)] for _ in range(cfg.R)]

    def step(t):
        nonlocal h2d, d2h
        for r, rep in enumerate(model.replicas):
            slot = t % ring
            src, dst = pinned[r][slot], dev[r][slot]
            with torch.cuda.stream(copy_streams[r]):
                if slot_free[r][slot] is not None:
                    copy_streams[r].wait_event(slot_free[r][slot])
                dst.storage.copy_(src, non_blocking=True)    # indices, offsets, dense features and labels in one copy
                slot_ready[r][slot].record(copy_streams[r])
            with torch.cuda.stream(rep.stream):
                rep.stream.wait_event(slot_ready[r][slot])
                graphs[r][slot].replay()
                loss_host[r].copy_(rep.loss, non_blocking=True)
                if slot_free[r][slot] is None:
                    slot_free[r][slot] = torch.cuda.Event()
                slot_free[r][slot].record(rep.stream)
            h2d += src.numel()
            d2h += 4
        if paced and (t + 1) % paced == 0:
            model.sync(**sync_args(cfg))

    loop = None if paced else trainer.ShadowLoop(model, cfg.sync, cfg.alpha, cfg.eta, cfg.mu).start()
    for t in range(W):
        step(t)
    torch.cuda.synchronize()
    times = []
    while len(times) < 3 or (sum(times) < 0.5 * args.min_seconds and len(times) < 200):
        h2d = d2h = 0
        t0 = time.perf_counter()
        for t in range(W, W + K):
            step(t)
        for rep in model.replicas:
            rep.stream.synchronize()
        times.append(time.perf_counter() - t0)
    if loop is not None:
        loop.stop()
    torch.cuda.synchronize()
    dt = statistics.median(times)
    return {"value": cfg.R * cfg.B * K / dt, "unit": UNIT, "h2d_bytes_per_step": h2d // K, "d2h_bytes_per_step": d2h // K,
            "regions": {"median_ms": dt * 1e3, "min_ms": min(times) * 1e3, "max_ms": max(times) * 1e3, "repeats": len(times)},
            "timing": "host wall clock around K steps, ending with a synchronise of every replica stream; median of the repeats"}


# ----------------------------------------------------------------------------------------------
def oracle_sample(cfg, budget_s):
    """Times the oracle on replica steps of the workload's shape with a reduced batch (same bag mix, index
    skew, layer widths); returns (examples, seconds, description)."""
    from oracle import shadowsync_oracle as O
    from paper_2003_03477_b200 import synth
    Bs = min(cfg.B, 64)
    small = synth.scaled(cfg, B=Bs, R=1)
    batch = synth.make_batch(small, 0, 0)
    # compact table: only the rows this sample touches (the full table does not need to exist on the host)
    lens = np.diff(batch.offsets.astype(np.int64))
    tbl = np.repeat(np.arange(cfg.T * Bs) // Bs, lens)
    keys = tbl.astype(np.int64) * cfg.N + batch.indices
    uniq, inv = np.unique(keys, return_inverse=True)
    rows_per_t = [uniq[(uniq // cfg.N) == t] % cfg.N for t in range(cfg.T)]
    nmax = max(len(r) for r in rows_per_t)
    tables = np.zeros((cfg.T, nmax, cfg.D), np.float32)
    remap = np.zeros(len(uniq), np.int64)
    for t in range(cfg.T):
        tables[t, :len(rows_per_t[t])] = synth.table_rows(cfg, t, rows_per_t[t])
        remap[(uniq // cfg.N) == t] = np.arange(len(rows_per_t[t]))
    batch.indices = remap[inv].astype(np.int32)
    layers = synth.initial_weights(cfg)
    accs = [(np.zeros_like(W), np.zeros_like(b)) for W, b in layers]
    state = np.zeros((cfg.T, nmax), np.float32)
    n, t0 = 0, time.perf_counter()
    while True:
        O.replica_step(tables, state, layers, accs, len(cfg.bottom) - 1, batch, cfg.lr, cfg.eps, cfg.bf16)
        n += Bs
        dt = time.perf_counter() - t0
        if dt > budget_s:
            break
    return n, dt, f"{n // Bs} replica steps of batch {Bs} (full model widths, same bag/index recipe, touched rows only)"


def cpu_baseline(cfg, budget_s):
    n, dt, what = oracle_sample(cfg, budget_s)
    blas = threads_used()
    return {"value": n / dt, "unit": UNIT, "cores": blas, "kind": "oracle",
            "threads": {"python": 1, "blas": blas},
            "sample": what + f"; one Python thread (pooling, sort and segment loops), numpy matrix products on up to "
                             f"{blas} BLAS threads"}


def threads_used():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def bench_reference(args):
    """The oracle as it stands on the host cores, on the same workload's shapes (bounded sample per step)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2003_03477_b200 import synth
    cfg = synth.CONFIGS[args.workload]
    K, W = args.steps, args.warmup
    per_step = max(1.0, min(10.0, 120.0 / max(1, K + W)))
    for _ in range(min(W, 1)):
        oracle_sample(cfg, 0.0)
    n = dt = 0.0
    what = ""
    for _ in range(K):
        a, b, what = oracle_sample(cfg, per_step)
        n += a
        dt += b
    v = n / dt
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": K, "warmup": W, "ms_per_step": 1e3 * dt / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name} (CPU oracle on a bounded sample)"},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": threads_used(), "kind": "oracle",
                         "threads": {"python": 1, "blas": threads_used()},
                         "sample": what + " per step; one Python thread, numpy matrix products on the BLAS threads"},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def bench_sweep(args):
    """Isolated sync-kernel sweep: n in {1M, 8M, 64M, 256M} floats per replica, R in {2, 4, 8, 16}, all three
    rules (S-EASGD alpha 0.1, S-MA alpha 0.1, S-BMUF mu 0.9 eta 1); one JSON line with GB/s against the HBM peak."""
    import torch
    from paper_2003_03477_b200 import binding as ss
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    s = torch.cuda.current_stream()
    rows = []
    for n in (1 << 20, 1 << 23, 1 << 26, 1 << 28):
        for R in (2, 4, 8, 16):
            if (R + 2) * n * 4 > 60e9:
                continue
            ws = [torch.randn(n, device="cuda") * 0.02 for _ in range(R)]
            c = torch.randn(n, device="cuda") * 0.02
            d = torch.zeros(n, device="cuda")
            for rule, fn, per in (("easgd", lambda i: ss.ss_sync_easgd(ws, c, n, 0.1, 0, None, s), 2 * R + 2),
                                  ("ma", lambda i: ss.ss_sync_ma(ws, c, n, 0.1, 0, None, s), 2 * R + 1),
                                  ("bmuf", lambda i: ss.ss_sync_bmuf(ws, c, d, n, 0.1, 1.0, 0.9, 0, None, s), 2 * R + 4)):
                time_kernel_call(fn, s, 3)
                reps = 50 if n <= (1 << 23) else 10
                ms = time_kernel_call(fn, s, reps)
                gbs = per * 4 * n / (ms * 1e-3) / 1e9
                rows.append({"rule": rule, "R": R, "n": n, "us": round(ms * 1e3, 2), "GB/s": round(gbs, 1),
                             "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 3),
                             "l2_resident": bool(per * 4 * n < 100e6)})
            del ws, c, d
    print(json.dumps({"sweep": "sync kernels alone", "peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "rows": rows}))


def plain_steps(args):
    """A few plain (un-captured) replica steps of a workload on one GPU, every library call launched directly on the
    replica's stream so that each kernel shows up as its own launch: the program profilers are pointed at.
    --tables / --rows / --batch shrink the workload (fewer or shorter tables, smaller batch) while keeping its layer
    widths, bag-length mix and index skew; --plain-sync adds one synchronisation pass after every step."""
    import torch
    from paper_2003_03477_b200 import binding as ss, synth, trainer
    cfg = synth.CONFIGS[args.workload]
    if args.tables:
        cfg = synth.scaled(cfg, T=args.tables, top=((1 + args.tables) * cfg.D,) + tuple(cfg.top[1:]))
    if args.rows:
        cfg = synth.scaled(cfg, N=args.rows)
    if args.batch:
        cfg = synth.scaled(cfg, B=args.batch)
    cfg = synth.scaled(cfg, R=args.replicas or 1)
    torch.cuda.set_device(0)
    model, host, dev, _ = build_job(cfg, torch.device("cuda", 0), ring=2)
    for t in range(args.steps):
        for r in range(cfg.R):
            model.step(r, dev[r][t % 2])
        if args.plain_sync:
            model.sync(cfg.sync, cfg.alpha, cfg.eta, cfg.mu)
    torch.cuda.synchronize()
    print(json.dumps({"plain": workload_text(cfg), "steps": args.steps, "loss": float(model.replicas[0].loss.item()),
                      "status_word": model.status()}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="medium", choices=["tiny", "medium", "medium_bmuf", "large"])
    ap.add_argument("--sync-in-flight", type=int, default=2)
    ap.add_argument("--sync-pause", type=float, default=0.0)
    ap.add_argument("--steps-ahead", type=int, default=16,
                    help="steps of a replica the host keeps queued on the device (0 = unbounded)")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="the K-step region is repeated until this much has been timed per arm (sync on, sync off)")
    ap.add_argument("--min-repeats", type=int, default=10)
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--replicas", type=int, default=0, help="override the workload's replica count (experiments)")
    ap.add_argument("--quick", action="store_true", help="skip the e2e, CPU-baseline, concurrent-sweep and other-workload legs")
    ap.add_argument("--no-legs", action="store_true", help="skip the medium_bmuf and large legs")
    ap.add_argument("--no-sweep", action="store_true", help="skip the sync sweep concurrent with training")
    ap.add_argument("--sweep-seconds", type=float, default=0.25, help="training time per point of the concurrent sweep")
    ap.add_argument("--sweep-all-r", action="store_true", help="concurrent sweep over R = 2, 4, 8, 16 instead of the workload's R")
    ap.add_argument("--flow-ctas", type=int, default=0,
                    help="CTAs of the persistent tensor-core launches of the MLP (0 = the library's rule)")
    ap.add_argument("--foreground", type=int, default=0,
                    help="also time the foreground variant: one sync pass on the training streams every k steps")
    ap.add_argument("--workers", type=int, default=1,
                    help="also time m lock-free workers per replica sharing its parameters (intra-trainer Hogwild)")
    ap.add_argument("--sweep", action="store_true", help="isolated sync-kernel sweep instead of the training benchmark")
    ap.add_argument("--plain", action="store_true", help="run --steps un-captured replica steps and exit (for profilers)")
    ap.add_argument("--tables", type=int, default=0, help="--plain: number of tables")
    ap.add_argument("--rows", type=int, default=0, help="--plain: rows per table")
    ap.add_argument("--batch", type=int, default=0, help="--plain: per-replica batch")
    ap.add_argument("--plain-sync", action="store_true", help="--plain: one sync pass after every step")
    args = ap.parse_args()
    global STEPS_AHEAD
    STEPS_AHEAD = max(0, args.steps_ahead)
    if args.plain:
        plain_steps(args)
    elif args.sweep:
        bench_sweep(args)
    elif args.impl == "reference":
        bench_reference(args)
    else:
        bench_gpu(args)


if __name__ == "__main__":
    main()
