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

`--impl reference` times the CPU oracle (oracle/, test infrastructure) on a bounded sample of the same
workload on the host cores; it is deliberately slow and is a reported baseline, not a target.
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
    "gemm_tc_kernel": {
        "workload": "medium",
        "bytes_per_launch": 4887352,      # mean over the 9 GEMM launches of a replica step
        "capture": "profiles/step_medium_top_kernels.md",
        "sources": {
            "gemm_tc.cu": "14567cfb0dbd4a7a16394e5e5b169de194ea2f38254bf0ec44ffbb10551c1479",
            "mlp.cu": "9ebfdc7cb9de27e940592657a1445a3989af3655ecfafc592519c4e215891479",
            "gemm.cuh": "7491d2079ed234aeda8b58fdac00e6c5965a825b21e58246e8fc0e3b9a32b6f8",
            "mlp_plan.cuh": "0c026b6ce9a10e26eec5b857317a2fda0152cc17fa8989500e7fba16f35a7bbb",
        },
    },
}


def ncu_traffic(kernel, workload):
    """Bytes per launch from the stored ncu capture, or None when it does not cover this kernel, this workload
    or the current sources."""
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
    return e["bytes_per_launch"]


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
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------
def build_job(cfg, device, workers=1):
    """Tables, replicas and a ring of device-resident batches for one GPU."""
    import torch
    from paper_2003_03477_b200 import binding as ss, synth, trainer
    tables = trainer.device_tables(cfg, device)
    spec = ss.MlpSpec(cfg.bottom, cfg.top, cfg.bf16)
    w0 = torch.from_numpy(trainer.pack_params(spec, synth.initial_weights(cfg))).to(device)
    host = [[synth.make_batch(cfg, r, t) for t in range(RING)] for r in range(cfg.R)]
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


def run_steps(model, graphs, first_step, n_steps):
    """Replays the replicas' step graphs.  The host keeps at most STEPS_AHEAD steps of a replica queued on the device
    (it waits for the event of step t - STEPS_AHEAD before it enqueues step t; 0 = no bound).  An unbounded queue
    changes nothing for training but makes the shadow thread's launches wait behind thousands of queued graph
    launches: measured 76 sync rounds/s (a pass every 25 steps) unbounded, 312/s (every 6 steps) with 16, 1416/s
    (every 1.3 steps, training -1 %) with 4."""
    import torch
    evs = [[] for _ in model.replicas]
    for t in range(first_step, first_step + n_steps):
        for r, rep in enumerate(model.replicas):
            if STEPS_AHEAD and len(evs[r]) >= STEPS_AHEAD:
                evs[r].pop(0).synchronize()
            with torch.cuda.stream(rep.stream):
                graphs[r][t % RING].replay()
                if STEPS_AHEAD:
                    e = torch.cuda.Event()
                    e.record(rep.stream)
                    evs[r].append(e)


def timed_region(model, graphs, first_step, n_steps):
    """Device time of n_steps steps over all replica streams (ms)."""
    import torch
    main = torch.cuda.current_stream()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record(main)
    for rep in model.replicas:
        rep.stream.wait_event(start)
    run_steps(model, graphs, first_step, n_steps)
    for rep in model.replicas:
        e = torch.cuda.Event()
        e.record(rep.stream)
        main.wait_event(e)
    stop.record(main)
    stop.synchronize()
    return start.elapsed_time(stop)


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

    model, host, dev, max_L = build_job(cfg, device, workers=max(1, args.workers))
    # un-captured warm-up: first-use set-up inside the library (function attributes, symbol addresses)
    for r in range(cfg.R):
        model.step(r, dev[r][0])
    model.sync(**sync_args(cfg))
    torch.cuda.synchronize()
    graphs = capture_graphs(model, dev)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- sync off ------------------------------------------------------------------------
    run_steps(model, graphs, 0, W)
    barrier()
    ms_off = timed_region(model, graphs, W, K)

    # ---- sync on (the headline) -------------------------------------------------------------
    loop = trainer.ShadowLoop(model, max_in_flight=args.sync_in_flight, pause_s=args.sync_pause, **sync_args(cfg)).start()
    run_steps(model, graphs, 0, W)
    barrier()
    sampler = ClockSampler(local).start()
    rounds0 = loop.rounds
    ms_on = timed_region(model, graphs, W, K)
    rounds = loop.rounds - rounds0
    clocks = sampler.stop()
    barrier()
    loop.stop()
    torch.cuda.synchronize()
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
        m = args.workers
        for r in range(cfg.R):
            for k in range(1, m):
                model.step(r, dev[r][k % RING], worker=k)
        torch.cuda.synchronize()
        wg = []
        for r in range(cfg.R):
            per_worker = []
            for k in range(m):
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
                    for k in range(m):
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
    (ms_on, ms_off), examples = reduce_over_ranks([ms_on, ms_off], cfg.R * cfg.B * K, device)
    value = examples / (ms_on * 1e-3)
    value_off = examples / (ms_off * 1e-3)
    status = model.status() | (ss.ss_device_error() << 8)

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_on / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.bf16 else "f32", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: R={cfg.R} T={cfg.T} N={cfg.N} D={cfg.D} B={cfg.B} "
                               f"bottom={'-'.join(map(str, cfg.bottom))} top={'-'.join(map(str, cfg.top))} "
                               f"sync={cfg.sync} alpha={cfg.alpha} background",
                   "l2": "inputs larger than L2: tables 6.7 GB gathered by Zipf indices, 8 rotating batches per replica",
                   "multi_gpu": "replicas only (no cross-GPU exchange on this path)",
                   "steps_ahead": STEPS_AHEAD},
        "clocks": clocks,
        "status_word": status,
    }
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- extra measurements on rank 0 ---------------------------------------------------------
    out["sync"] = {"rounds_per_s": rounds / (ms_on * 1e-3), "avg_sync_gap_steps": (K / rounds) if rounds else None,
                   "examples_per_s_sync_off": value_off, "throughput_loss_pct": 100.0 * (1.0 - value / value_off)}

    if ms_fg is not None:
        out["sync"]["foreground"] = {"every_k_steps": args.foreground, "examples_per_s": cfg.R * cfg.B * K / (ms_fg * 1e-3),
                                     "note": "same kernels enqueued on the training streams (FR-* of the paper)"}
    if ms_hw is not None:
        out["hogwild"] = {"workers_per_replica": args.workers, "sync": "off",
                          "examples_per_s": cfg.R * args.workers * cfg.B * K / (ms_hw * 1e-3)}
    kernels, per_step = profile_pass(model, dev, cfg)
    out["kernels"] = kernels
    out["gpu_launches"] = int(round(per_step * cfg.R * K)) + int(rounds)
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
        per = {"easgd": 2 * R + 2, "ma": 2 * R + 1, "bmuf": 2 * R + 4}[cfg.sync]
        gbs = per * 4 * n / (ms * 1e-3) / 1e9
        return {"n": n, "R": R, "us": ms * 1e3, "GB/s": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"]}
    out["sync"]["kernel_alone_64M"] = time_sync(1 << 26, cfg.R)
    torch.cuda.synchronize()
    if cfg.bf16:
        out["gemm_alone"] = gemm_alone(s, peaks)
    if cfg.D <= 128:
        out["embedding_alone"] = embedding_alone(model, host, dev, cfg, peaks)
        torch.cuda.synchronize()

    # ---- end to end through the public API with host buffers ------------------------------------
    if not args.quick:
        out["e2e"] = bench_e2e(model, host, dev, graphs, cfg, K, W)
        out["cpu_baseline"] = cpu_baseline(cfg, budget_s=args.cpu_budget)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def gemm_alone(stream, peaks):
    """The tensor-core GEMM kernel on its own (ss_gemm_bf16, bf16 in, fp32 out), timed with events around a
    captured graph of back-to-back launches: a product large enough to fill the machine, and the largest
    product of the medium model's step, against the measured burst bf16 peak."""
    import torch
    from paper_2003_03477_b200 import binding as ss
    res = []
    for M, N, K, reps in ((4096, 4096, 4096, 10), (2048, 1728, 512, 20)):
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
    for name, fn, nbytes in (
            ("embbag_fwd", fwd, hb.L * (4 * D + 4) + 4 * (T * B + 1) + T * B * D * (2 if cfg.bf16 else 4)),
            ("embbag_bwd_apply", apply, hb.L * (4 * D + 16) + U * (2 * 4 * D + 8))):
        us = (graph_ms(fn) - base) * 1e3 / reps
        gbs = nbytes / (us * 1e-6) / 1e9
        out[name] = {"us": us, "algorithmic_bytes": nbytes, "GB/s": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"]}
    out["note"] = ("L2 flushed before every launch; Zipf-hot rows and the gathered gradient rows are re-read through L2 "
                   "within a launch; embbag_bwd_apply = fused window kernel + combine kernel")
    return out


def profile_pass(model, dev, cfg, steps=6, replicas=None):
    """Per-kernel device times from the library's event timers over a short region in which all replicas
    train concurrently (plain launches: timing events cannot be read back from a captured graph).
    Returns ({kernel: {launches_per_replica_step, us_per_launch, share}}, launches per replica step)."""
    import torch
    from paper_2003_03477_b200 import binding as ss
    reps = list(range(cfg.R)) if replicas is None else list(replicas)
    for t in range(2):
        for r in reps:
            model.step(r, dev[r][t % RING])
    torch.cuda.synchronize()
    ss.ss_profile(True)
    for t in range(steps):
        for r in reps:
            model.step(r, dev[r][t % RING])
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
    return {"kernel": name, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
            "traffic": ncu_traffic(name, cfg.name), "traffic_unit": "bytes per launch (ncu, DRAM read + write)",
            "peak_source": peaks["source"], "launches_per_replica_step": n_launch,
            "us_per_launch": k["us_per_launch"], "share_of_kernel_time": k["share"],
            "work_per_replica_step": amount,
            "timing": "CUDA events around every launch on its stream, all replicas training concurrently"}


def bench_e2e(model, host, dev, graphs, cfg, K, W):
    """Same metric with the step's inputs in pinned host memory: every step copies its batch host->device
    into the ring slot's device buffers, replays that slot's captured step and reads the loss back."""
    import torch
    from paper_2003_03477_b200 import trainer
    pinned = [[tuple(torch.from_numpy(np.ascontiguousarray(a)).pin_memory() for a in
                     (b.indices, b.offsets, b.dense, b.labels)) for b in bs] for bs in host]
    loss_host = [torch.zeros(1).pin_memory() for _ in range(cfg.R)]
    h2d = d2h = 0

    def step(t):
        nonlocal h2d, d2h
        for r, rep in enumerate(model.replicas):
            slot = t % RING
            src, dst = pinned[r][slot], dev[r][slot]
            with torch.cuda.stream(rep.stream):
                dst.indices.copy_(src[0], non_blocking=True)
                dst.offsets.copy_(src[1], non_blocking=True)
                dst.dense.copy_(src[2], non_blocking=True)
                dst.labels.copy_(src[3], non_blocking=True)
                graphs[r][slot].replay()
                loss_host[r].copy_(rep.loss, non_blocking=True)
            h2d += sum(x.numel() * x.element_size() for x in src)
            d2h += 4

    loop = trainer.ShadowLoop(model, cfg.sync, cfg.alpha, cfg.eta, cfg.mu).start()
    for t in range(W):
        step(t)
    torch.cuda.synchronize()
    h2d = d2h = 0
    t0 = time.perf_counter()
    for t in range(W, W + K):
        step(t)
    for rep in model.replicas:
        rep.stream.synchronize()
    dt = time.perf_counter() - t0
    loop.stop()
    torch.cuda.synchronize()
    return {"value": cfg.R * cfg.B * K / dt, "unit": UNIT, "h2d_bytes_per_step": h2d // K, "d2h_bytes_per_step": d2h // K,
            "timing": "host wall clock around K steps, ending with a synchronise of every replica stream"}


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
    return {"value": n / dt, "unit": UNIT, "cores": threads_used(), "kind": "oracle", "sample": what}


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
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": threads_used(), "kind": "oracle", "sample": what + " per step"},
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="medium", choices=["tiny", "medium", "medium_bmuf", "large"])
    ap.add_argument("--sync-in-flight", type=int, default=2)
    ap.add_argument("--sync-pause", type=float, default=0.0)
    ap.add_argument("--steps-ahead", type=int, default=16,
                    help="steps of a replica the host keeps queued on the device (0 = unbounded)")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--replicas", type=int, default=0, help="override the workload's replica count (experiments)")
    ap.add_argument("--quick", action="store_true", help="skip the e2e and CPU-baseline legs (experiments)")
    ap.add_argument("--foreground", type=int, default=0,
                    help="also time the foreground variant: one sync pass on the training streams every k steps")
    ap.add_argument("--workers", type=int, default=1,
                    help="also time m lock-free workers per replica sharing its parameters (intra-trainer Hogwild)")
    ap.add_argument("--sweep", action="store_true", help="isolated sync-kernel sweep instead of the training benchmark")
    args = ap.parse_args()
    global STEPS_AHEAD
    STEPS_AHEAD = max(0, args.steps_ahead)
    if args.sweep:
        bench_sweep(args)
    elif args.impl == "reference":
        bench_reference(args)
    else:
        bench_gpu(args)


if __name__ == "__main__":
    main()
