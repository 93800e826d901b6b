"""Runs a few plain (un-captured) replica steps of a synthetic workload on one GPU.

    python -m paper_2003_03477_b200.run_steps --workload medium --tables 8 --steps 3 [--sync]

A small driver for profilers and quick checks: every library call is launched directly on the
replica's stream, so each kernel shows up as its own launch.  --tables / --rows / --batch shrink the workload
(fewer or shorter tables, smaller batch) while keeping its layer widths, bag-length mix and index skew.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as ss
from . import synth, trainer


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="medium", choices=sorted(synth.CONFIGS))
    ap.add_argument("--tables", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--rows", type=int, default=0, help="rows per table")
    ap.add_argument("--replicas", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--sync", action="store_true", help="one synchronisation pass after every step")
    args = ap.parse_args()
    cfg = synth.CONFIGS[args.workload]
    if args.tables:
        top = ((1 + args.tables) * cfg.D,) + tuple(cfg.top[1:])
        cfg = synth.scaled(cfg, T=args.tables, top=top)
    if args.rows:
        cfg = synth.scaled(cfg, N=args.rows)
    if args.batch:
        cfg = synth.scaled(cfg, B=args.batch)
    cfg = synth.scaled(cfg, R=args.replicas)
    tables = trainer.device_tables(cfg)
    spec = ss.MlpSpec(cfg.bottom, cfg.top, cfg.bf16)
    w0 = torch.from_numpy(trainer.pack_params(spec, synth.initial_weights(cfg))).cuda()
    host = [[synth.make_batch(cfg, r, t) for t in range(2)] for r in range(cfg.R)]
    model = trainer.Model(cfg.T, cfg.N, cfg.D, cfg.B, cfg.bottom, cfg.top, cfg.bf16, cfg.R, w0, tables, cfg.lr,
                          cfg.eps, max_L=max(b.L for bs in host for b in bs))
    dev = [[trainer.DeviceBatch(b.indices, b.offsets, b.dense, b.labels) for b in bs] for bs in host]
    for t in range(args.steps):
        for r in range(cfg.R):
            model.step(r, dev[r][t % 2])
        if args.sync:
            model.sync(cfg.sync, cfg.alpha, cfg.eta, cfg.mu)
    torch.cuda.synchronize()
    print(f"{cfg.name}: T={cfg.T} B={cfg.B} R={cfg.R} steps={args.steps} loss={float(model.replicas[0].loss.item()):.5f} "
          f"status={model.status()} device_error={ss.ss_device_error()}")


if __name__ == "__main__":
    main()
