"""Runs one shape of the gossip step (and optionally the consensus reduction) a few times and
prints the CUDA-event timing: a small driver for profiling a single kernel with ncu.

  python -m paper_1705_09056_b200.run_case --n 64 --N 2000000 --topology ring --steps 3
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding, build, workloads as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--n", type=int, default=64)
    ap.add_argument("--N", type=int, default=2_000_000)
    ap.add_argument("--topology", default="ring")
    ap.add_argument("--kind", type=int, default=-1, help="force a DPSGD_MIX_* kernel")
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--consensus", action="store_true", help="also run the consensus reduction")
    ap.add_argument("--fused", action="store_true", help="time the gossip step that also returns the consensus distance")
    ap.add_argument("--swapped", action="store_true", help="footnote c: update locally, then average")
    ap.add_argument("--momentum", type=float, default=0.0, help="momentum of the Section 5.3 runs (one more matrix)")
    args = ap.parse_args()

    build.build()
    dev = torch.device("cuda", 0)
    ld = wl.padded_ld(args.N)
    X0 = wl.stress_matrix(args.n, ld, args.N, 1, dev)
    X1 = torch.zeros_like(X0)
    G = wl.stress_matrix(args.n, ld, args.N, 2, dev)
    ctx = binding.Dpsgd(args.n, args.N, *wl.topology(args.topology, args.n), gamma=0.01)
    ctx.bind(X0, X1, G)
    if args.kind >= 0:
        ctx.mix_kind(args.kind)
    if args.swapped:
        ctx.set_order(True)
    if args.momentum > 0.0:
        V = torch.zeros_like(X0)
        ctx.set_momentum(args.momentum, V)
    out = torch.zeros(1, dtype=torch.float64, device=dev)
    step = (lambda: ctx.mix_update_consensus(out)) if args.fused else ctx.mix_update
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        step()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / max(1, args.steps)
    out = {"n": args.n, "N": args.N, "topology": args.topology,
           "kernel": binding.MIX_NAMES[ctx.mix_kind()], "ms_per_step": ms,
           "GBps": (20.0 if args.momentum > 0.0 else 12.0) * args.n * args.N / (ms * 1e-3) / 1e9}
    if args.consensus:
        out["consensus"] = ctx.consensus_dist()
    print(json.dumps(out))
    ctx.close()


if __name__ == "__main__":
    main()
