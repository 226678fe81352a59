"""The measurement command of the package: runs one configuration a few times and prints CUDA-event
timings as one JSON line.  Also the command to put under a profiler for a single kernel.

  python -m paper_1705_09056_b200.run_config --config 2 --steps 50
      whole D-PSGD iterations (sample + gradient + mix + update): replica-steps/s and the split
      between gradient and gossip step (0 least squares, 1 logistic, 2 MLP 784-1024-10,
      4 MLP 1024-2048-2048-10)
  python -m paper_1705_09056_b200.run_config --config 3 --n 64 --N 2000000 --topology ring --steps 3
      the gossip step alone on supplied N(0,1) gradients (the bandwidth configuration, any shape)
  python -m paper_1705_09056_b200.run_config --conv --n 32 --batch 32 --steps 5
      forward pass of the CIFAR-shaped 3x3 convolution layers, every node with its own filters
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding, build, workloads as wl


def gossip_step_alone(args, dev):
    """dpsgd_mix_update (or dpsgd_mix_update_consensus) on an n x N matrix with supplied gradients."""
    n, N = args.n or 64, args.N or 25_000_000
    topology = args.topology or "ring"
    ld = wl.padded_ld(N)
    X0 = wl.stress_matrix(n, ld, N, 1, dev)
    X1 = torch.zeros_like(X0)
    G = wl.stress_matrix(n, ld, N, 2, dev)
    ctx = binding.Dpsgd(n, N, *wl.topology(topology, n), gamma=0.01)
    ctx.bind(X0, X1, G)
    if args.kind >= 0:
        ctx.mix_kind(args.kind)
    if args.swapped:
        ctx.set_order(True)
    if args.momentum > 0.0:
        V = torch.zeros_like(X0)
        ctx.set_momentum(args.momentum, V)
    out = torch.zeros(1, dtype=torch.float64, device=dev)
    step = (lambda: ctx.mix_update_consensus(out)) if args.fused_consensus else ctx.mix_update
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
    res = {"workload": "stress", "n": n, "N": N, "topology": topology,
           "kernel": binding.MIX_NAMES[ctx.mix_kind()], "ms_per_step": ms,
           "GBps": (20.0 if args.momentum > 0.0 else 12.0) * n * N / (ms * 1e-3) / 1e9}
    if args.consensus:
        res["consensus"] = ctx.consensus_dist()
    ctx.sync()
    print(json.dumps(res))
    ctx.close()


def conv_layers(args, dev):
    """dpsgd_conv3x3_forward on the six CIFAR-shaped layers: total and per-layer CUDA-event times."""
    n = args.n or 32
    w = wl.conv_workload(n=n, batch=args.batch, device=dev)
    N = w.params.shape[1]
    X0 = torch.zeros((n, wl.padded_ld(N)), device=dev)
    X0[:, :N] = w.params
    ctx = binding.Dpsgd(n, N, *wl.ring(n), gamma=0.1)
    ctx.bind(X0, torch.zeros_like(X0), torch.zeros_like(X0))
    offs, off = [], 0
    for (cin, cout, _) in w.plan:
        offs.append((off, off + cout * cin * 9))
        off += cout * cin * 9 + cout
    acts, hw = [w.inputs], 32
    for (cin, cout, stride) in w.plan:
        hw = (hw - 1) // stride + 1
        acts.append(torch.empty((n, args.batch, cout, hw, hw), device=dev))

    def layer(l):
        (cin, cout, stride), (wo, bo) = w.plan[l], offs[l]
        ctx.conv3x3_forward(acts[l], cout, stride, wo, bo, True, acts[l + 1])

    for _ in range(args.warmup):
        for l in range(len(w.plan)):
            layer(l)
    per_layer = []
    for l, (cin, cout, stride) in enumerate(w.plan):
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.steps):
            layer(l)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / args.steps
        flops = 2.0 * 9 * cin * cout * acts[l + 1].shape[3] * acts[l + 1].shape[4] * n * args.batch
        moved = 4 * (acts[l].numel() + acts[l + 1].numel())
        per_layer.append({"layer": [cin, cout, stride], "ms": ms, "fp32_equivalent_TFLOPs": flops / ms / 1e9,
                          "GBps": moved / ms / 1e6})
    out = {"workload": "conv3x3 forward, CIFAR-shaped layers", "n": n, "batch": args.batch,
           "ms_per_forward": sum(p["ms"] for p in per_layer), "layers": per_layer}
    if args.backward:
        # filter, bias and input gradients of every layer from a random gradient at its output (layer 1: no input gradient)
        for l, (cin, cout, stride) in enumerate(w.plan):
            dy = torch.randn_like(acts[l + 1])
            run = lambda: ctx.conv3x3_backward(acts[l], acts[l + 1], dy, stride, offs[l][0], offs[l][1], True, cin % 16 == 0)
            for _ in range(args.warmup):
                run()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(args.steps):
                run()
            b.record()
            torch.cuda.synchronize()
            per_layer[l]["ms_backward"] = a.elapsed_time(b) / args.steps
        out["ms_per_backward"] = sum(p["ms_backward"] for p in per_layer)
    ctx.sync()
    print(json.dumps(out))
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=2, choices=[0, 1, 2, 3, 4])
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--n", type=int, default=0, help="override the node count")
    ap.add_argument("--N", type=int, default=0, help="config 3: parameters per replica (default 25,000,000)")
    ap.add_argument("--kind", type=int, default=-1, help="config 3: force a DPSGD_MIX_* kernel")
    ap.add_argument("--conv", action="store_true", help="time the convolution layer family instead of a configuration")
    ap.add_argument("--batch", type=int, default=32, help="--conv: images per node")
    ap.add_argument("--backward", action="store_true", help="--conv: also time the backward of every layer")
    ap.add_argument("--momentum", type=float, default=0.0,
                    help="config 3: momentum of the Section 5.3 runs (one more matrix)")
    ap.add_argument("--m", type=int, default=0, help="override the local dataset size")
    ap.add_argument("--topology", default="")
    ap.add_argument("--precision", type=int, default=0, help="MLP: 0 fp32-faithful, 1 single TF32 pass")
    ap.add_argument("--consensus", action="store_true", help="evaluate the consensus distance every step")
    ap.add_argument("--fused-consensus", action="store_true",
                    help="log the consensus distance every step from inside the gossip kernel")
    ap.add_argument("--swapped", action="store_true", help="footnote c: update locally, then average")
    ap.add_argument("--fused-step", type=int, default=None, nargs="?", const=1,
                    help="MLP: gossip step inside the weight-gradient kernels (those blocks of G are never "
                         "written): 0 two stages, 1 where it is faster (the library's default), 2 wherever a "
                         "fused kernel applies, 3 as 2 without the ring kernel")
    args = ap.parse_args()

    build.build()
    dev = torch.device("cuda", 0)
    if args.conv:
        return conv_layers(args, dev)
    if args.config == 3:
        return gossip_step_alone(args, dev)
    over = {}
    if args.n:
        over["n"] = args.n
    if args.m:
        over["m"] = args.m
    if args.topology:
        over["topology"] = args.topology
    w = wl.config(args.config, device=dev, **over)
    X0 = wl.stack_rows(w.x0, w.n, w.ld)
    X1, G = torch.zeros_like(X0), torch.zeros_like(X0)
    ctx = binding.Dpsgd(w.n, w.N, *w.csr(), gamma=w.gamma, seed=1)
    ctx.bind(X0, X1, G)
    ctx.set_model(w.model, w.dims, w.l2_lambda, w.batch, args.precision)
    ctx.set_data(w.A, w.y)

    def timed(fn, reps):
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for k in range(reps):
            fn(k)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    if args.swapped:
        ctx.set_order(True)
    if args.fused_step is not None:
        ctx.set_fused_step(args.fused_step)
    for k in range(args.warmup):
        ctx.step(k)
    l0 = ctx.launch_count()
    log = torch.zeros(args.steps + args.warmup + 8, dtype=torch.float64, device=dev)
    if args.fused_consensus:
        def whole(k):
            ctx.step_consensus(args.warmup + k, log[k:k + 1])
    elif args.consensus:
        def whole(k):
            ctx.step(args.warmup + k)
            ctx.consensus_dist()
    else:
        def whole(k):
            ctx.step(args.warmup + k)
    ms_step = timed(whole, args.steps)
    launches = (ctx.launch_count() - l0) / args.steps
    # the same iterations enqueued by one library call (no per-step binding overhead)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    ctx.run(args.warmup + args.steps, args.steps)
    b.record()
    torch.cuda.synchronize()
    ms_run = a.elapsed_time(b) / args.steps
    ms_grad = timed(lambda k: ctx.grad(k), max(3, args.steps // 5))
    ms_mix = timed(lambda k: ctx.mix_update(), max(3, args.steps // 5))
    print(json.dumps({
        "workload": w.name, "n": w.n, "N": w.N, "dims": list(w.dims), "batch": w.batch, "topology": w.topology,
        "fused_step": args.fused_step, "mix_kernel": binding.MIX_NAMES[ctx.mix_kind()], "ms_per_step": ms_step, "ms_per_step_one_call": ms_run,
        "replica_steps_per_s": w.n / (ms_step * 1e-3), "ms_grad": ms_grad, "ms_mix_update": ms_mix,
        "launches_per_step": launches, "consensus": ctx.consensus_dist()}))
    ctx.close()


if __name__ == "__main__":
    main()
