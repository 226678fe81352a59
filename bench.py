#!/usr/bin/env python
"""Benchmark of the D-PSGD gossip step on the bandwidth configuration.

Workload: n = 64 replicas x N = 25,000,000 fp32 parameters (6.4 GB of X), gradients supplied
(N(0,1)), gamma = 0.01, ring topology of Theorem 3 (the 8x8 torus and the dense averaging
matrix are timed as well and reported under "topologies").  A step is one call of
dpsgd_mix_update: X_next = W X - gamma G for all replicas.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  With --gpus N > 1 (launched under torchrun) every rank runs an
independent replica of the workload on its own GPU (the path does not shard: no data-path
collective); the reported time is the maximum over ranks.
--impl reference times the CPU oracle on the host cores on a bounded column sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

N_NODES = 64
N_PARAMS = 25_000_000
GAMMA = 0.01
BYTES_PER_REPLICA_PARAM = 12          # read X, read G, write X_next (fp32 each)
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
METRIC = "replica-steps/s at n nodes; fused mix+update HBM GB/s vs B200 peak"
ORACLE_SAMPLE_COLS = 5_000_000          # columns per oracle step in BOTH CPU legs (vectors beyond any host cache)


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "25"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [t.strip() for t in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.2 and len(r) >= 7] or \
               [r for (_, r) in self.rows if len(r) >= 7]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(float(r[0]) for r in rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [nm for j, nm in enumerate(names) if any(r[3 + j].lower().startswith("active") for r in rows)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][1]),
                "power_w_max": max(float(r[2]) for r in rows), "samples": len(rows), "reasons": reasons}


def oracle_gossip_sample(cols, steps, warmup):
    """Times the oracle's gossip step, as it stands (one numpy thread), on the first `cols` columns of
    all 64 rows.  Returns seconds per call."""
    import numpy as np
    from oracle import dpsgd_oracle as orc
    from paper_1705_09056_b200 import workloads as wl
    rng = np.random.default_rng(1)
    X = rng.standard_normal((N_NODES, cols), dtype=np.float32)
    G = rng.standard_normal((N_NODES, cols), dtype=np.float32)
    csr = wl.topology("ring", N_NODES)
    for _ in range(warmup):
        orc.mix_update(X[:, :cols // 16], G[:, :cols // 16], *csr, GAMMA)
    t0 = time.perf_counter()
    for _ in range(steps):
        X = orc.mix_update(X, G, *csr, GAMMA)
    return (time.perf_counter() - t0) / steps


def oracle_sample_text(cols):
    return (f"first {cols} of {N_PARAMS} columns of all {N_NODES} rows per step (the step acts on every column "
            "alone); value = replica-steps/s of a full step extrapolated linearly in the columns")


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: a bounded column sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cols = min(N_PARAMS, max(1, args.ref_cols))
    dt = oracle_gossip_sample(cols, args.steps, args.warmup)
    scale = N_PARAMS / cols
    value = N_NODES / (dt * scale)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "replica-steps/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3,                      # measured: one call on the sample
        "sample_to_full_step_scale": scale,           # a full step = scale x the sample
        "ms_per_full_step_extrapolated": dt * 1e3 * scale,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config("ring"),
        "cpu_baseline": {"value": value, "unit": "replica-steps/s", "cores": 1, "kind": "oracle",
                         "host_cores_available": os.cpu_count(), "sample": oracle_sample_text(cols)},
        "e2e": {"value": value, "unit": "replica-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(topology):
    return {"workload": "mix+update bandwidth stress: n=64 replicas x N=25,000,000 fp32 (6.4 GB of X), "
                        "gradients supplied, gamma=0.01",
            "n": N_NODES, "N": N_PARAMS, "topology": topology, "gamma": GAMMA,
            "l2": "no flush needed: 19.2 GB touched per step >> 126 MB L2",
            "parallelism": "replicas only (one GPU per independent replica)"}


def max_over_ranks(seconds_or_ms: float, device) -> float:
    """Slowest rank's time.  A timing reduction only: the replicas exchange no data."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(seconds_or_ms)
    t = torch.tensor([seconds_or_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(replicas_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job replica-steps/s of `world` independent replicas timed by the slowest rank."""
    return world * replicas_per_rank / (ms_per_step * 1e-3)


def time_steps(ctx, steps, warmup, torch):
    for _ in range(warmup):
        ctx.mix_update()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        ctx.mix_update()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / steps    # ms per step == per launch (one kernel per step)


# dpsgd_step_consensus after a fused MLP iteration: False while the distance is a pass of its own over the
# new X; the two-stage ring / uniform gossip kernels always accumulate it on the way.
FUSED_STEP_CONSENSUS_IN_PASS = False


def _event_ms(torch, fn, reps):
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    fn(reps)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def _entry(n, ms, launches, bytes_per_step, peak, l2_resident=False):
    """One timed variant: rate, launches, algorithmic HBM bytes of an iteration and what bounds it."""
    gbs = bytes_per_step / (ms * 1e-3) / 1e9
    e = {"ms_per_step": ms, "replica_steps_per_s": n / (ms * 1e-3), "launches_per_step": launches,
         "algorithmic_bytes_per_step": bytes_per_step, "GBps": gbs}
    if l2_resident:
        e["bound"] = f"latency: {launches:g} dependent launches of {ms * 1e3 / max(launches, 1):.1f} us each"
    else:
        e["bound"] = "hbm"
        e["frac_of_measured_peak"] = gbs / peak
    return e


def mlp_bytes(n, dims, fused, consensus_pass):
    """Algorithmic HBM bytes of one MLP iteration, per replica-parameter of each weight block (fp32):
    forward reads the weights (4); the input gradient re-reads the hidden layers' weights (4, not layer 1);
    two stages: the gradient is written (4) and the gossip step reads X and G and writes X' (12);
    fused: the weight-gradient kernel reads X and writes X' (8); a separate consensus pass reads X' (4)."""
    P = sum(dims[l + 1] * dims[l] + dims[l + 1] for l in range(len(dims) - 1))
    hidden = sum(dims[l + 1] * dims[l] for l in range(1, len(dims) - 1))
    per = 4 * P + 4 * hidden + (8 * P if fused else 16 * P) + (4 * P if consensus_pass else 0)
    return n * per


def oracle_mlp_baseline(orc, w, nodes, cols):
    """Oracle, one numpy thread: gradients of `nodes` of the n nodes and the gossip step on the first `cols`
    columns of all rows, each scaled linearly to the whole iteration."""
    import numpy as np
    A, y, x0 = w.A[:nodes].cpu().numpy(), w.y[:nodes].cpu().numpy(), w.x0.cpu().numpy()
    idx = orc.sample_indices(1, 0, w.n, w.batch, w.m_per_node)
    t0 = time.perf_counter()
    for i in range(nodes):
        orc.grad_mlp(x0, w.dims, A[i], y[i], idx[i])
    t_grad = (time.perf_counter() - t0) * w.n / nodes
    cols = min(cols, w.N)
    X = np.tile(x0[:cols], (w.n, 1))
    t0 = time.perf_counter()
    orc.mix_update(X, X, *w.csr(), w.gamma)
    t_mix = (time.perf_counter() - t0) * w.N / cols
    return {"value": w.n / (t_grad + t_mix), "unit": "replica-steps/s", "cores": 1, "kind": "oracle",
            "host_cores_available": os.cpu_count(),
            "sample": f"gradients of {nodes} of {w.n} nodes and the gossip step on the first {cols} of {w.N} columns, "
                      f"each scaled linearly to one whole iteration ({t_grad:.2f} s + {t_mix:.2f} s)"}


def linear_iterations(torch, binding, wl, dev, peak, cpu_legs, steps=200, warmup=10):
    """Configurations 1 and 2 (least squares n=8; logistic regression n=16 with 65536 x 4096 samples per node):
    whole iterations per dpsgd_step call and enqueued by one dpsgd_run call."""
    import numpy as np
    out = {}
    for name, idx in (("lsq_64_n8_ring", 0), ("logistic_4096_n16_ring_65536_samples_per_node", 1)):
        free, _ = torch.cuda.mem_get_info()
        if idx == 1 and free < 24 * 2 ** 30:
            out[name] = {"skipped": "needs 24 GiB of free device memory for the 17.2 GB dataset"}
            continue
        w = wl.config(idx, device=dev)
        X0 = wl.stack_rows(w.x0, w.n, w.ld)
        X1, G = torch.zeros_like(X0), torch.zeros_like(X0)
        ctx = binding.Dpsgd(w.n, w.N, *w.csr(), gamma=w.gamma, seed=1)
        ctx.bind(X0, X1, G)
        ctx.set_model(w.model, w.dims, w.l2_lambda, w.batch, 0)
        ctx.set_data(w.A, w.y)
        for k in range(warmup):
            ctx.step(k)
        ctx.run(warmup, 64)                 # first use of the replay path (captures its graph where it applies)
        # sampled rows are read once (second use from the chip), then the 12 B/unit gossip step
        bytes_step = 4 * w.n * w.batch * (w.dims[0] + 1) + 12 * w.n * w.N
        l0 = ctx.launch_count()
        ms_step = _event_ms(torch, lambda r: [ctx.step(100 + k) for k in range(r)], steps)
        launches = (ctx.launch_count() - l0) / steps
        l0 = ctx.launch_count()
        ms_run = _event_ms(torch, lambda r: ctx.run(1000, r), steps)
        launches_run = (ctx.launch_count() - l0) / steps
        res = {"n": w.n, "N": w.N, "batch": w.batch, "iterations_of_the_configuration": w.iterations,
               "per_dpsgd_step_call": _entry(w.n, ms_step, launches, bytes_step, peak, l2_resident=True),
               "one_dpsgd_run_call": _entry(w.n, ms_run, launches_run, bytes_step, peak, l2_resident=True)}
        ctx.sync()
        if cpu_legs:
            from oracle import dpsgd_oracle as orc
            reps = 20 if idx == 0 else 3
            ids = orc.sample_indices(1, 0, w.n, w.batch, w.m_per_node)
            it = torch.from_numpy(ids.astype(np.int64)).to(dev)
            node = torch.arange(w.n, device=dev)[:, None]
            A_s, y_s = w.A[node, it].cpu().numpy(), w.y[node, it].cpu().numpy()     # the sampled rows only
            local = np.tile(np.arange(w.batch, dtype=np.int32), (w.n, 1))
            X = np.zeros((w.n, w.N), dtype=np.float32)
            t0 = time.perf_counter()
            for _ in range(reps):
                Gr = orc.gradients(X, w.model, w.dims, A_s, y_s, local, w.l2_lambda)
                X = orc.mix_update(X, Gr, *w.csr(), w.gamma)
            dt = (time.perf_counter() - t0) / reps
            res["cpu_baseline"] = {"value": w.n / dt, "unit": "replica-steps/s", "cores": 1, "kind": "oracle",
                                   "host_cores_available": os.cpu_count(),
                                   "sample": f"{reps} whole iterations (gradients of all {w.n} nodes + gossip step) on the "
                                             "rows one minibatch draws, gathered outside the timed region"}
        ctx.close()
        out[name] = res
        del X0, X1, G, w
        torch.cuda.empty_cache()
    return out


def mlp_iterations(torch, binding, wl, dev, peak, cpu_legs, steps=20, warmup=3):
    """Configurations 3 and 5: whole iterations, two-stage and with the gossip step inside the gradient
    kernels.  Configuration 5 (n = 112, ring beside the averaging matrix of C-PSGD) is defined as reporting
    the consensus distance in every iteration, so dpsgd_step_consensus is the timed call there; the same
    iterations without the distance are given beside it."""
    out = {}
    for name, idx, topo, per_step_consensus in (
            ("mlp_784-1024-10_n32_ring", 2, "ring", False),
            ("mlp_1024-2048-2048-10_n112_ring", 4, "ring", True),
            ("mlp_1024-2048-2048-10_n112_dense_cpsgd_averaging", 4, "dense", True)):
        w = wl.config(idx, device=dev, topology=topo)
        X0 = wl.stack_rows(w.x0, w.n, w.ld)
        X1, G = torch.zeros_like(X0), torch.zeros_like(X0)
        log = torch.zeros(steps + warmup, dtype=torch.float64, device=dev)
        res = {"n": w.n, "N": w.N, "batch": w.batch, "iterations_of_the_configuration": w.iterations}
        l2_resident = 3 * w.n * w.ld * 4 < 126e6 * 3          # configuration 3: X (104 MB) stays in L2
        for label, mode in (("two_stage", 0), ("fused", 1)):
            X0.copy_(wl.stack_rows(w.x0, w.n, w.ld))
            ctx = binding.Dpsgd(w.n, w.N, *w.csr(), gamma=w.gamma, seed=1)
            ctx.bind(X0, X1, G)
            ctx.set_model(w.model, w.dims, w.l2_lambda, w.batch, 0)
            ctx.set_data(w.A, w.y)
            ctx.set_fused_step(mode)
            variants = [("", lambda k: ctx.step(k), False)]
            if per_step_consensus:
                variants = [("_consensus_every_step", lambda k: ctx.step_consensus(k, log[k:k + 1]), True)] + variants
            for suffix, call, with_c in variants:
                for k in range(warmup):
                    call(k)
                l0 = ctx.launch_count()
                ms = _event_ms(torch, lambda r: [call(warmup + k) for k in range(r)], steps)
                launches = (ctx.launch_count() - l0) / steps
                # the distance costs a pass of its own unless the gossip kernel accumulates it on the way
                own_pass = with_c and mode == 1 and not FUSED_STEP_CONSENSUS_IN_PASS
                e = _entry(w.n, ms, launches, mlp_bytes(w.n, w.dims, mode == 1, own_pass), peak, l2_resident)
                if with_c:
                    e["consensus_dist_last_step"] = float(log[warmup + steps - 1])
                    e["consensus_pass"] = "separate pass over the new X" if own_pass else "inside the gossip kernels"
                res[label + suffix] = e
            res[label]["consensus_dist"] = ctx.consensus_dist()
            ctx.close()
        if cpu_legs:
            from oracle import dpsgd_oracle as orc
            res["cpu_baseline"] = oracle_mlp_baseline(orc, w, nodes=4, cols=500_000)
        out[name] = res
        del X0, X1, G, w
        torch.cuda.empty_cache()
    return out


def conv_layers(torch, binding, wl, dev, peak, cpu_legs, n=32, batch=32, reps=20):
    """The convolution layer family of the paper's image workloads (3x3, CIFAR-shaped 32x32x3 inputs, widths
    16/32/64): forward pass of the six layers for n nodes, every node with the filters of its own row."""
    w = wl.conv_workload(n=n, batch=batch, device=dev)
    N = w.params.shape[1]
    X0 = torch.zeros((n, wl.padded_ld(N)), device=dev)
    X0[:, :N] = w.params
    X1, G = torch.zeros_like(X0), torch.zeros_like(X0)
    ctx = binding.Dpsgd(n, N, *wl.ring(n), gamma=0.1)
    ctx.bind(X0, X1, G)
    offs, off = [], 0
    for (cin, cout, _) in w.plan:
        offs.append((off, off + cout * cin * 9))
        off += cout * cin * 9 + cout
    acts, hw = [w.inputs], 32
    for (cin, cout, stride) in w.plan:
        hw = (hw - 1) // stride + 1
        acts.append(torch.empty((n, batch, cout, hw, hw), device=dev))

    def forward(r):
        for _ in range(r):
            for l, ((cin, cout, stride), (wo, bo)) in enumerate(zip(w.plan, offs)):
                ctx.conv3x3_forward(acts[l], cout, stride, wo, bo, True, acts[l + 1])

    forward(3)
    l0 = ctx.launch_count()
    ms = _event_ms(torch, forward, reps)
    launches = (ctx.launch_count() - l0) / reps
    flops = sum(2.0 * 9 * cin * cout * acts[l + 1].shape[3] * acts[l + 1].shape[4] * n * batch
                for l, (cin, cout, _) in enumerate(w.plan))
    bytes_step = 4 * sum(a.numel() for a in acts[:-1]) + 4 * sum(a.numel() for a in acts[1:])   # every layer reads its input, writes its output
    res = {"n": n, "batch": batch, "layers": [list(p) for p in w.plan], "ms_per_forward": ms, "launches_per_forward": launches,
           "images_per_s": n * batch / (ms * 1e-3), "fp32_equivalent_TFLOPs": flops / (ms * 1e-3) / 1e12,
           "algorithmic_bytes_per_forward": bytes_step, "GBps": bytes_step / (ms * 1e-3) / 1e9,
           "frac_of_measured_peak": bytes_step / (ms * 1e-3) / 1e9 / peak}
    ctx.sync()
    if cpu_legs:
        from oracle import conv_oracle as co
        x = w.inputs[0, :4].cpu().numpy()
        prm = w.params[0].cpu().numpy()
        t0 = time.perf_counter()
        co.layers_forward(x, prm, w.plan)
        dt = time.perf_counter() - t0
        res["cpu_baseline"] = {"value": 4 / dt, "unit": "images/s", "cores": 1, "kind": "oracle",
                               "host_cores_available": os.cpu_count(),
                               "sample": "the six layers on 4 images of one node (fp64 einsum per filter tap)"}
    ctx.close()
    return res


def whole_iterations(torch, binding, wl, dev, peak, cpu_legs=True):
    """Whole D-PSGD iterations (sample + gradient + mix + update) of the four model configurations.
    Context for the headline line, which times the gossip step alone on configuration 4."""
    out = linear_iterations(torch, binding, wl, dev, peak, cpu_legs)
    out.update(mlp_iterations(torch, binding, wl, dev, peak, cpu_legs))
    out["conv3x3_forward_cifar_layers_n32"] = conv_layers(torch, binding, wl, dev, peak, cpu_legs)
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1705_09056_b200 import binding, workloads as wl, build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    binding.load_library()

    n, N = N_NODES, N_PARAMS
    ld = wl.padded_ld(N)
    X0 = wl.stress_matrix(n, ld, N, 100 + rank, dev)
    X1 = torch.zeros_like(X0)
    G = wl.stress_matrix(n, ld, N, 200 + rank, dev)
    peak, peak_kind = measured_peak()
    bytes_per_launch = BYTES_PER_REPLICA_PARAM * n * N

    results = {}
    clocks = None
    launches = 0
    for topo in ("torus", "dense", "ring"):            # the headline topology last
        ctx = binding.Dpsgd(n, N, *wl.topology(topo, n), gamma=GAMMA, seed=rank)
        ctx.bind(X0, X1, G)
        kind = binding.MIX_NAMES[ctx.mix_kind()]
        if topo != "ring":
            ms = time_steps(ctx, max(5, args.steps // 5), args.warmup, torch)
        else:
            for _ in range(args.warmup):
                ctx.mix_update()
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            sampler = ClockSampler(local)
            if rank == 0:
                sampler.start()
                time.sleep(0.3)
            l0 = ctx.launch_count()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.time()
            a.record()
            for _ in range(args.steps):
                ctx.mix_update()
            b.record()
            torch.cuda.synchronize()
            t1 = time.time()
            if world > 1:
                dist.barrier()
            ms = a.elapsed_time(b) / args.steps
            launches = ctx.launch_count() - l0
            if rank == 0:
                clocks = sampler.stop(t0, t1)
            ms = max_over_ranks(ms, dev)
        gbs = bytes_per_launch / (ms * 1e-3) / 1e9
        results[topo] = {"kernel": kind, "ms_per_step": ms, "replica_steps_per_s": n / (ms * 1e-3),
                         "GBps": gbs, "frac_of_measured_peak": gbs / peak,
                         "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS}
        ring_ctx = ctx if topo == "ring" else None
        if topo != "ring":
            ctx.close()

    # a read-only streaming pass over the same 6.4 GB (the consensus reduction, 4 B per unit): the copy figure the
    # fractions are quoted against mixes reads and writes 1:1, the gossip step 2:1; this one is the read-only end
    read_only_gbs = None
    if rank == 0:
        outd = torch.zeros(1, dtype=torch.float64, device=dev)
        for _ in range(3):
            binding.consensus_dist_noalloc(X0, N, outd)
        ms_r = _event_ms(torch, lambda r: [binding.consensus_dist_noalloc(X0, N, outd) for _ in range(r)], 10)
        read_only_gbs = 4.0 * n * N / (ms_r * 1e-3) / 1e9

    # end to end through the host-buffer entry point: pinned G -> device, step, consensus -> host
    e2e = None
    if rank == 0 or world > 1:
        try:
            Gh = torch.empty((n, N), dtype=torch.float32, pin_memory=True)
            Gh.normal_()
            ring_ctx.mix_update_host(Gh)           # warm-up
            torch.cuda.synchronize()
            k_e2e = max(1, min(args.steps, args.e2e_steps))
            t0 = time.perf_counter()
            for _ in range(k_e2e):
                ring_ctx.mix_update_host(Gh)
            torch.cuda.synchronize()
            dt = (time.perf_counter() - t0) / k_e2e
            dt = max_over_ranks(dt, dev)
            e2e = {"value": world * n / dt, "unit": "replica-steps/s", "h2d_bytes_per_step": 4 * n * N,
                   "d2h_bytes_per_step": 8, "steps": k_e2e, "ms_per_step": dt * 1e3,
                   "call": "dpsgd_mix_update_host (pinned host G -> device, mix+update, consensus distance -> host)"}
            del Gh
        except Exception as ex:               # e.g. the host cannot pin 6.4 GB
            e2e = {"value": None, "unit": "replica-steps/s", "error": str(ex)[:200]}
    ring_ctx.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cols = ORACLE_SAMPLE_COLS
        dt = oracle_gossip_sample(cols, 2, 1)
        cpu = {"value": n / (dt * N / cols), "unit": "replica-steps/s", "cores": 1, "kind": "oracle",
               "host_cores_available": os.cpu_count(), "seconds_per_sample_step": dt,
               "sample": oracle_sample_text(cols)}

    iterations = None
    if world == 1 and not args.no_iterations:
        del X0, X1, G
        torch.cuda.empty_cache()
        iterations = whole_iterations(torch, binding, wl, dev, peak, cpu_legs=not args.no_cpu_baseline)

    ring = results["ring"]
    line = {
        "metric": METRIC, "value": aggregate_throughput(n, world, ring["ms_per_step"]), "unit": "replica-steps/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ring["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": workload_config("ring"),
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": "mix_ring_kernel", "achieved": ring["GBps"], "peak": peak,
                     "peak_source": f"{peak_kind} HBM copy bandwidth (GB/s): a torch copy, a baseline rather than a ceiling",
                     "read_only_stream_GBps": read_only_gbs, "unit": "GB/s",
                     "frac": ring["GBps"] / peak, "frac_of_nominal_8TBps": ring["GBps"] / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_launch": bytes_per_launch, "traffic": traffic_bytes_per_launch()},
        "cpu_baseline": cpu, "topologies": results, "iterations": iterations,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of one mix_ring_kernel launch.  Captured with ncu on
# n = 64 x N = 2,000,000 (1.499 GB against 1.536 GB algorithmic) and scaled by 25,000,000 / 2,000,000:
# traffic grows in proportion to N.  The figure belongs to the kernel source it was captured from: when
# the file's hash differs, the line reports null until the counters are taken again.
TRAFFIC_CAPTURE = {"bytes_per_launch": 18.74e9, "source": "paper_1705_09056_b200/csrc/mix_update.cu",
                   "sha256_16": "e24eac603b395f6a"}


def traffic_bytes_per_launch():
    import hashlib
    try:
        with open(os.path.join(ROOT, TRAFFIC_CAPTURE["source"]), "rb") as f:
            same = hashlib.sha256(f.read()).hexdigest()[:16] == TRAFFIC_CAPTURE["sha256_16"]
    except OSError:
        same = False
    return TRAFFIC_CAPTURE["bytes_per_launch"] if same else None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--ref-cols", type=int, default=ORACLE_SAMPLE_COLS,
                    help="columns per step of the CPU reference arm (bounded sample)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-iterations", action="store_true",
                    help="skip the whole-iteration timings of the MLP configurations")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
