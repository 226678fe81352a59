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
ORACLE_SAMPLE_COLS = 10_000_000


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


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: a bounded column sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from oracle import dpsgd_oracle as orc
    from paper_1705_09056_b200 import workloads as wl
    cols = min(N_PARAMS, max(1, args.ref_cols))
    rng = np.random.default_rng(1)
    X = rng.standard_normal((N_NODES, cols), dtype=np.float32)
    G = rng.standard_normal((N_NODES, cols), dtype=np.float32)
    csr = wl.topology("ring", N_NODES)
    for _ in range(args.warmup):
        orc.mix_update(X[:, :cols // 16], G[:, :cols // 16], *csr, GAMMA)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        X = orc.mix_update(X, G, *csr, GAMMA)
    dt = (time.perf_counter() - t0) / args.steps
    value = N_NODES * (cols / N_PARAMS) / dt
    sample = f"first {cols} of {N_PARAMS} columns of all {N_NODES} rows per step (the step is separable per column), scaled linearly"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "replica-steps/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3 * N_PARAMS / cols,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config("ring"),
        "cpu_baseline": {"value": value, "unit": "replica-steps/s", "cores": 1, "kind": "oracle", "sample": sample},
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


def whole_iterations(torch, binding, wl, dev, steps=20, warmup=3):
    """Whole D-PSGD iterations (sample + gradient + mix + update; consensus distance read once at the end)
    on the two MLP configurations (the larger one also with the dense averaging matrix, its C-PSGD
    baseline), two-stage and with the gossip step inside the gradient kernels.
    Context for the headline line, which times the gossip step alone."""
    out = {}
    for name, idx, topo in (("mlp_784-1024-10_n32_ring", 2, "ring"), ("mlp_1024-2048-2048-10_n112_ring", 4, "ring"),
                            ("mlp_1024-2048-2048-10_n112_dense_cpsgd_averaging", 4, "dense")):
        w = wl.config(idx, device=dev, topology=topo)
        X0 = wl.stack_rows(w.x0, w.n, w.ld)
        X1, G = torch.zeros_like(X0), torch.zeros_like(X0)
        log = torch.zeros(steps + warmup, dtype=torch.float64, device=dev)
        res = {"n": w.n, "N": w.N, "batch": w.batch}
        for label, mode in (("two_stage", 0), ("fused", 1)):
            X0.copy_(wl.stack_rows(w.x0, w.n, w.ld))
            ctx = binding.Dpsgd(w.n, w.N, *w.csr(), gamma=w.gamma, seed=1)
            ctx.bind(X0, X1, G)
            ctx.set_model(w.model, w.dims, w.l2_lambda, w.batch, 0)
            ctx.set_data(w.A, w.y)
            ctx.set_fused_step(mode)
            for k in range(warmup):
                ctx.step(k)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            l0 = ctx.launch_count()
            a.record()
            for k in range(steps):
                ctx.step(warmup + k)
            b.record()
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / steps
            res[label] = {"ms_per_step": ms, "replica_steps_per_s": w.n / (ms * 1e-3),
                          "launches_per_step": (ctx.launch_count() - l0) / steps,
                          "consensus_dist": ctx.consensus_dist()}
            ctx.close()
        out[name] = res
        del X0, X1, G, w
        torch.cuda.empty_cache()
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
        import numpy as np
        from oracle import dpsgd_oracle as orc
        cols = ORACLE_SAMPLE_COLS
        rng = np.random.default_rng(1)
        Xs = rng.standard_normal((n, cols), dtype=np.float32)
        Gs = rng.standard_normal((n, cols), dtype=np.float32)
        csr = wl.topology("ring", n)
        t0 = time.perf_counter()
        orc.mix_update(Xs, Gs, *csr, GAMMA)
        dt = time.perf_counter() - t0
        cpu = {"value": n * (cols / N) / dt, "unit": "replica-steps/s", "cores": 1, "kind": "oracle",
               "host_cores_available": os.cpu_count(), "seconds": dt,
               "sample": f"one step on the first {cols} of {N} columns of all {n} rows "
                         "(separable per column), scaled linearly to a full step"}

    iterations = None
    if world == 1 and not args.no_iterations:
        del X0, X1, G
        torch.cuda.empty_cache()
        iterations = whole_iterations(torch, binding, wl, dev)

    ring = results["ring"]
    line = {
        "metric": METRIC, "value": aggregate_throughput(n, world, ring["ms_per_step"]), "unit": "replica-steps/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ring["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": workload_config("ring"),
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": "mix_ring_kernel", "achieved": ring["GBps"], "peak": peak,
                     "peak_source": f"{peak_kind} HBM copy bandwidth (GB/s)", "unit": "GB/s",
                     "frac": ring["GBps"] / peak, "frac_of_nominal_8TBps": ring["GBps"] / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_launch": bytes_per_launch, "traffic": TRAFFIC_BYTES_PER_LAUNCH},
        "cpu_baseline": cpu, "topologies": results, "iterations": iterations,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of one mix_ring_kernel launch.  Captured with ncu on
# n = 64 x N = 2,000,000 (1.499 GB against 1.536 GB algorithmic) and scaled by 25,000,000 / 2,000,000:
# traffic grows in proportion to N.  Set to None whenever mix_ring_kernel changes.
TRAFFIC_BYTES_PER_LAUNCH = 18.74e9


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--ref-cols", type=int, default=1_000_000,
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
