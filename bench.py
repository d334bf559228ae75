#!/usr/bin/env python
"""Benchmark of the DD-EF-SGD hot path (error-feedback Top-k compress + stale aggregate +
apply) on B200.  One "step" is one pass of the whole path over one batch of synthetic
gradients for all n simulated workers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is gradient GB/s (n*d*sizeof(g) bytes per step over
the device-timed step), whole job; with N > 1 every rank runs an independent replica (the
path does not shard), timed as the max over ranks.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "ef_topk_compress_stale_aggregate_step_gradient_throughput"
UNIT = "GB/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18")
    ap.add_argument("--select-mode", default="auto", choices=["auto", "exact"])
    ap.add_argument("--pool", type=int, default=0, help="distinct gradient batches kept in HBM")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--delta", type=float, default=None)
    ap.add_argument("--tau", type=int, default=None)
    ap.add_argument("--compressor", default="topk", choices=["topk", "randk"])
    ap.add_argument("--shard-workers", action="store_true",
                    help="N > 1: split the workers over the ranks (sparse all-gather per step) "
                         "instead of running N replicas; strong scaling")
    ap.add_argument("--per-layer", action="store_true",
                    help="per-layer Top-k variant: k(delta, d_l) entries of every tensor of the workload "
                         "(deco_layered_step); no per-kernel timing, no e2e")
    ap.add_argument("--scale", type=float, default=1.0,
                    help="shrink the workload's layer widths (profiling captures of the large shapes)")
    return ap.parse_args()


# --------------------------------------------------------------------------- helpers

def measured_peaks():
    """HBM copy bandwidth measured on this machine (generated file), else the fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append((time.time(), ln.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        inside = [ln for (ts, ln) in self.lines if t0 <= ts <= t1 + 0.1]
        rows = inside if inside else [ln for _, ln in self.lines[-3:]]
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in rows:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm),
                "samples_in_timed_region": len(inside)}


def max_over_ranks(ms, dist, device):
    """Slowest rank's time: every rank ends up with the same number (MAX all-reduce)."""
    if dist is None:
        return float(ms)
    import torch
    tt = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_value(bytes_per_replica_step, world, ms_per_step):
    """Gradient GB/s of the whole job: every replica processes its own batch per step."""
    return world * bytes_per_replica_step / (ms_per_step * 1e-3) / 1e9


def workload_for(args):
    from paper_2507_17346_b200 import workloads as W
    wl = W.make_workload(args.workload, args.scale)
    if args.delta is not None:
        wl.delta = args.delta
    if args.tau is not None:
        wl.tau = args.tau
    return wl


def grad_bytes(wl):
    return wl.n * wl.d * (4 if wl.grad_dtype == "f32" else 2)


# DRAM read + write bytes of one ef_accumulate_kernel launch from the ncu captures summarised in
# profiles/ef_accumulate_kernel_dram_traffic.md (taken on this kernel version).  resnet18 was
# captured at full size; the others at reduced size (--scale) and are scaled by the entry count:
# the kernel streams every entry once, so its traffic grows in proportion.
NCU_TRAFFIC_BYTES = {
    "resnet18": 1075.3e6,
    "gpt2_small": 1585.7e6 * (995518464 / 163946496),
    "decoder_1b": 2110.6e6 * (4400193536 / 216158400),
    "sweep_100m": 1155.0e6 * (400000000 / 100000000),
}


def algorithmic_bytes_accumulate(wl):
    """Streaming pass: read e (4), read g (4 or 2), write e (4) per entry and worker."""
    return wl.n * wl.d * (8 + (4 if wl.grad_dtype == "f32" else 2))


# --------------------------------------------------------------------- reference arm

def oracle_throughput(wl, steps, warmup, budget_s=25.0):
    """The CPU oracle as it stands, on a bounded sample of the workload: `m` of the n workers
    at full d, chosen so one step is a few seconds.  Returns (GB/s, ms_per_step, sample)."""
    import numpy as np
    import torch
    from oracle import dd_ef_sgd as O
    from paper_2507_17346_b200 import workloads as W
    torch.manual_seed(0)
    sz = 4 if wl.grad_dtype == "f32" else 2
    # about 0.1 us per entry and worker for accumulate + full sort + aggregate
    per_worker_s = 6e-8 * wl.d
    m = max(1, min(wl.n, int(budget_s / max(1e-9, per_worker_s * max(1, steps + warmup)))))
    d = wl.d
    if per_worker_s * (steps + warmup) > budget_s:
        d = max(1 << 16, int(wl.d * budget_s / (per_worker_s * (steps + warmup))))
    rng = np.random.default_rng(wl.seed)
    if wl.grad_dtype == "f32":
        g = (rng.standard_normal((m, d), dtype=np.float32) * np.float32(wl.sigma))
    else:
        g32 = rng.standard_normal((m, d), dtype=np.float32) * np.float32(wl.sigma)
        g = (g32.view(np.uint32) >> 16).astype(np.uint16)
    orc = O.DDEFSGD(d, m, wl.delta, wl.tau, wl.lr)
    for _ in range(warmup):
        orc.step(g)
    t0 = time.perf_counter()
    for _ in range(steps):
        orc.step(g)
    dt = time.perf_counter() - t0
    ms = 1e3 * dt / max(1, steps)
    gbs = m * d * sz * steps / dt / 1e9
    sample = "%d of %d workers, d=%d of %d, %d steps, oracle as is (numpy + C fmaf, 1 thread)" % (
        m, wl.n, d, wl.d, steps)
    return gbs, ms, sample


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = workload_for(args)
    steps = args.steps if args.steps is not None else 2
    warmup = args.warmup if args.warmup is not None else 1
    gbs, ms, sample = oracle_throughput(wl, steps, warmup)
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT,
            "n_gpus": args.gpus, "steps": steps, "warmup": warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "d": wl.d, "n": wl.n, "delta": wl.delta,
                       "tau": wl.tau, "grad_dtype": wl.grad_dtype},
            "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- our arm

def run_ours(args):
    import torch
    from paper_2507_17346_b200 import build as lib_build
    from paper_2507_17346_b200 import binding as B
    from paper_2507_17346_b200 import workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        lib_build.build()
    if dist is not None:
        dist.barrier()
    B.load()

    wl = workload_for(args)
    sz = 4 if wl.grad_dtype == "f32" else 2
    gbytes = grad_bytes(wl)
    # enough steps for a timed region that nvidia-smi can sample
    steps = args.steps if args.steps is not None else max(50, min(4000, int(8.0e12 / (6 * gbytes))))
    warmup = args.warmup if args.warmup is not None else 10
    warmup = max(3, warmup)
    pool_n = args.pool if args.pool > 0 else max(2, min(8, int(6e9 // gbytes)))
    pool = [W.gradients(wl, p, "cuda") for p in range(pool_n)]
    mode = B.DECO_SELECT_AUTO if args.select_mode == "auto" else B.DECO_SELECT_EXACT_PASSES
    sharded = args.shard_workers and world > 1
    n_local, base = wl.n, 0
    if sharded:
        if wl.n % world:
            raise SystemExit("--shard-workers needs the worker count to be a multiple of --gpus")
        n_local, base = wl.n // world, rank * (wl.n // world)
        pool = [p[base:base + n_local].clone() for p in pool]      # this rank's workers only
    if args.per_layer:
        return run_per_layer(args, wl, pool, pool_n, steps, warmup, local, world, rank, dist)
    ctx = B.deco_init(wl.d, n_local, wl.delta, wl.tau, wl.lr,
                      grad_dtype=B.DECO_F32 if wl.grad_dtype == "f32" else B.DECO_BF16,
                      device=local, select_mode=mode,
                      compressor=B.DECO_COMPRESSOR_RANDK if args.compressor == "randk"
                      else B.DECO_COMPRESSOR_TOPK, seed=wl.seed,
                      n_total=wl.n if sharded else 0, worker_base=base)
    stream = torch.cuda.current_stream()

    def one_step(g):
        if sharded:
            B.deco_step_sharded(ctx, g, None, stream, local)
        else:
            B.deco_step(ctx, g, stream)

    for t in range(warmup):
        one_step(pool[t % pool_n])
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    B.deco_set_kernel_timing(ctx, True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = B.deco_launch_count(ctx)
    t_wall0 = time.time()
    ev0.record(stream)
    for t in range(steps):
        one_step(pool[(warmup + t) % pool_n])
    B.deco_join(ctx, stream)            # the last aggregation ends inside the timed region
    ev1.record(stream)
    torch.cuda.synchronize()
    t_wall1 = time.time()
    if dist is not None:
        dist.barrier()
    launches = B.deco_launch_count(ctx) - launches0
    ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop(t_wall0, t_wall1)
    parts, iters = B.deco_get_kernel_timing(ctx, stream)
    B.deco_set_kernel_timing(ctx, False)
    stats = B.deco_get_stats(ctx, stream)

    ms_max = max_over_ranks(ms_total, dist, "cuda")
    ms_per_step = ms_max / steps
    # replicas: every rank steps the whole workload; sharded: the ranks share one workload
    value = whole_job_value(gbytes, 1 if sharded else world, ms_per_step)

    # end to end through the host-buffer entry point: H2D gradients, step, D2H messages
    e2e = None
    if not args.no_e2e and not sharded:
        k = B.deco_get_k(ctx)
        host_g = [p.cpu().pin_memory() for p in pool[:2]]
        host_msg = torch.empty((wl.n, k, 2), dtype=torch.int32).pin_memory()
        e_steps = max(3, min(steps, int(3.0 / max(1e-4, gbytes / 20e9))))
        for t in range(3):
            B.deco_step_host(ctx, host_g[t % 2], host_msg, None, stream)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for t in range(e_steps):
            B.deco_step_host(ctx, host_g[t % 2], host_msg, None, stream)
        B.deco_join(ctx, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        e_ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
        e2e = {"value": whole_job_value(gbytes, world, e_ms / e_steps), "unit": UNIT,
               "h2d_bytes_per_step": gbytes, "d2h_bytes_per_step": wl.n * k * 8,
               "steps": e_steps, "ms_per_step": e_ms / e_steps}
    B.deco_destroy(ctx)
    del pool

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    acc_ms = parts["accumulate"] / max(1, iters)
    acc_bytes = algorithmic_bytes_accumulate(wl) * n_local // wl.n      # this rank's launch
    achieved = acc_bytes / (acc_ms * 1e-3) / 1e9 if acc_ms > 0 else None
    roofline = {"bound": "hbm", "kernel": "ef_accumulate_kernel", "achieved": achieved,
                "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": (achieved / peak) if achieved else None,
                "traffic": NCU_TRAFFIC_BYTES.get(wl.name)
                if (args.scale == 1.0 and args.delta is None and args.compressor == "topk") else None,
                "algorithmic_bytes_per_launch": acc_bytes,
                "avg_launch_ms": acc_ms, "launches_timed": iters}
    step_alg_bytes = algorithmic_bytes_accumulate(wl)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "strong" if sharded else "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": wl.name, "d": wl.d, "n": wl.n, "delta": wl.delta,
                       "tau": wl.tau, "lr": wl.lr, "grad_dtype": wl.grad_dtype,
                       "k": stats["k"], "select_mode": args.select_mode,
                       "compressor": args.compressor,
                       "l2": "inputs larger than L2 (e and g of one step exceed 126 MB)"
                       if 2 * gbytes > 126e6 else "working set fits in L2",
                       "gradient_pool": pool_n, "replicas": 1 if sharded else world,
                       "parallelism": ("workers sharded over %d ranks" % world) if sharded
                       else "replicas only"},
            "step_algorithmic_GBps": step_alg_bytes / (ms_per_step * 1e-3) / 1e9,
            "step_frac_of_hbm_peak": step_alg_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
            "phases_ms": {k_: v / max(1, iters) for k_, v in parts.items()},
            "exact_pass_worker_steps": stats["exact_pass_workers"],
            "roofline": roofline, "clocks": clocks, "gpu_launches": launches}
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        gbs, ms, sample = oracle_throughput(wl, 2, 1)
        line["cpu_baseline"] = {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": sample, "ms_per_step_sample": ms}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_per_layer(args, wl, pool, pool_n, steps, warmup, local, world, rank, dist):
    """The per-layer Top-k variant on the workload's tensors: whole-step timing only."""
    import torch
    from paper_2507_17346_b200 import binding as B
    offsets = [0]
    for t in wl.tensors:
        offsets.append(offsets[-1] + int(t.numel))
    ctx = B.deco_layered_init(wl.d, wl.n, offsets, wl.delta, wl.tau, wl.lr,
                              grad_dtype=B.DECO_F32 if wl.grad_dtype == "f32" else B.DECO_BF16,
                              device=local)
    stream = torch.cuda.current_stream()
    for t in range(warmup):
        B.deco_layered_step(ctx, pool[t % pool_n], stream)
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t_wall0 = time.time()
    ev0.record(stream)
    for t in range(steps):
        B.deco_layered_step(ctx, pool[(warmup + t) % pool_n], stream)
    B.deco_layered_join(ctx, stream)
    ev1.record(stream)
    torch.cuda.synchronize()
    t_wall1 = time.time()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop(t_wall0, t_wall1)
    ms_per_step = max_over_ranks(ev0.elapsed_time(ev1), dist, "cuda") / steps
    info = B.deco_layered_info(ctx)
    fallbacks = 0
    for l in range(info["n_layers"]):
        sub, _, _ = B.deco_layered_layer(ctx, l)
        st = B.deco_get_stats(sub, stream)
        fallbacks += st["exact_pass_workers"]
        assert st["device_status"] == 0, (l, st)
    B.deco_layered_destroy(ctx)
    if rank == 0:
        peak, peak_kind = measured_peaks()
        alg = algorithmic_bytes_accumulate(wl)
        line = {"metric": METRIC, "value": whole_job_value(grad_bytes(wl), world, ms_per_step), "unit": UNIT,
                "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic",
                "config": {"workload": wl.name, "variant": "per-layer Top-k", "layers": info["n_layers"],
                           "d": wl.d, "n": wl.n, "delta": wl.delta, "tau": wl.tau, "lr": wl.lr,
                           "grad_dtype": wl.grad_dtype, "k_total": info["k_total"],
                           "gradient_pool": pool_n, "parallelism": "replicas only"},
                "step_algorithmic_GBps": alg / (ms_per_step * 1e-3) / 1e9,
                "step_frac_of_hbm_peak": alg / (ms_per_step * 1e-3) / 1e9 / peak,
                "peak": peak, "peak_kind": peak_kind,
                "exact_pass_worker_steps": fallbacks, "clocks": clocks}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
