#!/usr/bin/env python
"""Benchmark of the DD-EF-SGD hot path (error-feedback Top-k compress + stale aggregate +
apply, Algorithm 1) on B200.  One "step" is one pass of the whole path over one batch of
synthetic gradients for all n simulated workers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is gradient GB/s (n*d*sizeof(g) bytes per step over
the device-timed step), whole job; with N > 1 every rank runs an independent replica (the
path does not shard), timed as the max over ranks.

The default workload is the largest single-GPU configuration (`decoder_1b`: d = 1.1 G entries,
n = 4, bf16 gradients, fp32 error terms and parameters, delta = 0.001, tau = 4).  With one GPU
the line also carries, under `other_workloads`, the other configurations with d >= 10 M timed
in the same process (each with its own clock samples), and for the d = 10^8 configuration the
delta x tau grid and the adaptive run in which the host policy (Algorithm 2 with DeCo,
Algorithm 3) re-selects (delta, tau) every 10 iterations from a synthetic network trace.
`--sweep` prints only that grid and run.
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
NOMINAL_HBM_GBS = 8000.0
DEFAULT_WORKLOAD = "decoder_1b"
OTHER_WORKLOADS = ["gpt2_small", "sweep_100m", "resnet18"]

# policy constants of the adaptive run (stand-ins: the paper gives no values)
SWEEP_DELTAS = [0.1, 0.01, 0.001, 0.0001]
SWEEP_TAUS = [0, 1, 2, 4, 8, 16]
ADAPT_E, ADAPT_STEPS, ADAPT_T_COMP, ADAPT_TAU_MAX, ADAPT_DELTA_MAX = 10, 200, 0.05, 16, 0.2


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--select-mode", default="auto", choices=["auto", "exact"])
    ap.add_argument("--pool", type=int, default=0, help="distinct gradient batches kept in HBM")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", action="store_true",
                    help="skip the other workloads and the delta x tau grid of the default line")
    ap.add_argument("--sweep", action="store_true",
                    help="only the delta x tau grid and the adaptive run at d = 10^8")
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


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


class ClockSampler:
    """SM clock and throttle reasons while the timed region runs.  Reads through NVML every few
    milliseconds (reading only; nothing is set); falls back to an nvidia-smi loop."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    # NVML clocks-event-reason bits
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
               "sw_power_cap": 0x4}

    def __init__(self, index, period_s=0.004):
        self.index = index
        self.period = period_s
        self.proc = None
        self.thread = None
        self.rows = []              # (wall time, sm MHz, max MHz, set of reasons, watts)
        self.stop_flag = False
        self.nvml = None
        self.handle = None
        self.how = "none"

    def _nvml_handle(self):
        import pynvml
        pynvml.nvmlInit()
        handle = None
        try:
            import torch
            uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
        except Exception:
            handle = None
        if handle is None:
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            idx = self.index
            if vis:
                ent = vis.split(",")[self.index].strip()
                if ent.isdigit():
                    idx = int(ent)
                else:
                    return pynvml, pynvml.nvmlDeviceGetHandleByUUID(ent.encode())
            handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
        return pynvml, handle

    def _poll_nvml(self):
        nv, h = self.nvml, self.handle
        try:
            smax = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
        except Exception:
            smax = None
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons", None)
        while not self.stop_flag:
            try:
                sm = float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                mask = int(get_reasons(h)) if get_reasons else 0
                try:
                    watts = nv.nvmlDeviceGetPowerUsage(h) / 1000.0
                except Exception:
                    watts = None
                rs = {name for name, bit in self.REASONS.items() if mask & bit}
                self.rows.append((time.time(), sm, smax, rs, watts))
            except Exception:
                pass
            time.sleep(self.period)

    def _poll_smi(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.proc.stdout:
            parts = [p.strip() for p in ln.strip().split(",")]
            if len(parts) < 8:
                continue
            try:
                sm, smax = float(parts[0]), float(parts[1])
            except ValueError:
                continue
            try:
                watts = float(parts[2])
            except ValueError:
                watts = None
            rs = {name for name, val in zip(names, parts[4:8]) if val.lower().startswith("active")}
            self.rows.append((time.time(), sm, smax, rs, watts))

    def start(self):
        try:
            self.nvml, self.handle = self._nvml_handle()
            self.how = "nvml"
            self.thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.how = "nvidia-smi"
            self.thread = threading.Thread(target=self._poll_smi, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def stop(self, t0, t1):
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock source"]}
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        else:
            self.stop_flag = True
            self.thread.join(timeout=2)
        inside = [r for r in self.rows if t0 <= r[0] <= t1 + (0.1 if self.proc else 0.0)]
        rows = inside if inside else self.rows[-3:]
        sm = [r[1] for r in rows]
        smax = [r[2] for r in rows if r[2] is not None]
        reasons = set()
        for r in rows:
            reasons |= r[3]
        watts = [r[4] for r in rows if r[4] is not None]
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm),
                "samples_in_timed_region": len(inside),
                "power_w_max": max(watts) if watts else None, "source": self.how}


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


def workload_for(args, name=None):
    from paper_2507_17346_b200 import workloads as W
    wl = W.make_workload(name or args.workload, args.scale)
    if name is None or name == args.workload:
        if args.delta is not None:
            wl.delta = args.delta
        if args.tau is not None:
            wl.tau = args.tau
    return wl


def grad_bytes(wl):
    return wl.n * wl.d * (4 if wl.grad_dtype == "f32" else 2)


def dtype_label(wl):
    return "f32" if wl.grad_dtype == "f32" else "bf16 gradients, f32 state"


# DRAM read + write bytes of one ef_accumulate_kernel launch from the ncu captures summarised in
# profiles/ef_accumulate_kernel_dram_traffic.md (taken on this kernel version).  resnet18 was
# captured at full size; the others at reduced size (--scale) and are scaled by the entry count:
# the kernel streams every entry once, so its traffic grows in proportion.
NCU_TRAFFIC_BYTES = {
    "resnet18": 1072.9e6,
    "gpt2_small": 1583.8e6 * (995518464 / 163946496),
    "decoder_1b": 2108.3e6 * (4400193536 / 216158400),
    "sweep_100m": 1150.4e6 * (400000000 / 100000000),
}


def algorithmic_bytes_accumulate(wl):
    """Streaming pass: read e (4), read g (4 or 2), write e (4) per entry and worker."""
    return wl.n * wl.d * (8 + (4 if wl.grad_dtype == "f32" else 2))


def algorithmic_bytes_step(wl, k):
    """Everything one iteration has to move: the streaming pass, the messages written and read
    once (8 n k each), the cached aggregate written and read once (at most 8 n k each) and the
    parameters read and written where touched (at most 8 min(d, n k))."""
    nk = wl.n * k
    return algorithmic_bytes_accumulate(wl) + 4 * 8 * nk + 8 * min(wl.d, nk)


# --------------------------------------------------------------------- reference arm

def oracle_throughput(wl, steps, warmup, budget_s=25.0):
    """The CPU oracle as it stands, on a bounded sample of the workload: `m` of the n workers
    at full d (or a prefix of it), chosen so that the whole run is some tens of seconds.
    Returns (GB/s, ms_per_step, sample)."""
    import numpy as np
    import torch
    from oracle import dd_ef_sgd as O
    torch.manual_seed(0)
    sz = 4 if wl.grad_dtype == "f32" else 2
    # about 0.06 us per entry and worker for accumulate + full sort + aggregate
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
    sample = ("%d of %d workers, d=%d of %d, %d steps, N(0, sigma) gradients, oracle as is "
              "(numpy + C fmaf, 1 thread); GB/s of the sample, not extrapolated") % (
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
            "dtype": dtype_label(wl), "data": "synthetic",
            "config": {"workload": wl.name, "d": wl.d, "n": wl.n, "delta": wl.delta,
                       "tau": wl.tau, "grad_dtype": wl.grad_dtype, "sample": sample},
            "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": 1, "host_cores": host_cores(),
                             "kind": "oracle", "sample": sample},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- our arm

def make_context(B, wl, args, local, n_local=None, base=0, sharded=False, **kw):
    mode = B.DECO_SELECT_AUTO if args.select_mode == "auto" else B.DECO_SELECT_EXACT_PASSES
    return B.deco_init(wl.d, wl.n if n_local is None else n_local, wl.delta, wl.tau, wl.lr,
                       grad_dtype=B.DECO_F32 if wl.grad_dtype == "f32" else B.DECO_BF16,
                       device=local, select_mode=mode,
                       compressor=B.DECO_COMPRESSOR_RANDK if args.compressor == "randk"
                       else B.DECO_COMPRESSOR_TOPK, seed=wl.seed,
                       n_total=wl.n if sharded else 0, worker_base=base, **kw)


def default_steps(gbytes):
    """Enough steps for a timed region of about a second."""
    return max(50, min(4000, int(8.0e12 / (6 * gbytes))))


def time_workload(B, W, wl, args, steps, warmup, local, world, rank, dist, sharded=False,
                  with_e2e=False):
    """One workload through deco_step: W warm-up iterations, then K timed ones between CUDA
    events on the caller's stream (barrier + synchronize on both sides), clocks sampled
    meanwhile.  Returns a dict of everything measured."""
    import torch
    gbytes = grad_bytes(wl)
    pool_n = args.pool if args.pool > 0 else max(2, min(8, int(6e9 // gbytes)))
    pool = [W.gradients(wl, p, "cuda") for p in range(pool_n)]
    n_local, base = wl.n, 0
    if sharded:
        n_local, base = wl.n // world, rank * (wl.n // world)
        pool = [p[base:base + n_local].clone() for p in pool]      # this rank's workers only
    ctx = make_context(B, wl, args, local, n_local, base, sharded)
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
    time.sleep(0.05)
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
    ms_per_step = max_over_ranks(ms_total, dist, "cuda") / steps

    # end to end through the host-buffer entry point: H2D gradients, step, D2H messages
    e2e = None
    if with_e2e:
        k = stats["k"]
        n_host = 2 if gbytes < 4e9 else 1
        host_g = []
        for p in pool[:n_host]:
            h = torch.empty(p.shape, dtype=p.dtype, pin_memory=True)
            h.copy_(p)
            host_g.append(h)
        del pool
        pool = []
        host_msg = torch.empty((wl.n, k, 2), dtype=torch.int32, pin_memory=True)
        e_steps = max(3, min(steps, int(3.0 / max(1e-4, gbytes / 20e9))))
        for t in range(3):
            B.deco_step_host(ctx, host_g[t % n_host], host_msg, None, stream)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for t in range(e_steps):
            B.deco_step_host(ctx, host_g[t % n_host], host_msg, None, stream)
        B.deco_join(ctx, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        e_ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
        e2e = {"value": whole_job_value(gbytes, world, e_ms / e_steps), "unit": UNIT,
               "h2d_bytes_per_step": gbytes, "d2h_bytes_per_step": wl.n * k * 8,
               "steps": e_steps, "ms_per_step": e_ms / e_steps}
        del host_g, host_msg
    B.deco_destroy(ctx)
    del pool
    torch.cuda.empty_cache()

    peak, peak_kind = measured_peaks()
    acc_ms = parts["accumulate"] / max(1, iters)
    acc_bytes = algorithmic_bytes_accumulate(wl) * n_local // wl.n      # this rank's launch
    achieved = acc_bytes / (acc_ms * 1e-3) / 1e9 if acc_ms > 0 else None
    as_configured = (args.scale == 1.0 and args.compressor == "topk" and
                     wl.delta == W.make_workload(wl.name).delta)
    roofline = {"bound": "hbm", "kernel": "ef_accumulate_kernel", "achieved": achieved,
                "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": (achieved / peak) if achieved else None,
                "traffic": NCU_TRAFFIC_BYTES.get(wl.name) if as_configured else None,
                "algorithmic_bytes_per_launch": acc_bytes,
                "avg_launch_ms": acc_ms, "launches_timed": iters}
    dominant = algorithmic_bytes_accumulate(wl)
    full = algorithmic_bytes_step(wl, stats["k"])
    gbps = dominant / (ms_per_step * 1e-3) / 1e9
    return {"ms_per_step": ms_per_step, "gbytes": gbytes, "pool_n": pool_n, "stats": stats,
            "steps": steps, "warmup": warmup,
            "step_algorithmic_GBps": gbps,
            "step_frac_of_hbm_peak": gbps / peak,
            "step_frac_of_nominal_8TBps": gbps / NOMINAL_HBM_GBS,
            "step_all_terms_GBps": full / (ms_per_step * 1e-3) / 1e9,
            "step_all_terms_frac_of_hbm_peak": full / (ms_per_step * 1e-3) / 1e9 / peak,
            "phases_ms": {k_: v / max(1, iters) for k_, v in parts.items()},
            "roofline": roofline, "clocks": clocks, "launches": launches, "e2e": e2e,
            "peak": peak, "peak_kind": peak_kind}


def summary_of(res, wl):
    """The short form a workload takes under `other_workloads`."""
    return {"d": wl.d, "n": wl.n, "delta": wl.delta, "tau": wl.tau, "k": res["stats"]["k"],
            "dtype": dtype_label(wl), "steps": res["steps"], "warmup": res["warmup"],
            "ms_per_step": res["ms_per_step"],
            "gradient_GBps": res["gbytes"] / (res["ms_per_step"] * 1e-3) / 1e9,
            "step_algorithmic_GBps": res["step_algorithmic_GBps"],
            "step_frac_of_hbm_peak": res["step_frac_of_hbm_peak"],
            "step_frac_of_nominal_8TBps": res["step_frac_of_nominal_8TBps"],
            "step_all_terms_frac_of_hbm_peak": res["step_all_terms_frac_of_hbm_peak"],
            "accumulate_frac_of_hbm_peak": res["roofline"]["frac"],
            "phases_ms": res["phases_ms"],
            "exact_pass_worker_steps": res["stats"]["exact_pass_workers"],
            "gpu_launches": res["launches"], "clocks": res["clocks"]}


def run_sweep(B, W, args, local):
    """The d = 10^8 configuration as stated: delta x tau grid (fresh context, 3 warm-up + 20
    timed iterations per combination), then 200 iterations in which DeCo (Algorithm 3) re-selects
    (delta, tau) every E = 10 iterations from the synthetic trace (Algorithm 2)."""
    import numpy as np
    import torch
    wl = W.make_workload("sweep_100m", args.scale)
    peak, _ = measured_peaks()
    stream = torch.cuda.current_stream()
    pool = [W.gradients(wl, p, "cuda") for p in range(2)]
    alg = algorithmic_bytes_accumulate(wl)
    grid = []
    for delta in SWEEP_DELTAS:
        for tau in SWEEP_TAUS:
            wl.delta, wl.tau = delta, tau
            ctx = make_context(B, wl, args, local)
            for t in range(3):
                B.deco_step(ctx, pool[t % 2], stream)
            torch.cuda.synchronize()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(stream)
            for t in range(20):
                B.deco_step(ctx, pool[(t + 1) % 2], stream)
            B.deco_join(ctx, stream)
            ev1.record(stream)
            torch.cuda.synchronize()
            ms = ev0.elapsed_time(ev1) / 20
            st = B.deco_get_stats(ctx, stream)
            B.deco_destroy(ctx)
            full = algorithmic_bytes_step(wl, st["k"])
            grid.append({"delta": delta, "tau": tau, "k": st["k"], "ms_per_step": ms,
                         "step_frac_of_hbm_peak": alg / (ms * 1e-3) / 1e9 / peak,
                         "step_all_terms_frac_of_hbm_peak": full / (ms * 1e-3) / 1e9 / peak,
                         "exact_pass_worker_steps": st["exact_pass_workers"]})
    # adaptive run
    wl.delta, wl.tau = 0.01, 2
    V_g = 32.0 * wl.d
    lat, bw = W.network_trace(wl.seed, ADAPT_STEPS)
    ctx = make_context(B, wl, args, local, tau_max=ADAPT_TAU_MAX, delta_max=ADAPT_DELTA_MAX)
    for t in range(3):
        B.deco_step(ctx, pool[t % 2], stream)
    B.deco_join(ctx, stream)
    torch.cuda.synchronize()
    B.deco_reset(ctx, stream)
    decisions = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for t in range(ADAPT_STEPS):
        if t and t % ADAPT_E == 0:
            a_bar, b = float(np.mean(bw[t - ADAPT_E:t])), float(lat[t - 1])
            tau, delta = B.deco_policy_select(V_g, a_bar, b, ADAPT_T_COMP, ADAPT_TAU_MAX, False)
            delta = min(ADAPT_DELTA_MAX, max(delta, 1.0 / wl.d))
            B.deco_set_policy(ctx, delta, tau)
            decisions.append((t, delta, tau))
        B.deco_step(ctx, pool[t % 2], stream)
    B.deco_join(ctx, stream)
    ev1.record(stream)
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / ADAPT_STEPS
    st = B.deco_get_stats(ctx, stream)
    B.deco_destroy(ctx)
    del pool
    torch.cuda.empty_cache()
    adaptive = {"steps": ADAPT_STEPS, "E": ADAPT_E, "T_comp_s": ADAPT_T_COMP,
                "tau_max": ADAPT_TAU_MAX, "delta_max": ADAPT_DELTA_MAX, "ms_per_step": ms,
                "step_frac_of_hbm_peak": alg / (ms * 1e-3) / 1e9 / peak,
                "decisions": len(decisions),
                "delta_range": [min(x[1] for x in decisions), max(x[1] for x in decisions)],
                "tau_range": [min(x[2] for x in decisions), max(x[2] for x in decisions)],
                "exact_pass_worker_steps": st["exact_pass_workers"],
                "device_status": st["device_status"],
                "note": "host-side policy calls sit inside the timed region"}
    return {"d": wl.d, "n": wl.n, "grid": grid, "adaptive": adaptive}


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

    if args.sweep:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "unit": UNIT, "sweep": run_sweep(B, W, args, local)}),
                  flush=True)
        if dist is not None:
            dist.destroy_process_group()
        return

    wl = workload_for(args)
    gbytes = grad_bytes(wl)
    steps = args.steps if args.steps is not None else default_steps(gbytes)
    warmup = max(3, args.warmup if args.warmup is not None else 10)
    sharded = args.shard_workers and world > 1
    if sharded and wl.n % world:
        raise SystemExit("--shard-workers needs the worker count to be a multiple of --gpus")
    if args.per_layer:
        pool_n = args.pool if args.pool > 0 else max(2, min(8, int(6e9 // gbytes)))
        pool = [W.gradients(wl, p, "cuda") for p in range(pool_n)]
        return run_per_layer(args, wl, pool, pool_n, steps, warmup, local, world, rank, dist)

    res = time_workload(B, W, wl, args, steps, warmup, local, world, rank, dist, sharded,
                        with_e2e=not args.no_e2e and not sharded)
    # replicas: every rank steps the whole workload; sharded: the ranks share one workload
    value = whole_job_value(gbytes, 1 if sharded else world, res["ms_per_step"])

    # the oracle's sample on the host cores comes next: ten seconds in which the card rests
    # between the 1.1 G workload and the smaller ones
    cpu_base = None
    if not args.no_cpu_baseline and world == 1:
        gbs, ms, sample = oracle_throughput(wl, 2, 1)
        cpu_base = {"value": gbs, "unit": UNIT, "cores": 1, "host_cores": host_cores(),
                    "kind": "oracle", "sample": sample, "ms_per_step_sample": ms}

    others = None
    if world == 1 and not args.no_others and args.workload == DEFAULT_WORKLOAD and args.scale == 1.0:
        others = {}
        for name in OTHER_WORKLOADS:
            owl = workload_for(args, name)
            osteps = min(default_steps(grad_bytes(owl)), 150)
            r = time_workload(B, W, owl, args, osteps, 10, local, world, rank, dist)
            others[name] = summary_of(r, owl)
        others["sweep_100m"]["delta_tau_grid_and_adaptive_run"] = run_sweep(B, W, args, local)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    stats = res["stats"]
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True,
            "scaling": "strong" if sharded else "weak", "vs_baseline": None,
            "dtype": dtype_label(wl), "data": "synthetic",
            "config": {"workload": wl.name, "d": wl.d, "n": wl.n, "delta": wl.delta,
                       "tau": wl.tau, "lr": wl.lr, "grad_dtype": wl.grad_dtype,
                       "k": stats["k"], "select_mode": args.select_mode,
                       "compressor": args.compressor,
                       "l2": "inputs larger than L2 (e and g of one step exceed 126 MB)"
                       if 2 * gbytes > 126e6 else "working set fits in L2",
                       "gradient_pool": res["pool_n"], "replicas": 1 if sharded else world,
                       "parallelism": ("workers sharded over %d ranks" % world) if sharded
                       else "replicas only"},
            "step_algorithmic_GBps": res["step_algorithmic_GBps"],
            "step_frac_of_hbm_peak": res["step_frac_of_hbm_peak"],
            "step_frac_of_nominal_8TBps": res["step_frac_of_nominal_8TBps"],
            "step_all_terms_frac_of_hbm_peak": res["step_all_terms_frac_of_hbm_peak"],
            "phases_ms": res["phases_ms"],
            "exact_pass_worker_steps": stats["exact_pass_workers"],
            "roofline": res["roofline"], "clocks": res["clocks"], "gpu_launches": res["launches"]}
    if res["e2e"] is not None:
        line["e2e"] = res["e2e"]
    if cpu_base is not None:
        line["cpu_baseline"] = cpu_base
        line["config"]["cpu_baseline_sample"] = cpu_base["sample"]
    if others is not None:
        line["other_workloads"] = others
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
    time.sleep(0.05)
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
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": dtype_label(wl), "data": "synthetic",
                "config": {"workload": wl.name, "variant": "per-layer Top-k", "layers": info["n_layers"],
                           "d": wl.d, "n": wl.n, "delta": wl.delta, "tau": wl.tau, "lr": wl.lr,
                           "grad_dtype": wl.grad_dtype, "k_total": info["k_total"],
                           "gradient_pool": pool_n, "parallelism": "replicas only"},
                "step_algorithmic_GBps": alg / (ms_per_step * 1e-3) / 1e9,
                "step_frac_of_hbm_peak": alg / (ms_per_step * 1e-3) / 1e9 / peak,
                "step_frac_of_nominal_8TBps": alg / (ms_per_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
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
