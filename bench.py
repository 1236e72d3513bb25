#!/usr/bin/env python
"""Benchmark of the nested-gradient-code hot path: decoded gradients per second.

One "step" = one full iteration for a fresh seeded straggler pattern: stopping rule, fused
partial gradients + encode for the chosen component code, decoding-vector solve, decode.

    python bench.py --gpus 1 --steps 200 --warmup 20            # CUDA library
    python bench.py --impl reference --steps 2 --warmup 1       # the CPU oracle, on the host cores
    torchrun --nproc-per-node N ... bench.py --gpus N ...       # N independent replicas (weak scaling)

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import ngc_inputs  # noqa: E402

METRIC = "decoded NGC gradients/sec"
UNIT = "gradients/s"
DEFAULT_WORKLOAD = "logistic20"
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------- small helpers
def env_rank():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def rank_max(value: float, world: int, device=None) -> float:
    """Largest value over all ranks (the job is as slow as its slowest rank)."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_sum(value: float, world: int, device=None) -> float:
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def replica_workload(w: ngc_inputs.Workload, rank: int) -> ngc_inputs.Workload:
    """Each rank works on its own seeded replica of the workload (independent problems, no exchange)."""
    from dataclasses import replace
    return replace(w, index=w.index + 1000 * rank)


def decodable_patterns(w, plan_levels, count, select_fn):
    """First `count` straggler patterns of the workload's seed list that some component code can decode."""
    out, skipped, it = [], 0, 0
    while len(out) < count:
        t = ngc_inputs.pattern_times(w, it)
        it += 1
        if select_fn(t):
            out.append(t)
        else:
            skipped += 1
    return out, skipped


def algorithmic_bytes(w: ngc_inputs.Workload, coded_bytes_per_value: int) -> int:
    """Bytes one fused gradient+encode launch has to move: the data matrix and labels once, theta, the coded matrix."""
    xb = 2 if w.x_dtype == "bf16" else 4
    return w.n * w.rows * w.d * xb + w.n * w.rows * 4 + w.n_params * 4 + w.n * w.n_params * coded_bytes_per_value


def algorithmic_flops(w: ngc_inputs.Workload) -> int:
    """Flops of the dense contractions one gradient launch performs (2 per multiply-add)."""
    if w.kind == "softmax":
        return 4 * w.n * w.rows * w.d * w.n_classes
    return w.n * w.rows * (4 * w.d * w.hidden + 6 * w.hidden * w.n_classes)


# dram__bytes_read + dram__bytes_write per full-size launch of the timed kernel (the dense workloads: summed over the
# gradient kernels the events bracket), from the ncu captures summarised under profiles/ (None = not captured for
# the kernels as they stand).
TRAFFIC_BYTES = {"logistic20": 2_689_000_000, "lsq100": 6_585_000_000,
                 "softmax50": 1_075_000_000, "mlp30": 643_000_000}
FALLBACK_BF16_TFLOPS_SUSTAINED = 1400.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        clocks, reasons, mx = [], set(), None
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    clocks.append(float(f[1])); mx = float(f[2])
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if clocks:
            out["sm_mhz"] = statistics.median(clocks)
            out["sm_max_mhz"] = mx
            out["samples"] = len(clocks)
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def oracle_step_seconds(w, X, y, theta, times, sample_rows: int):
    """Times the oracle as it stands on a bounded sample of one step.

    The partial gradients are computed on the first `sample_rows` rows of the workload (whole partitions
    first, then a row prefix of the next one) and that time is scaled to all n * rows rows; selection,
    encode, decoding vector and decode are timed in full (on the sampled gradients tiled to n rows).
    """
    from oracle import ngc_oracle as orc
    levels = list(w.levels)
    pl = orc.plan(w.n, levels, w.seed)
    t0 = time.perf_counter()
    sel = orc.select(times, levels, 0.0, 0.0)
    t_sel = time.perf_counter() - t0
    th = theta.double().numpy()
    t0 = time.perf_counter()
    Gs, left, j = [], sample_rows, 0
    while left > 0:
        r = min(left, w.rows)
        yj = y[j, :r].double().numpy() if y.dtype.is_floating_point else y[j, :r].numpy()
        Gs.append(orc.partial_gradient(w.kind, X[j, :r].double().numpy(), yj, th, w.hidden, w.n_classes))
        left -= r
        j += 1
    t_grad = (time.perf_counter() - t0) * (w.n * w.rows / sample_rows)
    G = np.stack([Gs[j % len(Gs)] for j in range(w.n)])
    t0 = time.perf_counter()
    B = pl["B"][sel["level"]]
    coded = orc.encode(B, G)
    a = orc.decode_vector(B, sel["S"])
    orc.decode(a, coded)
    t_rest = time.perf_counter() - t0
    return t_sel + t_grad + t_rest


def sample_description(w, sample_rows, secs=None):
    s = (f"partial gradients on the first {sample_rows} of {w.n * w.rows} rows, time scaled "
         f"x{w.n * w.rows / sample_rows:.4g}; selection, encode, decoding vector and decode in full")
    return s + (f" ({secs:.2f} s/step)" if secs is not None else "")


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores (rank 0 only)."""
    rank, _, world = env_rank()
    if rank != 0:
        return
    from dataclasses import replace

    from oracle import ngc_oracle as orc
    w = ngc_inputs.WORKLOADS[args.workload]
    budget = args.cpu_budget_s / max(1, args.steps + args.warmup)      # seconds of oracle work per step
    # one partition first: how long does a row take?
    X, y, theta = ngc_inputs.make_data(replace(w, n=1), "cpu")
    probe_rows = min(w.rows, 256)
    pats = [ngc_inputs.pattern_times(w, it) for it in range(args.warmup + args.steps + 64)]
    pats = [t for t in pats if orc.select(t, list(w.levels), 0.0, 0.0) is not None]
    t0 = time.perf_counter()
    oracle_step_seconds(w, X, y, theta, pats[0], probe_rows)
    per_row = max((time.perf_counter() - t0) / probe_rows, 1e-9)
    sample_rows = int(min(w.n * w.rows, max(16, budget / per_row)))
    parts = -(-sample_rows // w.rows)
    if parts > 1:
        X, y, theta = ngc_inputs.make_data(replace(w, n=parts), "cpu")
    for i in range(args.warmup):
        oracle_step_seconds(w, X, y, theta, pats[i], sample_rows)
    secs = [oracle_step_seconds(w, X, y, theta, pats[args.warmup + i], sample_rows) for i in range(args.steps)]
    total = sum(secs)
    value = args.steps / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "n_workers": w.n, "levels": list(w.levels), "kind": w.kind,
                   "rows_per_partition": w.rows, "d": w.d, "x_dtype": w.x_dtype},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": sample_description(w, sample_rows)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- CUDA arm
def run_cuda(args):
    import torch
    import paper_2212_08580_b200 as ngc

    rank, local_rank, world = env_rank()
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch N>1 with torch.distributed.run")
    if not torch.cuda.is_available():
        raise SystemExit("no CUDA device: the CUDA arm has no CPU fallback (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    w = replica_workload(ngc_inputs.WORKLOADS[args.workload], rank)
    if args.rows:                      # reduced case for profiler captures; never the reported workload
        w = ngc_inputs.shrink(w, rows=args.rows)
    X, y, theta = ngc_inputs.make_data(w, dev)
    m = ngc.Model.make(w.kind, w.x_dtype, w.rows, w.d, w.n_classes, w.hidden)
    plan = ngc.Plan(w.n, w.levels, seed=w.seed)
    cdt = plan.coded_dtype(m)
    l = w.n_params
    coded = torch.empty((w.n, l), dtype=torch.float64 if cdt == ngc.NGC_F64 else torch.float32, device=dev)
    grad = torch.empty(l, dtype=torch.float32, device=dev)

    def decodable(t):
        try:
            plan.select(t)
            return True
        except ngc.NgcError:
            return False

    pats, skipped = decodable_patterns(w, w.levels, args.warmup + args.steps, decodable)
    stream = torch.cuda.current_stream().cuda_stream

    for i in range(args.warmup):
        plan.step(m, theta, X, y, pats[i], coded, grad, stream)
    torch.cuda.synchronize()
    plan.profile_read()
    plan.profile_enable(True)
    try:
        smi_index = int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank])
    except (KeyError, ValueError, IndexError):
        smi_index = local_rank
    sampler = ClockSampler(smi_index)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = plan.launch_count()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    levels_used = []
    e0.record()
    for i in range(args.steps):
        info = plan.step(m, theta, X, y, pats[args.warmup + i], coded, grad, stream)
        levels_used.append(info.layer)
    e1.record()
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    ms_total = rank_max(e0.elapsed_time(e1), world, dev)
    launches = plan.launch_count() - launches0
    kern_ms, kern_n = plan.profile_read()
    plan.profile_enable(False)
    clocks = sampler.stop() if rank == 0 else {}
    residual = plan.device_status()

    # ---- end to end through the host-buffer entry point: pinned host inputs copied every step
    e2e_steps = min(args.steps, args.e2e_steps)
    h2d = X.numel() * X.element_size() + y.numel() * y.element_size() + theta.numel() * 4
    d2h = l * 4
    e2e = None
    if e2e_steps > 0:
        Xh, yh, thh = X.cpu().pin_memory(), y.cpu().pin_memory(), theta.cpu().pin_memory()
        gh = torch.empty(l, dtype=torch.float32).pin_memory()
        for i in range(2):
            plan.step_host(m, thh, Xh, yh, pats[i], gh)
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            plan.step_host(m, thh, Xh, yh, pats[args.warmup + i], gh)
        torch.cuda.synchronize()
        e2e_s = rank_max(time.perf_counter() - t0, world, dev)
        e2e = {"value": world * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps}

    # ---- roofline of the dominant kernel(s) (the fused gradient kernels that ngc_profile brackets)
    peaks, which = measured_peaks()
    cbytes = 8 if cdt == ngc.NGC_F64 else 4
    kern_avg_ms = kern_ms / max(kern_n, 1)
    traffic = TRAFFIC_BYTES.get(w.name) if not args.rows else None
    if w.kind in ("lsq", "logistic"):
        alg = algorithmic_bytes(w, cbytes)
        achieved = alg / (kern_avg_ms * 1e-3) / 1e9 if kern_n else None
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": (achieved / peaks["hbm_gbs"]) if achieved else None, "traffic": traffic,
                    "kernel": "gemv_pair_kernel", "kernel_ms": kern_avg_ms, "algorithmic_bytes": alg,
                    "peak_source": f"of {which}"}
    else:
        flops = algorithmic_flops(w)
        peak = peaks.get("bf16_tflops_sustained", FALLBACK_BF16_TFLOPS_SUSTAINED)
        achieved = flops / (kern_avg_ms * 1e-3) / 1e12 if kern_n else None
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                    "frac": (achieved / peak) if achieved else None, "traffic": traffic,
                    "kernel": "forward + backward contraction kernels", "kernel_ms": kern_avg_ms,
                    "algorithmic_flops": flops, "peak_source": f"of {which} (sustained bf16)"}

    line = {
        "metric": METRIC, "value": world * args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if w.kind in ("lsq", "logistic") else "bf16", "data": "synthetic",
        "config": {"workload": w.name, "n_workers": w.n, "levels": list(w.levels), "kind": w.kind,
                   "rows_per_partition": w.rows, "d": w.d, "x_dtype": w.x_dtype,
                   "coded_dtype": "f64" if cdt == ngc.NGC_F64 else "f32",
                   "l2": "inputs larger than L2 (data matrix %.2f GB per step)" % (h2d / 1e9),
                   "patterns": "fresh seeded pattern per step", "undecodable_skipped": skipped,
                   "levels_chosen": {str(k): levels_used.count(k) for k in sorted(set(levels_used))},
                   "replicas": "independent per GPU, no data-path collective"},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(rank_sum(launches, world, dev)),
        "roofline": roofline,
        "decode_residual_max": residual,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline and e2e is not None:
        t0 = time.perf_counter()
        oracle_step_seconds(w, Xh, yh, thh, pats[0], min(w.rows, 256))
        per_row = max((time.perf_counter() - t0) / min(w.rows, 256), 1e-9)
        sample_rows = int(min(w.n * w.rows, max(16, args.cpu_budget_s / 6 / per_row)))
        secs = oracle_step_seconds(w, Xh, yh, thh, pats[0], sample_rows)
        line["cpu_baseline"] = {"value": 1.0 / secs, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                                "sample": sample_description(w, sample_rows, secs)}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(ngc_inputs.WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-budget-s", type=float, default=120.0,
                    help="seconds of CPU-oracle work the reference arm may spend in total")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--rows", type=int, default=0,
                    help="rows per partition override: a reduced case for profiler captures only")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 2 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 200 if args.steps is None else args.steps
        args.warmup = 20 if args.warmup is None else args.warmup
        run_cuda(args)


if __name__ == "__main__":
    main()
