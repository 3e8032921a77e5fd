#!/usr/bin/env python
"""Throughput of the fused MLP-Adam cross-validation evaluation.

One "step" = one ``evaluate(params_list)`` call over one batch of suggested
configurations (paper, Algorithm 1): every configuration is trained on each of the
five folds and scored on the held-out fold.  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--fits F] [--hidden H] [--batch B]

The default workload is the digits-shaped throughput cell: n=1797, d=64, 10 classes,
5 folds, 200 epochs, hidden width U{50..200}, batch size U{10..250}.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2012_04201_b200 import workloads  # noqa: E402

METRIC = "mlp_adam_cv_fits_per_sec"
UNIT = "fits/s"
SM_COUNT_FP32_LANES = 128  # FP32 lanes per SM on sm_100
# dram__bytes_read.sum + dram__bytes_write.sum of one fit-kernel launch (ncu capture summarised in
# profiles/mlp_cv_fit_kernel_small_cases_full.md): the dataset, the labels, the configurations
# and the fit list, read once; the same for every launch size because weights, moments and
# activations never leave the SM.
FIT_KERNEL_DRAM_BYTES_PER_LAUNCH = 621e3


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--fits", type=int, default=4000, help="fits per launch (5 per configuration)")
    ap.add_argument("--hidden", type=int, default=0, help="fixed hidden width (0 = U{50..200})")
    ap.add_argument("--batch", type=int, default=0, help="fixed batch size (0 = U{10..250})")
    ap.add_argument("--epochs", type=int, default=200)
    ap.add_argument("--workload", default="digits_sweep", choices=["digits_sweep", "housing10k", "collider10k"],
                    help="digits_sweep is the headline cell; the 10,000-row shapes are extra cells")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def make_workload(args, rank):
    n_configs = max(1, args.fits // 5)
    wl = workloads.workload(args.workload, seed=rank, n_configs=n_configs,
                            hidden=args.hidden or None, batch_size=args.batch or None, epochs=args.epochs)
    return wl


def algorithmic_work(wl):
    """Algorithmic FLOPs and sample-epochs of one step (padding and wasted lanes not counted).

    Per fit: E * n_train * (4dH + 6HC)   forward 2dH+2HC, backward 2HC + 2HC + 2dH
           + steps * (14 (dH+HC) + 12 (H+C))   L2 term and Adam, fused multiply-add = 2
           + n_val * 2 (dH + HC)               held-out scoring
    """
    X, cfg = wl["X"], wl["configs"]
    n, d = X.shape
    K = wl["n_folds"]
    C = 1 if wl["task"] == 1 else int(wl["y"].max()) + 1
    H = cfg["hidden"].astype(np.float64)
    E = cfg["epochs"].astype(np.float64)
    flops = 0.0
    gemm_flops = 0.0
    sample_epochs = 0.0
    for f in range(K):
        n_val = n // K + (1 if f < n % K else 0)
        n_tr = n - n_val
        B = np.minimum(cfg["batch_size"], n_tr).astype(np.float64)
        steps = E * np.ceil(n_tr / B)
        g = E * n_tr * (4 * d * H + 6 * H * C)
        gemm_flops += g.sum()
        flops += (g + steps * (14 * (d * H + H * C) + 12 * (H + C)) + n_val * 2 * (d * H + H * C)).sum()
        sample_epochs += (E * n_tr).sum()
    return dict(flops=flops, gemm_flops=gemm_flops, sample_epochs=sample_epochs, n_fits=cfg.size * K)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "200",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2])); power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                    samples=len(sm), power_w_max=max(power))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh), "measured"
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, sm_max_mhz=1965.0), "fallback"


def oracle_sample_rate(wl, seconds_target=20.0, n_threads=0):
    """Times the CPU checker, as it stands, on a sample of this workload: one fit per host
    thread (spread evenly over the step's fit list), each run for a reduced number of epochs
    so that the sample takes about ``seconds_target`` seconds; the rate is scaled to whole fits
    by the epoch ratio (cost is proportional to epochs)."""
    import oracle

    cores = oracle.num_procs() if n_threads <= 0 else n_threads
    cfg, K = wl["configs"], wl["n_folds"]
    n_fits = cfg.size * K
    n, d = wl["X"].shape
    epochs_full = int(cfg["epochs"][0])
    # about one full fit costs E*n_tr*(4dH+6HC) flops at roughly 0.25 GFLOP/s per busy thread
    mean_flops = float((cfg["epochs"].astype(np.float64) * (n - n // K) * (4 * d + 60) * cfg["hidden"]).mean())
    per_fit_s = mean_flops / 0.25e9
    epochs_run = int(max(1, min(epochs_full, round(epochs_full * seconds_target / max(per_fit_s, 1e-3)))))
    sample = int(min(n_fits, cores))
    idx = np.linspace(0, n_fits - 1, sample).astype(np.int64)
    fc, ff = (idx // K).astype(np.int32), (idx % K).astype(np.int32)
    short = cfg.copy()
    short["epochs"] = epochs_run
    t0 = time.perf_counter()
    oracle.cv_fits(wl["X"], wl["y"], wl["task"], K, short, wl["seed"], fc, ff, n_threads=cores)
    dt = time.perf_counter() - t0
    fits_equiv = sample * epochs_run / float(epochs_full)
    return dict(value=fits_equiv / dt, unit=UNIT, cores=cores, kind="oracle",
                sample=f"{sample} fits (every {max(1, n_fits // sample)}th of the step's {n_fits}) for "
                       f"{epochs_run} of {epochs_full} epochs, {dt:.1f} s wall on {cores} threads, "
                       f"scaled to whole fits by the epoch ratio", seconds=dt, fits=fits_equiv)


def run_reference(args, rank, world):
    """Reference arm: the CPU checker as it stands, on host cores; rank 0 only."""
    if rank != 0:
        return
    wl = make_workload(args, 0)
    work = algorithmic_work(wl)
    per_step = []
    info = None
    for i in range(args.warmup + args.steps):
        # warm-up steps are short samples too; each step is a bounded sample of the workload
        info = oracle_sample_rate(wl, seconds_target=8.0 if i >= args.warmup else 1.0)
        if i >= args.warmup:
            per_step.append(info)
    fits = sum(p["fits"] for p in per_step)
    secs = sum(p["seconds"] for p in per_step)
    value = fits / secs
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(args, wl, work),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": info["cores"], "kind": "oracle",
                         "sample": f"each step a sample of {info['fits']} whole fits of the step's {work['n_fits']}"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(args, wl, work):
    return {"workload": args.workload, "n": int(wl["X"].shape[0]), "d": int(wl["X"].shape[1]),
            "classes": 1 if wl["task"] == 1 else int(wl["y"].max()) + 1,
            "n_folds": 5, "epochs": int(args.epochs), "fits_per_step": int(work["n_fits"]),
            "hidden": args.hidden or "U{50..200}", "batch_size": args.batch or "U{10..250}",
            "l2_between_steps": "flushed (256 MiB write)", "variant": "fp32-cuda-core, one CTA per fit, one launch per hidden-width group"}


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch

    from paper_2012_04201_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the evaluation has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    wl = make_workload(args, rank)  # weak scaling: every rank evaluates its own batch of configurations
    work = algorithmic_work(wl)
    cfg = wl["configs"]
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    out = torch.empty(cfg.size, dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    h = binding.MlpCv(device=local_rank, stream=stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def step():
        flush.fill_(1)  # evict L2 between steps
        h.eval(X, y, wl["task"], wl["n_folds"], cfg, wl["seed"], out=out)

    for _ in range(args.warmup):
        step()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fit_ms, launches = [], 0
    ev0.record(stream)
    for _ in range(args.steps):
        step()
        _, fms, nl = h.last_timing()
        fit_ms.append(fms)
        launches += nl
    ev1.record(stream)
    barrier()
    total_ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop() if rank == 0 else None
    if dist is not None:
        t = torch.tensor([total_ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    secs = total_ms / 1e3
    value = world * work["n_fits"] * args.steps / secs

    # end to end through the C ABI with host buffers (pinned), copies inside the timed region
    Xh = torch.from_numpy(wl["X"]).pin_memory()
    yh = torch.from_numpy(wl["y"]).pin_memory()
    h.eval_host(Xh.numpy(), yh.numpy(), wl["task"], wl["n_folds"], cfg, wl["seed"])
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        flush.fill_(1)
        scores_h = h.eval_host(Xh.numpy(), yh.numpy(), wl["task"], wl["n_folds"], cfg, wl["seed"])
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if dist is not None:
        t = torch.tensor([e2e_s], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = world * work["n_fits"] * args.steps / e2e_s
    assert np.array_equal(scores_h, out.cpu().numpy())
    h2d = int(wl["X"].nbytes + wl["y"].nbytes + cfg.nbytes + cfg.size * wl["n_folds"] * 8)
    d2h = int(cfg.size * 4 + 8)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks, peak_kind = load_peaks()
    props = torch.cuda.get_device_properties(local_rank)
    sm_max = float(clocks.get("sm_max_mhz") or peaks.get("sm_max_mhz", 1965.0))
    fp32_peak = props.multi_processor_count * SM_COUNT_FP32_LANES * 2 * sm_max * 1e6 / 1e12
    fit_s = statistics.mean(fit_ms) / 1e3
    achieved = work["flops"] / fit_s / 1e12
    roofline = {
        "bound": "alu", "kernel": "mlp_cv_fit_kernel", "achieved": achieved, "peak": fp32_peak, "unit": "TFLOP/s",
        "frac": achieved / fp32_peak, "traffic": FIT_KERNEL_DRAM_BYTES_PER_LAUNCH,
        "peak_source": f"{props.multi_processor_count} SMs x 128 FP32 lanes x 2 x {sm_max:.0f} MHz (max SM clock); "
                       f"HBM/bf16 peaks are {peak_kind} and do not bound this kernel",
        "gemm_only_achieved": work["gemm_flops"] / fit_s / 1e12,
        "kernel_ms": statistics.mean(fit_ms),
    }
    if clocks.get("sm_mhz"):
        roofline["frac_at_sampled_clock"] = achieved / (fp32_peak * clocks["sm_mhz"] / sm_max)
    try:  # FMA rate this device sustains from registers, measured now
        ffma = h.debug_ffma_peak()
        roofline["peak_measured_ffma"] = ffma
        roofline["frac_of_measured_ffma"] = achieved / ffma
    except Exception as exc:  # pragma: no cover
        roofline["peak_measured_ffma"] = None
        roofline["peak_measured_ffma_error"] = str(exc)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": workload_config(args, wl, work),
        "sample_epochs_per_sec": world * work["sample_epochs"] * args.steps / secs,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "roofline": roofline,
    }
    if world == 1 and not args.no_cpu_baseline:
        cb = oracle_sample_rate(wl)
        line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line), flush=True)
    h.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
