#!/usr/bin/env python
"""Throughput of the fused MLP-Adam cross-validation evaluation.

One "step" = one ``evaluate(params_list)`` call over one batch of suggested
configurations (paper, Algorithm 1): every configuration is trained on each of the
five folds and scored on the held-out fold.  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload NAME] [--fits F] [--hidden H] [--batch B]

The default workload is the headline cell of the digits-shaped throughput sweep: n=1797, d=64,
10 classes, 5 folds, 200 epochs, 16,000 fits per step (3,200 suggested configurations), hidden
width U{50..200} and batch size U{10..250} as the suggestions of the paper-shaped workloads
draw them.  ``--hidden`` / ``--batch`` pin a cell of the sweep's grid; ``--workload`` selects the
iris-, breast-, digits- and diabetes-shaped workloads and the two 10,000-row shapes.  With N
ranks one list of N x F fits is dealt to the ranks by estimated cost (no data-path collective)
and the scores are gathered at the end.
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
# dram__bytes_read.sum + dram__bytes_write.sum of one fit-kernel launch on the digits-shaped data
# (ncu capture of a 60-fit launch, summarised in profiles/mlp_cv_fit_kernel_small_cases_full.md;
# a 592-fit launch of the same capture set read 627,968):
# the dataset, the labels, the configurations and the fit list, read once.  It does not grow with
# the number of fits in the launch, because weights, moments and activations never leave the SM
# and every later read of X hits the L2; so the figure is not scaled to the bench's launch size.
# Other workloads have no capture of their own and report null.
FIT_KERNEL_DRAM_BYTES_PER_LAUNCH = {"digits_sweep": 615168, "digits2048": 615168}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--fits", type=int, default=0,
                    help="fits per GPU and step, 5 per configuration (0 = 16000 for digits_sweep, else the workload's own size)")
    ap.add_argument("--hidden", type=int, default=0, help="fixed hidden width (0 = U{50..200})")
    ap.add_argument("--batch", type=int, default=0, help="fixed batch size (0 = U{10..250})")
    ap.add_argument("--epochs", type=int, default=0, help="0 = the workload's own epoch count")
    ap.add_argument("--workload", default="digits_sweep",
                    choices=["digits_sweep", "iris8", "breast128", "digits2048", "diabetes4096", "housing10k", "collider10k"],
                    help="digits_sweep is the headline cell; the others are the paper-shaped workloads and the 10,000-row shapes")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (sweeps of many cells)")
    return ap.parse_args()


HEADLINE_FITS = 16000


def make_workload(args, world=1):
    """One list for the whole job: `world` times the per-GPU fit count."""
    fits = args.fits or (HEADLINE_FITS if args.workload == "digits_sweep" else 0)
    n_configs = max(1, fits // 5) * world if fits else None
    if n_configs is None and world > 1:
        n_configs = workloads.workload(args.workload).get("configs").size * world
    wl = workloads.workload(args.workload, seed=0, n_configs=n_configs,
                            hidden=args.hidden or None, batch_size=args.batch or None, epochs=args.epochs or None)
    return wl


def subset(wl, idx):
    out = dict(wl)
    out["configs"] = wl["configs"][idx]
    return out


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


def cpu_model():
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def fit_costs(wl):
    """Algorithmic FLOPs of every (configuration, fold) fit, configuration-major."""
    X, cfg, K = wl["X"], wl["configs"], wl["n_folds"]
    n, d = X.shape
    C = 1 if wl["task"] == 1 else int(wl["y"].max()) + 1
    H, E = cfg["hidden"].astype(np.float64), cfg["epochs"].astype(np.float64)
    cost = np.zeros((cfg.size, K))
    for f in range(K):
        n_tr = n - (n // K + (1 if f < n % K else 0))
        B = np.minimum(cfg["batch_size"], n_tr).astype(np.float64)
        cost[:, f] = E * n_tr * (4 * d * H + 6 * H * C) + E * np.ceil(n_tr / B) * (14 * (d * H + H * C) + 12 * (H + C))
    return cost.reshape(-1)


def stratified_fits(wl, count, offset=0.5):
    """`count` fits at evenly spaced quantiles of the cost order (whole fits, every epoch),
    returned costliest first so that the checker's dynamic schedule balances its threads."""
    cost = fit_costs(wl)
    order = np.argsort(cost, kind="stable")
    count = int(min(count, order.size))
    q = ((np.arange(count) + offset) / count * order.size).astype(np.int64).clip(0, order.size - 1)
    pick = order[q][::-1]
    K = wl["n_folds"]
    return (pick // K).astype(np.int32), (pick % K).astype(np.int32)


def oracle_whole_fits(wl, count, n_threads, offset=0.5):
    """Times the CPU checker, as it stands, on `count` whole fits of the workload (all epochs, no
    scaling), spread over the cost distribution.  Returns fits, seconds and the rate."""
    import oracle

    fc, ff = stratified_fits(wl, count, offset)
    t0 = time.perf_counter()
    oracle.cv_fits(wl["X"], wl["y"], wl["task"], wl["n_folds"], wl["configs"], wl["seed"], fc, ff, n_threads=n_threads)
    dt = time.perf_counter() - t0
    return dict(fits=int(fc.size), seconds=dt, value=fc.size / dt)


def oracle_baseline(wl, with_single_thread=True):
    """The cpu_baseline record: one whole fit per host thread at evenly spaced cost quantiles on
    all threads, plus (optionally) the median-cost fit alone on one thread."""
    import oracle

    cores = oracle.num_procs()
    n_fits = wl["configs"].size * wl["n_folds"]
    many = oracle_whole_fits(wl, cores, cores)
    rec = dict(value=many["value"], unit=UNIT, cores=cores, kind="oracle", cpu=cpu_model(),
               sample=f"{many['fits']} whole fits (all epochs) at evenly spaced quantiles of the cost order of the "
                      f"step's {n_fits}, costliest first, {many['seconds']:.1f} s wall on {cores} threads; no scaling")
    if with_single_thread:
        one = oracle_whole_fits(wl, 1, 1)
        rec["one_thread_value"] = one["value"]
        rec["sample"] += f"; the median-cost fit alone on one thread took {one['seconds']:.1f} s"
    return rec


REFERENCE_TIME_LIMIT_S = 300.0  # the reference arm stops taking new steps after this long


def run_reference(args, rank, world):
    """Reference arm: the CPU checker as it stands, on host cores; rank 0 only.  Every step is a
    sample of whole fits (one per host thread, each step at different quantiles of the cost
    order); a whole fit takes tens of seconds on one thread, so after REFERENCE_TIME_LIMIT_S the
    arm stops and reports the steps it completed."""
    if rank != 0:
        return
    import oracle

    wl = make_workload(args, 1)
    work = algorithmic_work(wl)
    cores = oracle.num_procs()
    short = dict(wl)
    short["configs"] = wl["configs"].copy()
    short["configs"]["epochs"] = 1
    for _ in range(args.warmup):  # untimed: one epoch of the same fits, warms caches and the thread pool
        oracle_whole_fits(short, cores, cores)
    per_step = []
    t_start = time.perf_counter()
    for i in range(args.steps):
        if per_step and time.perf_counter() - t_start > REFERENCE_TIME_LIMIT_S:
            break
        per_step.append(oracle_whole_fits(wl, cores, cores, offset=(i + 0.5) / max(1, args.steps)))
    fits = sum(p["fits"] for p in per_step)
    secs = sum(p["seconds"] for p in per_step)
    value = fits / secs
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(per_step), "steps_requested": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * secs / max(1, len(per_step)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(args, wl, work),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "cpu": cpu_model(),
                         "sample": f"each step {per_step[0]['fits']} whole fits (all epochs) at evenly spaced quantiles "
                                   f"of the cost order of the step's {work['n_fits']}, a different set per step; no scaling"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(args, wl, work):
    return {"workload": args.workload, "n": int(wl["X"].shape[0]), "d": int(wl["X"].shape[1]),
            "classes": 1 if wl["task"] == 1 else int(wl["y"].max()) + 1,
            "n_folds": 5, "epochs": int(wl["configs"]["epochs"][0]), "fits_per_step": int(work["n_fits"]),
            "hidden": args.hidden or "U{50..200}",
            "batch_size": args.batch or f"U{{10..{int(max(150, wl['configs']['batch_size'].max() > 150 and 250))}}}",
            "l2_between_steps": "flushed (256 MiB write)", "variant": "fp32-cuda-core, one CTA per fit, W1 moments in tensor memory, one launch per cost tier and hidden-width group"}


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

    # Weak scaling: the job's list holds `world` times the per-GPU fit count; it is dealt to the
    # ranks by estimated cost, every rank evaluates its share with the entries' list positions as
    # random-stream keys, and the scores are gathered at the end (the only collective).
    from paper_2012_04201_b200 import sharding

    wl_all = make_workload(args, world)
    work_all = algorithmic_work(wl_all)
    n_classes = 1 if wl_all["task"] == 1 else int(wl_all["y"].max()) + 1
    assign = sharding.balanced_assignment(
        sharding.config_costs(wl_all["configs"], wl_all["X"].shape[0], wl_all["X"].shape[1], n_classes, wl_all["n_folds"]), world)
    mine = sharding.shard_indices(assign, rank)
    wl = subset(wl_all, mine)
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
        h.eval(X, y, wl["task"], wl["n_folds"], cfg, wl["seed"], out=out, config_keys=mine if world > 1 else None)

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
    full_scores = sharding.gather_scores_by_assignment(out, assign, rank, world, dist)  # inside the timed region
    ev1.record(stream)
    barrier()
    assert full_scores.numel() == wl_all["configs"].size
    total_ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop() if rank == 0 else None
    if dist is not None:
        t = torch.tensor([total_ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    secs = total_ms / 1e3
    value = work_all["n_fits"] * args.steps / secs

    # end to end through the C ABI with host buffers (pinned), copies inside the timed region
    Xh = torch.from_numpy(wl["X"]).pin_memory()
    yh = torch.from_numpy(wl["y"]).pin_memory()
    e2e_steps = 0 if args.no_e2e else min(args.steps, 2)  # bounded: a step of the headline cell takes about ten seconds
    scores_h = out.cpu().numpy()
    if world == 1 and e2e_steps:
        h.eval_host(Xh.numpy(), yh.numpy(), wl["task"], wl["n_folds"], cfg, wl["seed"])
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        flush.fill_(1)
        if world == 1:
            scores_h = h.eval_host(Xh.numpy(), yh.numpy(), wl["task"], wl["n_folds"], cfg, wl["seed"])
        else:  # host buffers in, keyed evaluation, host scores out
            Xd, yd = Xh.cuda(non_blocking=True), yh.cuda(non_blocking=True)
            scores_h = h.eval(Xd, yd, wl["task"], wl["n_folds"], cfg, wl["seed"], config_keys=mine).cpu().numpy()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if dist is not None:
        t = torch.tensor([e2e_s], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = work_all["n_fits"] * e2e_steps / e2e_s if e2e_steps else None
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
        "frac": achieved / fp32_peak, "traffic": FIT_KERNEL_DRAM_BYTES_PER_LAUNCH.get(args.workload),
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
        "dtype": "f32", "data": "synthetic", "config": workload_config(args, wl_all, work_all),
        "sample_epochs_per_sec": work_all["sample_epochs"] * args.steps / secs,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "roofline": roofline,
    }
    line["e2e"]["steps"] = e2e_steps
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = oracle_baseline(wl)
    print(json.dumps(line), flush=True)
    h.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
