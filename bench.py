#!/usr/bin/env python
"""Throughput of the GRAWA-family averaging update on B200, next to its HBM roofline and the
CPU oracle.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--variant lgrawa|mgrawa|grawa]
    python bench.py --impl reference ...        # times the float64 CPU oracle instead

A step is one whole update (gradient sums of squares -> scores -> weights -> centre -> pull of all
M workers) on one synthetic workload through the library's C ABI.  Prints one JSON line.
The update does not shard across GPUs by itself ("replicas only"): with --gpus N each rank runs
the same workload on its own GPU and the line reports the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

METRIC = "GRAWA update steps/sec (achieved HBM GB/s and fraction of roofline in `roofline`)"
DEFAULT_WORKLOAD = "vit_b16"
DEFAULT_VARIANT = "lgrawa"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak_gbs():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
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
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50", "-f", self.path], stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [r.strip().split(",") for r in open(self.path) if r.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        sm, reasons = [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0]))
                out["sm_max_mhz"] = float(r[1])
                for name, v in zip(names, r[3:7]):
                    if v.strip().lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------ the CUDA arm

def pinned_inputs(cfg):
    """Generates the workload straight into pinned host tensors (also used as the e2e source)."""
    import torch
    hp = [torch.empty(cfg.n, dtype=torch.float32).pin_memory() for _ in range(cfg.M)]
    hg = [torch.empty(cfg.n, dtype=torch.float32).pin_memory() for _ in range(cfg.M)]
    gen.make_inputs(cfg, [t.numpy() for t in hp], [t.numpy() for t in hg])
    return hp, hg


def workload_config(args):
    """The named workload, or (for small profiling captures) only its first --layers-limit layers
    with the same value recipe."""
    cfg = gen.CONFIGS[args.workload]
    if args.layers_limit and args.layers_limit < cfg.K:
        sizes = np.diff(cfg.offsets()[:args.layers_limit + 1])
        cfg = gen.custom_config(sizes, cfg.M, seed=cfg.seed, pull=cfg.pull, grad_recipe=cfg.grad_recipe,
                                log10_sigma=cfg.log10_sigma, loud_worker_factor=cfg.loud_worker_factor,
                                name=f"{cfg.name}[first {args.layers_limit} layers]")
    return cfg


def step_fn(grawa, variant):
    return {"lgrawa": grawa.grawa_lgrawa_step, "mgrawa": grawa.grawa_mgrawa_step, "grawa": grawa.grawa_grawa_step}[variant]


def time_device_steps(grawa, cfg, variant, x, g, center, steps, warmup, kernel_timing):
    """K back-to-back steps between two CUDA events on the launching stream.  Returns ms per step,
    launches in the timed region and (if asked) the per-phase kernel times."""
    import torch
    fn = step_fn(grawa, variant)
    off = cfg.offsets()
    for _ in range(warmup):
        fn(x, g, cfg.pull, off, center)
    torch.cuda.synchronize()
    grawa.grawa_set_option("kernel_timing", 1 if kernel_timing else 0)
    grawa.grawa_collect_kernel_times()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches = grawa.grawa_launch_count()
    e0.record()
    for _ in range(steps):
        fn(x, g, cfg.pull, off, center)
    e1.record()
    torch.cuda.synchronize()
    launches = grawa.grawa_launch_count() - launches
    grawa.grawa_set_option("kernel_timing", 0)
    phases = grawa.grawa_collect_kernel_times() if kernel_timing else None
    return e0.elapsed_time(e1) / steps, launches, phases


def time_e2e_steps(grawa, cfg, variant, hp, hg, hc, steps, warmup):
    """Steps through the host-buffer entry point: uploads, kernels and downloads are all inside
    the timed region.  Wall clock around a call that synchronises before it returns."""
    import torch
    off = cfg.offsets()
    for _ in range(warmup):
        grawa.grawa_step_host(variant, hp, hg, cfg.pull, off, hc)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        grawa.grawa_step_host(variant, hp, hg, cfg.pull, off, hc)
    torch.cuda.synchronize()
    return (time.perf_counter() - t0) * 1e3 / steps


def oracle_baseline(cfg, variant, params_np, grads_np, budget_s=15.0):
    """The CPU oracle as it stands (plain C, one thread) on a bounded sample of the workload: the
    first layers, all M workers, sized from a short probe to about `budget_s` seconds."""
    import oracle
    off = cfg.offsets()
    probe_n = min(cfg.n, 1 << 20)
    view = lambda arrs, hi: [a[:hi] for a in arrs]
    t0 = time.perf_counter()
    _oracle_sample(oracle, variant, view(params_np, probe_n), view(grads_np, probe_n), cfg.pull, np.array([0, probe_n]))
    per_elem = (time.perf_counter() - t0) / (probe_n * cfg.M)
    want = int(budget_s / (per_elem * cfg.M))
    k_hi = max(1, int(np.searchsorted(off, min(want, cfg.n), side="right")) - 1)
    n_s = int(off[k_hi])
    if n_s == 0:
        k_hi, n_s = cfg.K, cfg.n
    t0 = time.perf_counter()
    _oracle_sample(oracle, variant, view(params_np, n_s), view(grads_np, n_s), cfg.pull, off[:k_hi + 1])
    dt = time.perf_counter() - t0
    full = dt * cfg.n / n_s
    return {"value": 1.0 / full, "unit": "steps/s", "cores": 1, "kind": "oracle",
            "sample": f"first {k_hi} of {cfg.K} layers ({n_s} of {cfg.n} elements, all {cfg.M} workers), "
                      f"{dt:.2f} s measured, scaled by elements to a full step",
            "seconds_per_step_scaled": full}


def _oracle_sample(oracle, variant, p, g, pull, off):
    """One oracle step, streamed in chunks with reused output buffers (allocation is not the method)."""
    n, M = p[0].size, len(p)
    S = oracle.sumsq(g, off)
    beta, _ = oracle.weights(oracle.scores(S, variant))
    chunk = 1 << 18
    bufs = (np.zeros(chunk), [np.zeros(chunk) for _ in range(M)])
    for j0 in range(0, n, chunk):
        oracle.center_pull(p, beta, pull, off, j0, min(n, j0 + chunk), out=bufs)


def max_over_ranks(values, world, device):
    """Element-wise maximum of per-rank timings (the slowest rank defines the step time)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    import torch.distributed as dist
    if world > 1 or (dist.is_available() and dist.is_initialized()):
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_steps_per_s(world, ms_per_step_max):
    """Replicas only: every rank runs the same workload, so the job does `world` steps per step time."""
    return world * 1e3 / ms_per_step_max


# DRAM traffic of one centre+pull launch, from the ncu capture summarised in
# profiles/center_pull_kernel_vit_b16_28layers.md (M = 16; 1916.46 MB for 14 918 400 elements),
# scaled to a full launch by the number of elements.  Only valid for the kernel source it was taken
# from: the hash below is that of the centre+pull kernel's text in csrc/kernels.cuh (from its
# heading comment to the next kernel's) at capture time; anything else reports null.
TRAFFIC_CAPTURE = {"M": 16, "dram_bytes_per_element": (955.077376e6 + 961.380608e6) / 14918400,
                   "kernels_sha256": "e63e74aaf440bb7584d4f7c4bf30a29a04d4fe74544ad2ec2a8e2d6753ce5a49"}


# Same for the sum-of-squares kernel (profiles/sumsq_kernel_vit_b16_28layers.md: 954.82 MB read +
# 4.35 MB written for 14 918 400 elements at M = 16).
SUMSQ_TRAFFIC_CAPTURE = {"M": 16, "dram_bytes_per_element": (954.82112e6 + 4.346368e6) / 14918400,
                         "kernels_sha256": "3cad663f1177f4a514a5233796ed3df1eeae9242aa4c7b3b5f6ff7623fd66d56"}


def sumsq_traffic(cfg):
    import hashlib
    path = os.path.join(ROOT, "paper_2403_04206_b200", "csrc", "kernels.cuh")
    try:
        text = open(path).read()
        region = text[text.index("// Step 1 (Eq. 3 / Eq. 5): partial[m][s]"):text.index("// Steps 1b-3: one CTA per layer reduces")]
        digest = hashlib.sha256(region.encode()).hexdigest()
    except (OSError, ValueError):
        return None
    if digest != SUMSQ_TRAFFIC_CAPTURE["kernels_sha256"] or cfg.M != SUMSQ_TRAFFIC_CAPTURE["M"]:
        return None
    return SUMSQ_TRAFFIC_CAPTURE["dram_bytes_per_element"] * cfg.n


def center_pull_traffic(cfg):
    import hashlib
    path = os.path.join(ROOT, "paper_2403_04206_b200", "csrc", "kernels.cuh")
    try:
        text = open(path).read()
        region = text[text.index("// Steps 4-5, register variant"):text.index("// Steps 4-5 for any M up to")]
        digest = hashlib.sha256(region.encode()).hexdigest()
    except (OSError, ValueError):
        return None
    if digest != TRAFFIC_CAPTURE["kernels_sha256"] or cfg.M != TRAFFIC_CAPTURE["M"]:
        return None
    return TRAFFIC_CAPTURE["dram_bytes_per_element"] * cfg.n


def run_cuda(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    use_dist = "WORLD_SIZE" in os.environ and "MASTER_ADDR" in os.environ    # launched by torchrun, any world size
    if use_dist:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    import paper_2403_04206_b200 as grawa
    grawa.library()

    cfg = workload_config(args)
    variant = args.variant
    for kv in args.option:
        name, value = kv.split("=")
        grawa.grawa_set_option(name, int(value))
    hp, hg = pinned_inputs(cfg)
    x = [t.cuda(non_blocking=True) for t in hp]
    g = [t.cuda(non_blocking=True) for t in hg]
    center = torch.empty(cfg.n, device="cuda")
    torch.cuda.synchronize()

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: exactly K steps, device-resident inputs
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    ms, launches, _ = time_device_steps(grawa, cfg, variant, x, g, center, args.steps, args.warmup, False)
    clocks = sampler.stop()
    barrier()
    # ---- same region again with the library's per-phase events (for the kernel-level roofline)
    ms_k, _, phases = time_device_steps(grawa, cfg, variant, x, g, center, args.steps, 1, True)
    status = grawa.grawa_last_step_status()
    # ---- the other variant of the metric (MGRAWA when the headline is LGRAWA, and the reverse), same workload
    other = "mgrawa" if variant == "lgrawa" else "lgrawa"
    other_ms, _, _ = time_device_steps(grawa, cfg, other, x, g, center, max(20, args.steps // 4), 3, False)

    # ---- end to end through the host-buffer entry point
    hc = torch.empty(cfg.n, dtype=torch.float32).pin_memory()
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    e2e_ms = time_e2e_steps(grawa, cfg, variant, hp, hg, hc, e2e_steps, 1)

    ms_max, e2e_ms_max = max_over_ranks([ms, e2e_ms], world, "cuda")

    if rank == 0:
        peak, peak_src = measured_peak_gbs()
        alg_bytes = cfg.algorithmic_bytes()
        pull_bytes = (2 * cfg.M + 1) * 4 * cfg.n
        sumsq_bytes = cfg.M * 4 * cfg.n
        pull_ms = phases["center_pull_ms"] / phases["steps"]
        sumsq_ms = phases["sumsq_ms"] / phases["steps"]
        fin_ms = phases["finalize_ms"] / phases["steps"]
        achieved = pull_bytes / (pull_ms * 1e-3) / 1e9
        step_gbs = alg_bytes / (ms_max * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": whole_job_steps_per_s(world, ms_max), "unit": "steps/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_max, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{cfg.name} layer table, M={cfg.M} workers, n={cfg.n}, K={cfg.K} layers, "
                                   f"{variant.upper()} step, pull={cfg.pull}, seed={cfg.seed}",
                       "variant": variant, "M": cfg.M, "n": cfg.n, "n_layers": cfg.K,
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "l2": "inputs larger than L2 (no flush needed)" if alg_bytes > 4 * 126e6 else "L2-resident workload",
                       "algorithmic_bytes_per_step": alg_bytes},
            "step_hbm": {"achieved_gbs": step_gbs, "frac_of_measured_peak": step_gbs / peak,
                         "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS},
            "roofline": {"bound": "hbm", "kernel": "center_pull", "achieved": achieved, "peak": peak,
                         "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "traffic": center_pull_traffic(cfg),
                         "traffic_source": "ncu dram bytes of a 14.9M-element capture at the same M, scaled by elements",
                         "algorithmic_bytes_per_launch": pull_bytes, "kernel_ms": pull_ms,
                         "timed_with": "library CUDA events around each kernel in a second K-step region",
                         "other_kernels": {
                             "sumsq": {"algorithmic_bytes_per_launch": sumsq_bytes, "kernel_ms": sumsq_ms,
                                       "achieved": sumsq_bytes / (sumsq_ms * 1e-3) / 1e9,
                                       "frac": sumsq_bytes / (sumsq_ms * 1e-3) / 1e9 / peak,
                                       "traffic": sumsq_traffic(cfg)},
                             "finalize": {"kernel_ms": fin_ms}},
                         "ms_per_step_with_events": ms_k},
            "e2e": {"value": whole_job_steps_per_s(world, e2e_ms_max), "unit": "steps/s", "steps": e2e_steps,
                    "h2d_bytes_per_step": 2 * cfg.M * 4 * cfg.n, "d2h_bytes_per_step": (cfg.M + 1) * 4 * cfg.n,
                    "entry_point": "grawa_step_host (pinned host buffers)"},
            "other_variant": {"variant": other, "ms_per_step": other_ms, "steps_per_s": 1e3 / other_ms,
                              "achieved_gbs": alg_bytes / (other_ms * 1e-3) / 1e9,
                              "frac_of_measured_peak": alg_bytes / (other_ms * 1e-3) / 1e9 / peak,
                              "frac_of_nominal_8TBs": alg_bytes / (other_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
            "gpu_launches": launches, "clocks": clocks, "last_step_status": status,
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = oracle_baseline(cfg, variant, [t.numpy() for t in hp], [t.numpy() for t in hg])
        if world == 1 and args.also:
            line["also"] = also_runs(grawa, args, exclude=(args.workload, variant))
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()


def also_runs(grawa, args, exclude):
    """Short secondary measurements of the other large workloads and variants (not the headline)."""
    import torch
    out = []
    peak, _ = measured_peak_gbs()
    for name in ("resnet18_imagenet", "vgg16", "vit_b16"):
        cfg = gen.CONFIGS[name]
        hp, hg = pinned_inputs(cfg)
        x = [t.cuda() for t in hp]
        g = [t.cuda() for t in hg]
        center = torch.empty(cfg.n, device="cuda")
        del hp, hg
        for variant in ("mgrawa", "lgrawa"):
            if (name, variant) == exclude:
                continue
            steps = max(10, min(args.steps, 50))
            ms, _, _ = time_device_steps(grawa, cfg, variant, x, g, center, steps, 3, False)
            gbs = cfg.algorithmic_bytes() / (ms * 1e-3) / 1e9
            out.append({"workload": name, "variant": variant, "M": cfg.M, "n": cfg.n, "steps": steps,
                        "ms_per_step": ms, "steps_per_s": 1e3 / ms, "achieved_gbs": gbs,
                        "frac_of_measured_peak": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS})
        del x, g, center
        torch.cuda.empty_cache()
    return out


# ------------------------------------------------------------------ the reference arm (the CPU oracle)

def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cfg = workload_config(args)
    variant = args.variant
    off = cfg.offsets()
    total = args.steps + args.warmup
    budget = 150.0 / max(1, total)                      # whole run within a few minutes
    # bounded sample: a prefix of layers, all workers, sized from a probe
    probe_cfg = gen.custom_config([1 << 18], cfg.M, seed=cfg.seed)
    pp, pg = gen.make_inputs(probe_cfg)
    t0 = time.perf_counter()
    _oracle_sample(oracle, variant, pp, pg, cfg.pull, probe_cfg.offsets())
    per_elem = (time.perf_counter() - t0) / ((1 << 18) * cfg.M)
    want = max(1, int(budget / (per_elem * cfg.M)))
    k_hi = max(1, int(np.searchsorted(off, min(want, cfg.n), side="right")) - 1)
    while k_hi < cfg.K and off[k_hi] == 0:
        k_hi += 1
    n_s = int(off[k_hi])
    # generate only the sampled prefix: a custom workload with the same first layers and recipe
    sizes = np.diff(off[:k_hi + 1])
    sample_cfg = gen.custom_config(sizes, cfg.M, seed=cfg.seed, pull=cfg.pull, grad_recipe=cfg.grad_recipe,
                                   log10_sigma=cfg.log10_sigma, loud_worker_factor=cfg.loud_worker_factor)
    p_full, g_full = gen.make_inputs(sample_cfg)
    soff = off[:k_hi + 1]
    times = []
    for i in range(total):
        t0 = time.perf_counter()
        _oracle_sample(oracle, variant, p_full, g_full, cfg.pull, soff)
        if i >= args.warmup:
            times.append(time.perf_counter() - t0)
    sec = float(np.mean(times)) * cfg.n / n_s
    value = 1.0 / sec
    sample = (f"each step = the first {k_hi} of {cfg.K} layers ({n_s} of {cfg.n} elements, all {cfg.M} workers), "
              f"scaled by elements to a full step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{cfg.name} layer table, M={cfg.M} workers, n={cfg.n}, K={cfg.K} layers, "
                                   f"{variant.upper()} step, pull={cfg.pull}, seed={cfg.seed}",
                       "variant": variant, "M": cfg.M, "n": cfg.n, "n_layers": cfg.K},
            "cpu_baseline": {"value": value, "unit": "steps/s", "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(gen.CONFIGS))
    ap.add_argument("--variant", default=DEFAULT_VARIANT, choices=["lgrawa", "mgrawa", "grawa"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--also", action="store_true", help="add short runs of the other large workloads/variants")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers-limit", type=int, default=0, help="use only the first L layers (small profiling captures)")
    ap.add_argument("--option", action="append", default=[], help="library tuning knob, name=value (repeatable)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
