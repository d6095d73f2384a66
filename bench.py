#!/usr/bin/env python
"""Throughput of the GRAWA-family averaging update on B200, next to its HBM roofline and the
CPU oracle.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--variant lgrawa|mgrawa|grawa]
                    [--op step|prox|from_norms] [--dtype f32|bf16|f16] [--sharded]
    python bench.py --impl reference ...        # times the float64 CPU oracle instead

A step is one whole update (gradient sums of squares -> scores -> weights -> centre -> pull of all
M workers) on one synthetic workload through the library's C ABI.  Prints one JSON line.  Besides
the headline (ViT-B/16 table, LGRAWA) the default line carries short runs of every workload of at
least 10 M parameters in both variants (`targets`), of the proximity step, the step from given norms
and the step on bfloat16 storage (`ops`), and of the two small workloads eagerly and in a CUDA graph
(`small`).  The update does not shard across GPUs by itself ("replicas only"): with --gpus N each
rank runs the same workload on its own GPU and the line reports the aggregate; --sharded instead cuts
ONE problem by element range over the ranks (one all-gather of a [K, M] table per step).
"""
from __future__ import annotations

import argparse
import hashlib
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
TARGET_WORKLOADS = ("resnet18_imagenet", "vgg16", "vit_b16")       # the workloads of at least 10 M parameters
SMALL_WORKLOADS = ("toy10", "resnet20_cifar")
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
ELEM_BYTES = {"f32": 4, "bf16": 2, "f16": 2}


def measured_peak_gbs():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed regions run."""
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
        sm, power, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                watts = float(r[2])
                out["sm_max_mhz"] = float(r[1])
                if watts < 300.0:                    # idle sample (input generation on the host): not "under load"
                    continue
                sm.append(float(r[0]))
                power.append(watts)
                for name, v in zip(names, r[3:7]):
                    if v.strip().lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        if not sm:                                   # a run too short to catch a sample under load: use them all
            for r in rows:
                try:
                    sm.append(float(r[0]))
                    power.append(float(r[2]))
                except Exception:
                    continue
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["samples"] = len(sm)
            out["power_w_max"] = max(power)
        out["samples_total"] = len(rows)
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------ workloads on the device

def with_workers(cfg, M):
    """The same layer table and value recipe with another number of workers."""
    return gen.custom_config(np.diff(cfg.offsets()), M, seed=cfg.seed, pull=cfg.pull, grad_recipe=cfg.grad_recipe,
                             log10_sigma=cfg.log10_sigma, loud_worker_factor=cfg.loud_worker_factor, name=f"{cfg.name}[M={M}]")


def workload_config(args):
    """The named workload, or (for small profiling captures) only its first --layers-limit layers
    with the same value recipe."""
    cfg = gen.CONFIGS[args.workload]
    if args.workers and args.workers != cfg.M:
        cfg = with_workers(cfg, args.workers)
    if args.layers_limit and args.layers_limit < cfg.K:
        sizes = np.diff(cfg.offsets()[:args.layers_limit + 1])
        cfg = gen.custom_config(sizes, cfg.M, seed=cfg.seed, pull=cfg.pull, grad_recipe=cfg.grad_recipe,
                                log10_sigma=cfg.log10_sigma, loud_worker_factor=cfg.loud_worker_factor,
                                name=f"{cfg.name}[first {args.layers_limit} layers]")
    return cfg


def describe(cfg, variant, op="step", dtype="f32", world=1, sharded=False):
    """The `config` object of a line; both arms build it here so that they agree key by key."""
    what = {"step": f"{variant.upper()} step", "prox": "proximity step", "from_norms": f"{variant.upper()} step from given layer norms"}[op]
    par = "single GPU" if world == 1 else ("element-range sharded" if sharded else "replicas only")
    return {"workload": f"{cfg.name} layer table, M={cfg.M} workers, n={cfg.n}, K={cfg.K} layers, "
                        f"{what}, pull={cfg.pull}, seed={cfg.seed}",
            "variant": variant, "op": op, "storage": dtype, "M": cfg.M, "n": cfg.n, "n_layers": cfg.K, "parallelism": par,
            "l2": "inputs larger than L2 (no flush needed)" if op_bytes(cfg, op, dtype) > 4 * 126e6 else "L2-resident workload",
            "algorithmic_bytes_per_step": op_bytes(cfg, op, dtype)}


def op_bytes(cfg, op, dtype="f32", n=None):
    """Algorithmic bytes of one call: gradients read once (step only), parameters read and written
    once, centre written once (step) or read once (proximity step)."""
    n = cfg.n if n is None else n
    e = ELEM_BYTES[dtype]
    streams = {"step": 3 * cfg.M + 1, "from_norms": 2 * cfg.M + 1, "prox": 2 * cfg.M + 1}[op]
    return streams * e * n


def pinned_inputs(cfg):
    """Generates the workload straight into pinned host tensors (also the source of the e2e run)."""
    import torch
    hp = [torch.empty(cfg.n, dtype=torch.float32).pin_memory() for _ in range(cfg.M)]
    hg = [torch.empty(cfg.n, dtype=torch.float32).pin_memory() for _ in range(cfg.M)]
    gen.make_inputs(cfg, [t.numpy() for t in hp], [t.numpy() for t in hg])
    return hp, hg


def device_inputs(cfg, j0=0, j1=None):
    """The workload (or the element range [j0, j1) of it) in device memory, generated on the host."""
    import torch
    p, g = gen.make_inputs(cfg)
    j1 = cfg.n if j1 is None else j1
    x = [torch.from_numpy(a[j0:j1]).cuda() for a in p]
    gr = [torch.from_numpy(a[j0:j1]).cuda() for a in g]
    return x, gr


class Call:
    """One timed operation bound to its buffers: `fn()` enqueues one call on the current stream."""

    def __init__(self, grawa, cfg, variant, op, dtype, x, g, center, off=None):
        import torch
        self.grawa, self.cfg, self.variant, self.op, self.dtype = grawa, cfg, variant, op, dtype
        off = cfg.offsets() if off is None else off
        tdt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[dtype]
        if dtype != "f32":
            x, g, center = [t.to(tdt) for t in x], [t.to(tdt) for t in g], center.to(tdt)
        self.x, self.g, self.center = x, g, center
        if op == "prox":
            self.fn = lambda: grawa.grawa_prox_step_typed(x, center, 0.05 / 16)  # mu / tau of the paper's grid
        elif op == "from_norms":
            norms = torch.empty(cfg.K * cfg.M, dtype=torch.float64, device="cuda")
            grawa.grawa_step_typed("lgrawa", x, g, 0.0, off, None, scores_out=norms)   # per-layer norms, workers untouched
            torch.cuda.synchronize()
            self.norms = norms
            self.fn = lambda: grawa.grawa_step_from_layer_norms_typed(variant, x, norms, cfg.pull, off, center)
        elif dtype == "f32":
            step = {"lgrawa": grawa.grawa_lgrawa_step, "mgrawa": grawa.grawa_mgrawa_step, "grawa": grawa.grawa_grawa_step}[variant]
            self.fn = lambda: step(x, g, cfg.pull, off, center)
        else:
            self.fn = lambda: grawa.grawa_step_typed(variant, x, g, cfg.pull, off, center)

    def time(self, steps, warmup, phases=False):
        """K back-to-back calls between two CUDA events on the launching stream.  Returns ms per call,
        the library's launches inside the region and (if asked) the per-kernel times of a step."""
        import torch
        grawa = self.grawa
        for _ in range(warmup):
            self.fn()
        torch.cuda.synchronize()
        grawa.grawa_set_option("kernel_timing", 1 if phases else 0)
        grawa.grawa_collect_kernel_times()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches = grawa.grawa_launch_count()
        e0.record()
        for _ in range(steps):
            self.fn()
        e1.record()
        torch.cuda.synchronize()
        launches = grawa.grawa_launch_count() - launches
        grawa.grawa_set_option("kernel_timing", 0)
        ph = grawa.grawa_collect_kernel_times() if phases else None
        return e0.elapsed_time(e1) / steps, launches, ph


def per_step_times(call, steps):
    """Each of `steps` further calls between its own pair of CUDA events: median and minimum."""
    import torch
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record()
    for i in range(steps):
        call.fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    t = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(steps))
    return {"steps": steps, "median_ms": t[steps // 2], "min_ms": t[0], "max_ms": t[-1],
            "note": "one event pair per call, taken after the timed region; the headline is the K-call region"}


def rates(bytes_per_call, ms, peak):
    gbs = bytes_per_call / (ms * 1e-3) / 1e9
    return {"ms_per_step": ms, "steps_per_s": 1e3 / ms, "achieved_gbs": gbs, "frac_of_measured_peak": gbs / peak,
            "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}


def kernel_table(cfg, dtype, ph, peak, with_sumsq=True):
    """Per-kernel times of a step (library CUDA events around each kernel, dependent launch off) and the
    roofline of the two streaming kernels."""
    e, n, M = ELEM_BYTES[dtype], cfg.n, cfg.M
    k = ph["steps"]
    out = {"finalize": {"kernel_ms": ph["finalize_ms"] / k}}
    pull_ms, pull_bytes = ph["center_pull_ms"] / k, (2 * M + 1) * e * n
    out["center_pull"] = {"kernel_ms": pull_ms, "algorithmic_bytes_per_launch": pull_bytes,
                          "achieved_gbs": pull_bytes / (pull_ms * 1e-3) / 1e9, "frac_of_measured_peak": pull_bytes / (pull_ms * 1e-3) / 1e9 / peak}
    if with_sumsq:
        s_ms, s_bytes = ph["sumsq_ms"] / k, M * e * n
        out["sumsq"] = {"kernel_ms": s_ms, "algorithmic_bytes_per_launch": s_bytes,
                        "achieved_gbs": s_bytes / (s_ms * 1e-3) / 1e9, "frac_of_measured_peak": s_bytes / (s_ms * 1e-3) / 1e9 / peak}
    return out


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


# ------------------------------------------------------------------ the CPU oracle, timed

def _oracle_step(oracle, variant, p, g, pull, off, bufs):
    """One whole oracle step, streamed in chunks with reused output buffers (allocation is not the method)."""
    n = p[0].size
    S = oracle.sumsq(g, off)
    beta, _ = oracle.weights(oracle.scores(S, variant))
    chunk = bufs[0].size
    for j0 in range(0, n, chunk):
        oracle.center_pull(p, beta, pull, off, j0, min(n, j0 + chunk), out=bufs)


def oracle_timing(cfg, variant, p, g, budget_s, steps_wanted=1, warmup=1):
    """The CPU oracle as it stands (plain C, one thread) on the workload.  Whole steps when one step
    fits the budget; otherwise each step is a prefix of whole layers (all M workers), sized from a
    warmed probe, and the figure is scaled by elements.  Returns the `cpu_baseline` object and the
    measured seconds per (sampled) step."""
    import oracle
    off = cfg.offsets()
    chunk = 1 << 18
    bufs = (np.zeros(chunk), [np.zeros(chunk) for _ in range(cfg.M)])
    probe_n = int(min(cfg.n, 1 << 20))
    view = lambda arrs, hi: [a[:hi] for a in arrs]
    probe_off = np.array([0, probe_n])
    _oracle_step(oracle, variant, view(p, probe_n), view(g, probe_n), cfg.pull, probe_off, bufs)     # warms pages and caches
    t0 = time.perf_counter()
    _oracle_step(oracle, variant, view(p, probe_n), view(g, probe_n), cfg.pull, probe_off, bufs)
    per_elem = (time.perf_counter() - t0) / probe_n
    full_estimate = per_elem * cfg.n
    per_step_budget = budget_s / max(1, steps_wanted + warmup)
    if full_estimate <= per_step_budget:
        k_hi, n_s = cfg.K, cfg.n
    else:
        want = int(per_step_budget / per_elem)
        k_hi = max(1, int(np.searchsorted(off, min(want, cfg.n), side="right")) - 1)
        while k_hi < cfg.K and off[k_hi] == 0:
            k_hi += 1
        n_s = int(off[k_hi])
    soff = off[:k_hi + 1]
    ps, gs = view(p, n_s), view(g, n_s)
    times = []
    for i in range(warmup + steps_wanted):
        t0 = time.perf_counter()
        _oracle_step(oracle, variant, ps, gs, cfg.pull, soff, bufs)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    sec = float(np.mean(times))
    whole = n_s == cfg.n
    sample = (f"{len(times)} whole step(s): all {cfg.K} layers, {cfg.n} elements, {cfg.M} workers" if whole else
              f"{len(times)} step(s) of the first {k_hi} of {cfg.K} layers ({n_s} of {cfg.n} elements, all {cfg.M} workers), "
              f"scaled by elements to a full step")
    full = sec * cfg.n / n_s
    return {"value": 1.0 / full, "unit": "steps/s", "cores": 1, "kind": "oracle", "sample": sample,
            "seconds_per_sampled_step": sec, "whole_steps": whole}, full


def max_over_ranks(values, world, device):
    """Element-wise maximum of per-rank timings (the slowest rank defines the step time)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1 or (dist.is_available() and dist.is_initialized()):
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_steps_per_s(world, ms_per_step_max):
    """Replicas only: every rank runs the same workload, so the job does `world` steps per step time."""
    return world * 1e3 / ms_per_step_max


# DRAM bytes per element of one launch, from stored ncu captures of a smaller case of the same kernel
# (first 28 layers of the ViT-B/16 table, 14 918 400 elements, M = 16), scaled to a full launch by the
# number of elements.  A capture is only quoted for the kernel source and launch code it was taken
# from (hashes of the kernel's code in csrc/kernels.cuh and of the function that launches it in csrc/grawa.cu,
# comments and blank lines left out) and with every tuning
# knob at its default; anything else reports null.
CAPTURE_ELEMENTS = 14918400
STORED_CAPTURES = {
    "center_pull": {"M": 16, "dram_bytes": 955067392 + 953410560, "dram_bytes_full": (86567656, 5541940224 + 5825000448), "begin": "// Steps 4-5, register variant",
                    "end": "// Steps 4-5 for any M up to",
                    "host_begin": "static grawa_status enqueue_center_pull(StepContext", "host_end": "// Given scores of a step",
                    "kernel_sha256": "444a286cacebaa8d7c93389e88c2d8b630a66fc7505a9c644cc49f3a9e74fd66",
                    "host_sha256": "81b9d1b33c91036008ffb4b6a8cd8b72799b0b9f18d617d2a2a48f7b9d052c65"},
    "sumsq": {"M": 16, "dram_bytes": 954848768 + 3460864, "dram_bytes_full": (86567656, 5540634624 + 3330048), "begin": "// Step 1 (Eq. 3 / Eq. 5):",
              "end": "// Steps 4-5, register variant",
              "host_begin": "static grawa_status enqueue_weights_launches(StepContext& c)\n", "host_end": "// Steps 4-5 on 16-bit storage",
              "kernel_sha256": "6c8fcdcd2927db90fe40fdbb204bf18a7a4757f76906c7670ab4625309856fa1",
              "host_sha256": "749ab7388e3b22c197354e8780ec470ca204b4568ffb3a038fbabe3a23e9796a"},
}
DEFAULT_KNOBS = {"sumsq_tile": 8192, "pull_tile": 0, "pull_variant": 0, "bulk_tile": 0, "sumsq_ctas_per_sm": 0,
                 "pull_prefetch_waves": 3, "sumsq_prefetch_waves": 1,
                 "pull_ctas_per_sm": 0, "dependent_launch": 1, "pull_preload": 1, "pull_wide": 1}


def code_only(text):
    """Source text without `//` comments, blank lines and indentation: what a hash of the code should see."""
    lines = (line.split("//")[0].strip() for line in text.splitlines())
    return "\n".join(line for line in lines if line)


def source_hashes(which):
    cap = STORED_CAPTURES[which]
    try:
        text = open(os.path.join(ROOT, "paper_2403_04206_b200", "csrc", "kernels.cuh")).read()
        region = text[text.index(cap["begin"]):text.index(cap["end"])]
        host = open(os.path.join(ROOT, "paper_2403_04206_b200", "csrc", "grawa.cu")).read()
        host = host[host.index(cap["host_begin"]):host.index(cap["host_end"])]      # the code that launches this kernel
    except (OSError, ValueError):
        return None, None
    return hashlib.sha256(code_only(region).encode()).hexdigest(), hashlib.sha256(code_only(host).encode()).hexdigest()


def stored_traffic(grawa, which, cfg):
    """DRAM bytes of one full launch from the stored captures (the one taken at this very size if there
    is one, else the small one scaled by elements), or None when they do not apply."""
    cap = STORED_CAPTURES[which]
    if cap["dram_bytes"] is None or cfg.M != cap["M"]:
        return None
    if any(grawa.grawa_get_option(k) != v for k, v in DEFAULT_KNOBS.items()):
        return None
    if source_hashes(which) != (cap["kernel_sha256"], cap["host_sha256"]):
        return None
    full = cap.get("dram_bytes_full")
    if full and full[0] == cfg.n:
        return float(full[1])
    return cap["dram_bytes"] / CAPTURE_ELEMENTS * cfg.n


# ------------------------------------------------------------------ the CUDA arm

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
    for kv in args.option:
        name, value = kv.split("=")
        grawa.grawa_set_option(name, int(value))

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    peak, peak_src = measured_peak_gbs()
    cfg = workload_config(args)
    variant, op, dtype = args.variant, args.op, args.dtype
    sampler = ClockSampler(local_rank)
    sampler.start()

    # ---- headline: device-resident inputs, exactly K calls
    hp, hg = pinned_inputs(cfg)
    x = [t.cuda(non_blocking=True) for t in hp]
    g = [t.cuda(non_blocking=True) for t in hg]
    center = torch.zeros(cfg.n, device="cuda")
    torch.cuda.synchronize()
    call = Call(grawa, cfg, variant, op, dtype, x, g, center)
    barrier()
    ms, launches, _ = call.time(args.steps, args.warmup)
    barrier()
    each = per_step_times(call, max(10, min(args.steps, 100)))
    line = None
    alg_bytes = op_bytes(cfg, op, dtype)
    if op == "prox":
        kernels, ms_k = None, ms
    else:
        # the same region again with the library's events around each kernel (for the kernel-level roofline)
        ms_k, _, phases = call.time(args.steps, 1, phases=True)
        kernels = kernel_table(cfg, dtype, phases, peak, with_sumsq=(op == "step"))
    status = grawa.grawa_last_step_status() if op != "prox" else 0

    other = None
    if op == "step" and dtype == "f32":
        ov = "mgrawa" if variant == "lgrawa" else "lgrawa"
        o_ms, _, _ = Call(grawa, cfg, ov, "step", "f32", x, g, center).time(max(20, args.steps // 4), 3)
        other = dict(variant=ov, **rates(alg_bytes, o_ms, peak))

    # ---- end to end through the host-buffer entry point (fp32 step only)
    e2e_ms, e2e_steps = None, 0
    if op == "step" and dtype == "f32":
        hc = torch.empty(cfg.n, dtype=torch.float32).pin_memory()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        e2e_ms = time_e2e_steps(grawa, cfg, variant, hp, hg, hc, e2e_steps, 1)
        del hc

    # ---- one problem cut by element range over the ranks (with one rank: the same step through the sharded path)
    sharded_out = None
    if (args.sharded or world > 1) and op == "step" and dtype == "f32":      # always recorded by a multi-rank run
        sharded_out = run_sharded(grawa, cfg, variant, args, world, rank, peak, barrier, x, g, center)

    ms_max, e2e_ms_max = max_over_ranks([ms, e2e_ms if e2e_ms is not None else 0.0], world, "cuda")
    ops = targets = small = many = trace = None
    if world == 1 and not args.headline_only:
        ops = side_ops(grawa, cfg, variant, x, g, center, args, peak)
    del call, x, g, center
    torch.cuda.empty_cache()
    hp_np, hg_np = [t.numpy() for t in hp], [t.numpy() for t in hg]
    if world == 1 and not args.headline_only:
        targets = target_runs(grawa, args, peak, have=(cfg, hp, hg))
        many = many_worker_runs(grawa, args, peak)
        small = small_runs(grawa, args)
        if args.trace_finalize:
            trace = trace_breakdown("resnet18_imagenet")
    clocks = sampler.stop()

    if rank == 0:
        step_rates = rates(alg_bytes, ms_max, peak)
        dominant = "center_pull" if kernels else "prox"
        if kernels:
            kd = kernels["center_pull"]
            roof = {"bound": "hbm", "kernel": dominant, "achieved": kd["achieved_gbs"], "peak": peak, "peak_source": peak_src,
                    "unit": "GB/s", "frac": kd["frac_of_measured_peak"], "frac_of_nominal_8TBs": kd["achieved_gbs"] / NOMINAL_HBM_GBS,
                    "traffic": stored_traffic(grawa, "center_pull", cfg) if dtype == "f32" else None,
                    "traffic_source": "stored ncu capture (dram bytes read + written) of one launch at the same M: taken at this "
                                      f"workload's full size when n = 86567656, otherwise a launch over {CAPTURE_ELEMENTS} elements "
                                      "scaled by elements; null when the kernel, its launch code or a tuning knob differs from the capture's",
                    "traffic_scaled_from_n": None if cfg.n == 86567656 else CAPTURE_ELEMENTS,
                    "algorithmic_bytes_per_launch": kd["algorithmic_bytes_per_launch"], "kernel_ms": kd["kernel_ms"],
                    "timed_with": "library CUDA events around each kernel in a second K-step region (dependent launch off there)",
                    "other_kernels": {k: v for k, v in kernels.items() if k != "center_pull"},
                    "ms_per_step_with_events": ms_k}
            if "sumsq" in roof["other_kernels"]:
                roof["other_kernels"]["sumsq"]["traffic"] = stored_traffic(grawa, "sumsq", cfg) if dtype == "f32" else None
        else:
            roof = {"bound": "hbm", "kernel": "prox", "achieved": step_rates["achieved_gbs"], "peak": peak, "peak_source": peak_src,
                    "unit": "GB/s", "frac": step_rates["frac_of_measured_peak"], "frac_of_nominal_8TBs": step_rates["frac_of_nominal_8TBs"],
                    "traffic": None, "algorithmic_bytes_per_launch": alg_bytes, "kernel_ms": ms_max,
                    "timed_with": "CUDA events around K back-to-back launches (the call is one kernel)"}
        line = {
            "metric": METRIC, "value": whole_job_steps_per_s(world, ms_max), "unit": "steps/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_max, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": dtype, "data": "synthetic",
            "config": describe(cfg, variant, op, dtype, world),
            "step_hbm": {k: step_rates[k] for k in ("achieved_gbs", "frac_of_measured_peak", "frac_of_nominal_8TBs")},
            "roofline": roof, "per_step": each,
            "gpu_launches": launches, "clocks": clocks, "last_step_status": status,
        }
        if e2e_ms is not None:
            line["e2e"] = {"value": whole_job_steps_per_s(world, e2e_ms_max), "unit": "steps/s", "steps": e2e_steps,
                           "h2d_bytes_per_step": 2 * cfg.M * 4 * cfg.n, "d2h_bytes_per_step": (cfg.M + 1) * 4 * cfg.n,
                           "entry_point": "grawa_step_host (pinned host buffers)"}
        if other:
            line["other_variant"] = other
        if targets is not None:
            line["targets"] = targets
        if ops is not None:
            line["ops"] = ops
        if many is not None:
            line["many_workers"] = many
        if small is not None:
            line["small"] = small
        if trace is not None:
            line["in_step_finalize"] = trace
        if sharded_out is not None:
            line["sharded"] = sharded_out
        if world == 1 and not args.no_cpu_baseline and op == "step":
            line["cpu_baseline"], _ = oracle_timing(cfg, variant, hp_np, hg_np, budget_s=20.0)
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()


def side_ops(grawa, cfg, variant, x, g, center, args, peak):
    """Short runs of the other calls on the headline workload's buffers: the proximity step (runs every
    local iteration), the step from given layer norms (no gradient pass) and the step on bfloat16 storage."""
    import torch
    steps = max(20, min(args.steps, 60))
    out = []
    ms, _, _ = Call(grawa, cfg, variant, "prox", "f32", x, g, center).time(steps, 3)
    out.append(dict(op="prox", storage="f32", workload=cfg.name, steps=steps, algorithmic_bytes=op_bytes(cfg, "prox"),
                    **rates(op_bytes(cfg, "prox"), ms, peak)))
    c = Call(grawa, cfg, variant, "from_norms", "f32", x, g, center)
    ms, _, _ = c.time(steps, 3)
    _, _, ph = c.time(steps, 1, phases=True)
    out.append(dict(op="from_norms", variant=variant, storage="f32", workload=cfg.name, steps=steps,
                    algorithmic_bytes=op_bytes(cfg, "from_norms"), kernels=kernel_table(cfg, "f32", ph, peak, with_sumsq=False),
                    **rates(op_bytes(cfg, "from_norms"), ms, peak)))
    del c
    c = Call(grawa, cfg, variant, "step", "bf16", x, g, center)
    ms, _, _ = c.time(steps, 3)
    _, _, ph = c.time(steps, 1, phases=True)
    out.append(dict(op="step", variant=variant, storage="bf16", workload=cfg.name, steps=steps,
                    algorithmic_bytes=op_bytes(cfg, "step", "bf16"), kernels=kernel_table(cfg, "bf16", ph, peak),
                    **rates(op_bytes(cfg, "step", "bf16"), ms, peak)))
    c.op, c.fn = "prox", (lambda xs=c.x, cc=c.center: grawa.grawa_prox_step_typed(xs, cc, 0.05 / 16))   # same bf16 buffers
    ms, _, _ = c.time(steps, 3)
    out.append(dict(op="prox", storage="bf16", workload=cfg.name, steps=steps, algorithmic_bytes=op_bytes(cfg, "prox", "bf16"),
                    **rates(op_bytes(cfg, "prox", "bf16"), ms, peak)))
    del c
    torch.cuda.empty_cache()
    return out


def target_runs(grawa, args, peak, have=None):
    """Every workload of at least 10 M parameters, MGRAWA and LGRAWA: at least 50 steps after 3 warm-up
    steps, with the three kernels' times; buffers are freed between workloads."""
    import torch
    out = []
    steps = max(50, min(args.steps, 200))
    for name in TARGET_WORKLOADS:
        cfg = gen.CONFIGS[name]
        if have is not None and have[0].name == name:
            x, g = [t.cuda() for t in have[1]], [t.cuda() for t in have[2]]
        else:
            x, g = device_inputs(cfg)
        center = torch.zeros(cfg.n, device="cuda")
        for variant in ("mgrawa", "lgrawa"):
            c = Call(grawa, cfg, variant, "step", "f32", x, g, center)
            ms, _, _ = c.time(steps, 3)
            _, _, ph = c.time(steps, 1, phases=True)
            out.append(dict(workload=name, variant=variant, M=cfg.M, n=cfg.n, n_layers=cfg.K, steps=steps,
                            algorithmic_bytes=op_bytes(cfg, "step"), kernels=kernel_table(cfg, "f32", ph, peak),
                            **rates(op_bytes(cfg, "step"), ms, peak)))
            if name == "vgg16" and variant == "lgrawa":
                cb = Call(grawa, cfg, variant, "step", "bf16", x, g, center)
                ms, _, _ = cb.time(steps, 3)
                out.append(dict(workload=name, variant=variant, storage="bf16", M=cfg.M, n=cfg.n, steps=steps,
                                algorithmic_bytes=op_bytes(cfg, "step", "bf16"), **rates(op_bytes(cfg, "step", "bf16"), ms, peak)))
                del cb
        del c, x, g, center
        torch.cuda.empty_cache()
    return out


def many_worker_runs(grawa, args, peak):
    """More workers than the register kernels cover (32, on the ResNet-18 layer table and value recipe;
    3 GB): the centre+pull kernel with a run-time worker count, fp32 and bfloat16 storage."""
    import torch
    M = 32
    cfg = with_workers(gen.CONFIGS["resnet18_imagenet"], M)
    x, g = device_inputs(cfg)
    center = torch.zeros(cfg.n, device="cuda")
    steps = max(50, min(args.steps, 200))
    out = []
    for dtype in ("f32", "bf16"):
        c = Call(grawa, cfg, "lgrawa", "step", dtype, x, g, center)
        ms, _, _ = c.time(steps, 3)
        _, _, ph = c.time(steps, 1, phases=True)
        out.append(dict(workload=cfg.name, variant="lgrawa", storage=dtype, M=M, n=cfg.n, steps=steps,
                        algorithmic_bytes=op_bytes(cfg, "step", dtype), kernels=kernel_table(cfg, dtype, ph, peak),
                        **rates(op_bytes(cfg, "step", dtype), ms, peak)))
        del c
    del x, g, center
    torch.cuda.empty_cache()
    return out


def trace_child(name):
    """Runs in a child process with the trace build selected: eager back-to-back steps of one workload,
    both variants; prints the medians of the device-side stamps as one JSON line."""
    import torch
    import paper_2403_04206_b200 as grawa
    cfg = gen.CONFIGS[name]
    x, g = device_inputs(cfg)
    center = torch.empty(cfg.n, device="cuda")
    out = {}
    steps = 24
    for variant in ("lgrawa", "mgrawa"):
        fn = grawa.PreparedStep(variant, x, g, cfg.pull, cfg.offsets(), center)
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        if grawa.grawa_trace_read() is None:
            print(json.dumps({"unavailable": "not the trace build"}))
            return
        for _ in range(steps):
            fn()
        torch.cuda.synchronize()
        t = grawa.grawa_trace_read().astype(np.int64)[:steps]          # [step, kernel, stamp] in ns
        med = lambda a: float(np.median(a[2:])) / 1e3
        out[variant] = {"finalize_us": med(t[:, 1, 3] - t[:, 1, 1]),
                        "sumsq_exit_to_finalize_start_us": med(t[:, 1, 1] - t[:, 0, 3]),
                        "finalize_exit_to_center_pull_start_us": med(t[:, 2, 1] - t[:, 1, 3])}
    print(json.dumps(out))


def trace_breakdown(name):
    """The finalisation kernel and the two hand-overs around it as they run inside a step (dependent
    launch on), from `%globaltimer` stamps of the library's trace build in a child process.  The stamps
    slow the sum-of-squares kernel down, so only these three short intervals are reported.  The kernel's
    duration here is not what it adds to a step: while it runs, the centre+pull kernel's early loads and
    L2 hints keep DRAM busy (that is their purpose), which lengthens this kernel's few memory round trips."""
    import subprocess
    env = dict(os.environ, GRAWA_TRACE="1")
    try:
        r = subprocess.run([sys.executable, os.path.abspath(__file__), "--trace-child", name], env=env, capture_output=True,
                           text=True, timeout=300)
        line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
        return dict(workload=name, source="trace build of the library, device-side stamps, medians of 22 eager steps", **json.loads(line))
    except Exception as exc:                                     # a diagnostic: never fails the run
        return {"workload": name, "unavailable": repr(exc)[:200]}


def small_runs(grawa, args):
    """The two L2-resident workloads: launch-bound, no roofline target; eager calls and CUDA-graph replays."""
    import torch
    out = []
    for name in SMALL_WORKLOADS:
        cfg = gen.CONFIGS[name]
        x, g = device_inputs(cfg)
        center = torch.zeros(cfg.n, device="cuda")
        off = cfg.offsets()
        for variant in ("mgrawa", "lgrawa"):
            c = Call(grawa, cfg, variant, "step", "f32", x, g, center)
            eager_ms, _, _ = c.time(1000, 20)
            # the same C call with its arguments marshalled once (what a C caller pays per step)
            c.fn = grawa.PreparedStep(variant, x, g, cfg.pull, off, center)
            prepared_ms, _, _ = c.time(1000, 20)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                c.fn()                                             # builds the plan for this stream
                stream.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=stream):
                    c.fn()
                for _ in range(20):
                    graph.replay()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(1000):
                    graph.replay()
                e1.record()
                stream.synchronize()
                # ten steps in one graph: what a step costs inside a larger captured region (no host launch between steps)
                graph10 = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph10, stream=stream):
                    for _ in range(10):
                        c.fn()
                for _ in range(5):
                    graph10.replay()
                f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                f0.record()
                for _ in range(100):
                    graph10.replay()
                f1.record()
                stream.synchronize()
            out.append({"workload": name, "variant": variant, "M": cfg.M, "n": cfg.n, "eager_us": eager_ms * 1e3, "eager_prepared_args_us": prepared_ms * 1e3,
                        "graph_replay_us": e0.elapsed_time(e1), "step_us_inside_a_graph_of_10_steps": f0.elapsed_time(f1),
                        "traffic_time_us_at_8TBs": op_bytes(cfg, "step") / 8e12 * 1e6})
            del graph, graph10
        del x, g, center
    return out


def run_sharded(grawa, cfg, variant, args, world, rank, peak, barrier, x, g, center):
    """ONE problem cut by element range over the ranks: local sums of squares, one all-gather of a [K, M]
    table, the step from the gathered sums.  Strong scaling: the value is steps/s of that one problem."""
    import torch
    import torch.distributed as dist
    from paper_2403_04206_b200 import sharded
    own_group = False
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29551")
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", torch.cuda.current_device()))
        own_group = True
    j0, j1 = sharded.shard_range(cfg.n, world, rank)
    loc = sharded.local_layer_table(cfg.offsets(), j0, j1)
    xs, gs, cs = [t[j0:j1] for t in x], [t[j0:j1] for t in g], center[j0:j1]
    fn = lambda: sharded.sharded_step(variant, xs, gs, cfg.pull, loc, cs)
    steps = max(20, min(args.steps, 100))
    for _ in range(3):
        fn()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    barrier()
    ms = max_over_ranks([e0.elapsed_time(e1) / steps], world, "cuda")[0]
    if own_group:
        dist.destroy_process_group()
    out = {"parallelism": "element-range sharded", "scaling": "strong", "n_gpus": world, "steps": steps,
           "collective": "one all-gather of a [K, M] float64 table per step (NCCL)", "value": 1e3 / ms, "unit": "steps/s"}
    out.update(rates(op_bytes(cfg, "step"), ms, peak * world))
    return out


# ------------------------------------------------------------------ the reference arm (the CPU oracle)

def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = workload_config(args)
    variant = args.variant
    p, g = gen.make_inputs(cfg)
    base, sec = oracle_timing(cfg, variant, p, g, budget_s=150.0, steps_wanted=max(1, args.steps), warmup=max(0, args.warmup))
    value = 1.0 / sec
    base = {k: base[k] for k in ("value", "unit", "cores", "kind", "sample", "whole_steps")}
    world = int(os.environ.get("WORLD_SIZE", "1"))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": describe(cfg, variant, "step", "f32", world),      # rank 0 alone runs the oracle, one problem
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(gen.CONFIGS))
    ap.add_argument("--variant", default=DEFAULT_VARIANT, choices=["lgrawa", "mgrawa", "grawa"])
    ap.add_argument("--op", default="step", choices=["step", "prox", "from_norms"])
    ap.add_argument("--dtype", default="f32", choices=["f32", "bf16", "f16"], help="storage of parameters, gradients and centre")
    ap.add_argument("--sharded", action="store_true",
                    help="also time one problem cut by element range over the ranks (always on with more than one rank)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--headline-only", action="store_true", help="skip the short runs of the other workloads and calls")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workers", type=int, default=0, help="override the workload's number of workers (2..64)")
    ap.add_argument("--layers-limit", type=int, default=0, help="use only the first L layers (small profiling captures)")
    ap.add_argument("--option", action="append", default=[], help="library tuning knob, name=value (repeatable)")
    ap.add_argument("--trace-finalize", action="store_true",
                    help="add device-side stamps of the finalisation kernel inside ResNet-18 steps (trace build, child process)")
    ap.add_argument("--trace-child", default=None, help=argparse.SUPPRESS)
    ap.add_argument("--print-source-hashes", action="store_true",
                    help="print the hashes that tie a stored ncu capture to the kernel source, and exit")
    args = ap.parse_args()
    if args.print_source_hashes:
        print(json.dumps({k: source_hashes(k) for k in STORED_CAPTURES}))
        return
    if args.trace_child:
        trace_child(args.trace_child)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
