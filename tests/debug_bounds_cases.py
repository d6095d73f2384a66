"""Run by tests/test_gpu_debug_bounds.py in a process of its own with GRAWA_DEBUG_BOUNDS=1, so that the
bounds-checking build of the library is the one loaded.  Runs ragged problems through every
streaming kernel and prints the number of out-of-range accesses the kernels would have made."""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))


def main():
    import torch
    import gen
    import paper_2403_04206_b200 as grawa
    from gpu_util import compare_with_oracle, gpu_step

    assert os.environ.get("GRAWA_DEBUG_BOUNDS") == "1"
    grawa.library()
    out = {"selfcheck": grawa.grawa_debug_bounds_violations(selfcheck=True), "cases": 0}
    tables = [[1], [3], [7, 5, 3, 1, 2, 6], [0, 5, 0, 0, 9, 0], [10, 1000, 10, 8192, 3, 20000, 1], [8193], [33000],
              [1023, 1025, 2047, 2049, 4095, 4097, 8191, 8193], [9_000_001, 5]]
    for sizes in tables:
        for M in (1, 2, 3, 4, 8, 16, 17):
            cfg = gen.custom_config(sizes, M, seed=len(sizes) * 100 + M, log10_sigma=(-2.0, 0.0))
            p, g = gen.make_inputs(cfg)
            for variant in ("mgrawa", "lgrawa"):
                res = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets())
                if M in (2, 16) and cfg.n < 100000:
                    compare_with_oracle(res, variant, p, g, 0.5, cfg.offsets())
                out["cases"] += 1
            for dt in (torch.bfloat16, torch.float16):            # 16-bit kernels
                x = [torch.from_numpy(a).cuda().to(dt) for a in p]
                gr = [torch.from_numpy(a).cuda().to(dt) for a in g]
                c = torch.empty(cfg.n, dtype=dt, device="cuda")
                grawa.grawa_step_typed("lgrawa", x, gr, 0.5, cfg.offsets(), c)
                out["cases"] += 1
            xs32 = [torch.from_numpy(a).cuda() for a in p]         # proximity step, fp32 and 16-bit
            grawa.grawa_prox_step(xs32, torch.from_numpy(g[0]).cuda(), 0.01)
            grawa.grawa_prox_step_typed([t.bfloat16() for t in xs32], torch.from_numpy(g[0]).cuda().bfloat16(), 0.01)
            sq = torch.empty(M, dtype=torch.float64, device="cuda")  # the sums of squares on built-in scratch
            grawa.grawa_sumsq_static([torch.from_numpy(a).cuda() for a in g], sq)
            out["cases"] += 3
            if M > 1 and cfg.n < 100000:                           # bulk-copy kernel and the host-buffer path
                grawa.grawa_set_option("pull_variant", 2)
                gpu_step(grawa, "lgrawa", p, g, 0.5, cfg.offsets())
                grawa.grawa_set_option("pull_variant", 0)
                grawa.grawa_step_host("lgrawa", [a.copy() for a in p], g, 0.5, cfg.offsets(), np.empty(cfg.n, np.float32))
                out["cases"] += 2
    # unaligned bases (scalar kernels)
    cfg = gen.custom_config([10, 5000, 3, 9000], 4, seed=21)
    p, g = gen.make_inputs(cfg)
    xs = [torch.zeros(cfg.n + 1, device="cuda")[1:] for _ in range(4)]
    gs = [torch.zeros(cfg.n + 1, device="cuda")[1:] for _ in range(4)]
    gpu_step(grawa, "lgrawa", p, g, 0.5, cfg.offsets(), params_dev=xs, grads_dev=gs)
    out["cases"] += 1
    # thousands of tiny layers (finalisation over several CTAs) and many workers (run-time-M kernel)
    rng = np.random.default_rng(3)
    for M in (5, 33, 64):
        cfg = gen.custom_config([int(v) for v in rng.integers(0, 41, size=2500)] + [50001], M, seed=900 + M, log10_sigma=(-2.0, 0.0))
        p, g = gen.make_inputs(cfg)
        for variant in ("mgrawa", "lgrawa", "grawa"):
            res = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets())
            if M == 5:
                compare_with_oracle(res, variant, p, g, 0.5, cfg.offsets())
            out["cases"] += 1
        norms = torch.from_numpy(10.0 ** rng.uniform(-2, 1, size=(cfg.K, M))).cuda()
        grawa.grawa_step_from_layer_norms("lgrawa", [torch.from_numpy(a).cuda() for a in p], norms, 0.5, cfg.offsets(), None)
        x16 = [torch.from_numpy(a).cuda().bfloat16() for a in p]
        grawa.grawa_step_typed("lgrawa", x16, [torch.from_numpy(a).cuda().bfloat16() for a in g], 0.5, cfg.offsets(), None)
        out["cases"] += 2
    torch.cuda.synchronize()
    out["violations"] = grawa.grawa_debug_bounds_violations()
    print(json.dumps(out))


if __name__ == "__main__":
    main()
