"""The N > 1 path of bench.py on CPU: two gloo ranks.  The update itself does not shard
("replicas only"), so what has to work across ranks is the timing reduction (max over ranks), the
whole-job aggregate, and the reference arm's rule that only rank 0 works."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local = [2.0 + rank, 300.0 - 10 * rank]           # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(local, world, "cpu")
    dist.barrier()
    out[rank] = got
    dist.destroy_process_group()


def test_timing_is_the_max_over_two_gloo_ranks():
    with mp.get_context("spawn").Manager() as manager:
        out = manager.dict()
        mp.spawn(_worker, args=(2, 29533, out), nprocs=2, join=True)
        assert out[0] == out[1] == [3.0, 300.0]
    import bench
    assert bench.whole_job_steps_per_s(2, 4.0) == 500.0      # two replicas, 4 ms per step
    assert bench.max_over_ranks([1.5], 1, "cpu") == [1.5]


def test_reference_arm_only_rank_zero_prints():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_reference_arm_line_has_the_contract_keys():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "toy10",
                          "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "steps/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["higher_is_better"] is True and line["config"]["workload"].startswith("toy10")


def test_both_arms_describe_the_workload_with_one_function():
    """The reference arm's `config` equals the CUDA arm's key by key (one GPU, fp32 step)."""
    import bench
    import gen
    cfg = gen.CONFIGS["toy10"]
    a = bench.describe(cfg, "lgrawa", "step", "f32", 1)
    assert a["workload"].startswith("toy10") and a["parallelism"] == "single GPU"
    assert a["algorithmic_bytes_per_step"] == (3 * cfg.M + 1) * 4 * cfg.n == cfg.algorithmic_bytes()
    assert bench.op_bytes(cfg, "prox") == (2 * cfg.M + 1) * 4 * cfg.n == bench.op_bytes(cfg, "from_norms")
    assert bench.op_bytes(cfg, "step", "bf16") * 2 == bench.op_bytes(cfg, "step", "f32")
    assert bench.describe(cfg, "lgrawa", "step", "f32", 4)["parallelism"] == "replicas only"
    assert bench.describe(cfg, "lgrawa", "step", "f32", 4, sharded=True)["parallelism"] == "element-range sharded"


def test_stored_ncu_traffic_is_quoted_only_for_the_captured_kernel_and_default_knobs():
    import bench
    import gen

    class Knobs:
        def __init__(self, **changed):
            self.v = dict(bench.DEFAULT_KNOBS, **changed)

        def grawa_get_option(self, name):
            return self.v[name]

    vit, vgg = gen.CONFIGS["vit_b16"], gen.CONFIGS["vgg16"]
    for which in bench.STORED_CAPTURES:
        kernel_hash, host_hash = bench.source_hashes(which)
        cap = bench.STORED_CAPTURES[which]
        same_source = (kernel_hash, host_hash) == (cap["kernel_sha256"], cap["host_sha256"])
        got = bench.stored_traffic(Knobs(), which, vit)
        assert (got is not None) == (same_source and cap["dram_bytes"] is not None)
        if got is not None:
            assert got == cap["dram_bytes_full"][1] and cap["dram_bytes_full"][0] == vit.n    # the capture at this very size
            part = gen.custom_config([1000, 5_000_000], vit.M)                                # any other size: scaled by elements
            assert abs(bench.stored_traffic(Knobs(), which, part) / (cap["dram_bytes"] / bench.CAPTURE_ELEMENTS * part.n) - 1) < 1e-12
        assert bench.stored_traffic(Knobs(), which, vgg) is None                      # another M
        assert bench.stored_traffic(Knobs(pull_variant=2), which, vit) is None       # a knob off its default


def test_workers_override_keeps_the_layer_table_and_recipe():
    import argparse
    import bench
    import gen
    base = gen.CONFIGS["resnet18_imagenet"]
    args = argparse.Namespace(workload="resnet18_imagenet", workers=32, layers_limit=0)
    cfg = bench.workload_config(args)
    assert cfg.M == 32 and cfg.n == base.n and cfg.K == base.K and np.array_equal(cfg.offsets(), base.offsets())
    assert (cfg.seed, cfg.pull, cfg.grad_recipe, cfg.log10_sigma) == (base.seed, base.pull, base.grad_recipe, base.log10_sigma)
    assert bench.op_bytes(cfg, "step") == (3 * 32 + 1) * 4 * base.n and bench.op_bytes(cfg, "step", "bf16") == (3 * 32 + 1) * 2 * base.n
    small = bench.workload_config(argparse.Namespace(workload="vit_b16", workers=0, layers_limit=28))
    assert small.K == 28 and small.M == gen.CONFIGS["vit_b16"].M and small.n == 14918400 == bench.CAPTURE_ELEMENTS
