"""Element-range sharding: host-side range/table logic and the exchange on CPU (two gloo ranks,
checked with the oracle), and the GPU kernels with the ranks emulated one after another on one GPU."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import gen
import oracle
from paper_2403_04206_b200 import sharded

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_ranges_tile_the_vector_on_aligned_cuts():
    for n in (0, 1, 5, 1000, 269722, 11689512):
        for world in (1, 2, 3, 8):
            ranges = [sharded.shard_range(n, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            for (a0, a1), (b0, b1) in zip(ranges, ranges[1:]):
                assert a1 == b0 and a0 <= a1
            assert all(j0 % 4 == 0 for j0, _ in ranges)
    with pytest.raises(ValueError):
        sharded.shard_range(10, 2, 2)


def test_local_layer_tables_partition_every_layer():
    off = gen.CONFIGS["resnet20_cifar"].offsets()
    n = int(off[-1])
    world = 3
    total = np.zeros(len(off) - 1, dtype=np.int64)
    for r in range(world):
        j0, j1 = sharded.shard_range(n, world, r)
        loc = sharded.local_layer_table(off, j0, j1)
        assert loc[0] == 0 and loc[-1] == j1 - j0 and np.all(np.diff(loc) >= 0) and len(loc) == len(off)
        total += np.diff(loc)
    assert np.array_equal(total, np.diff(off))


def _gloo_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    cfg = gen.custom_config([10, 5000, 0, 3, 12001, 777], 3, seed=91, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    j0, j1 = sharded.shard_range(cfg.n, world, rank)
    loc = sharded.local_layer_table(off, j0, j1)
    # the exchange of the sharded step (the function sharded_step itself calls), with the oracle
    # standing in for the kernels on either side of it
    local = torch.from_numpy(oracle.sumsq([a[j0:j1] for a in g], loc))
    gathered = sharded.exchange_layer_sums(local)
    assert gathered.shape == (world, *local.shape) and bool((gathered[rank] == local).all())
    S = gathered[0].numpy().copy()
    for r in range(1, world):
        S += gathered[r].numpy()
    beta, _ = oracle.weights(oracle.scores(S, "lgrawa"))
    c, _ = oracle.center_pull([a[j0:j1] for a in p], beta, 0.5, loc)
    out[rank] = (j0, j1, S, c)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsharded_result():
    with mp.get_context("spawn").Manager() as manager:
        out = manager.dict()
        mp.spawn(_gloo_worker, args=(2, 29541, out), nprocs=2, join=True)
        cfg = gen.custom_config([10, 5000, 0, 3, 12001, 777], 3, seed=91, log10_sigma=(-2.0, 0.0))
        p, g = gen.make_inputs(cfg)
        ref = oracle.step(p, g, 0.5, "lgrawa", cfg.offsets())
        assert np.array_equal(out[0][2], out[1][2])                       # same table on every rank
        assert np.allclose(out[0][2], ref["S"], rtol=1e-13)
        centre = np.concatenate([out[0][3], out[1][3]])
        assert out[0][1] == out[1][0] and np.allclose(centre, ref["center"], rtol=1e-12, atol=1e-15)


# ------------------------------------------------------------------ GPU

@pytest.mark.gpu
@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
@pytest.mark.parametrize("world", [1, 3])
def test_emulated_ranks_on_one_gpu_match_the_oracle(variant, world):
    """The kernels of the sharded step, ranks run one after another (no rank waits on another):
    local sums per shard, the gathered table, then the step from sums on every shard."""
    import paper_2403_04206_b200 as grawa
    from gpu_util import TOL_BETA_REL, TOL_X_ABS_FACTOR
    cfg = gen.custom_config([10, 50000, 0, 3, 120001, 777], 5, seed=92, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    K, M = cfg.K, cfg.M
    shards = [sharded.shard_range(cfg.n, world, r) for r in range(world)]
    tables = [sharded.local_layer_table(off, j0, j1) for j0, j1 in shards]
    gathered = torch.zeros(world, K, M, dtype=torch.float64, device="cuda")
    for r, (j0, j1) in enumerate(shards):
        gr = [torch.from_numpy(a[j0:j1].copy()).cuda() for a in g]
        grawa.grawa_layer_sumsq(gr, tables[r], gathered[r])
    torch.cuda.synchronize()
    ref = oracle.step(p, g, 0.5, variant, off)
    assert np.allclose(gathered.sum(dim=0).cpu().numpy(), ref["S"], rtol=1e-6)
    tol = TOL_X_ABS_FACTOR * max(float(np.abs(a).max()) for a in p)
    G = K if variant == "lgrawa" else 1
    betas = []
    for r, (j0, j1) in enumerate(shards):
        x = [torch.from_numpy(a[j0:j1].copy()).cuda() for a in p]
        centre = torch.empty(j1 - j0, device="cuda")
        beta = torch.empty(G * M, device="cuda")
        grawa.grawa_step_from_layer_sums(variant, x, gathered, world, 0.5, tables[r], centre, weights_out=beta)
        torch.cuda.synchronize()
        betas.append(beta.cpu().numpy())
        assert np.abs(centre.cpu().numpy() - ref["center"][j0:j1]).max() <= tol
        for m in range(M):
            assert np.abs(x[m].cpu().numpy() - ref["workers"][m][j0:j1]).max() <= tol
    for b in betas[1:]:
        assert np.array_equal(b, betas[0])                                # every rank: the same weights, bit for bit
    nz = ref["beta"].ravel() != 0
    assert np.abs(betas[0][nz] / ref["beta"].ravel()[nz] - 1).max() <= TOL_BETA_REL


@pytest.mark.gpu
def test_sharded_step_through_nccl_with_one_rank():
    """The whole sharded_step call (kernels + NCCL all-gather) in a world of one rank."""
    import paper_2403_04206_b200 as grawa
    from gpu_util import compare_with_oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT="29547")
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        cfg = gen.CONFIGS["resnet20_cifar"]
        p, g = gen.make_inputs(cfg)
        off = cfg.offsets()
        j0, j1 = sharded.shard_range(cfg.n, 1, 0)
        x = [torch.from_numpy(a).cuda() for a in p]
        gr = [torch.from_numpy(a).cuda() for a in g]
        centre = torch.empty(cfg.n, device="cuda")
        sharded.sharded_step("lgrawa", x, gr, 0.5, sharded.local_layer_table(off, j0, j1), centre)
        torch.cuda.synchronize()
        ref = oracle.step(p, g, 0.5, "lgrawa", off)
        tol = 2e-6 * max(float(np.abs(a).max()) for a in p)
        assert np.abs(centre.cpu().numpy() - ref["center"]).max() <= tol
        for m in range(cfg.M):
            assert np.abs(x[m].cpu().numpy() - ref["workers"][m]).max() <= tol
        # bfloat16 replicas through the same call: bit-identical to the unsharded typed step
        xb = [torch.from_numpy(a).cuda().bfloat16() for a in p]
        xr = [t.clone() for t in xb]
        gb = [torch.from_numpy(a).cuda().bfloat16() for a in g]
        cb, cr = torch.zeros(cfg.n, dtype=torch.bfloat16, device="cuda"), torch.zeros(cfg.n, dtype=torch.bfloat16, device="cuda")
        sharded.sharded_step("lgrawa", xb, gb, 0.5, sharded.local_layer_table(off, j0, j1), cb)
        grawa.grawa_step_typed("lgrawa", xr, gb, 0.5, off, cr)
        torch.cuda.synchronize()
        assert bool((cb.view(torch.int16) == cr.view(torch.int16)).all())
        for u, v in zip(xb, xr):
            assert bool((u.view(torch.int16) == v.view(torch.int16)).all())
        # On a stream that is not the current one, behind work that produces the inputs there: the
        # step (kernels and all-gather) must queue up behind that work, not beside it.
        side = torch.cuda.Stream()
        x2 = [torch.empty(cfg.n, device="cuda") for _ in p]
        g2 = [torch.empty(cfg.n, device="cuda") for _ in g]
        centre2 = torch.empty(cfg.n, device="cuda")
        big = torch.empty(1 << 28, device="cuda")
        hp = [torch.from_numpy(a).cuda() for a in p]
        hg = [torch.from_numpy(a).cuda() for a in g]
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            for _ in range(4):
                big.mul_(1.0001)                      # keeps `side` busy while the host runs ahead
            for dst, src in zip(x2 + g2, hp + hg):
                dst.copy_(src)
        sharded.sharded_step("lgrawa", x2, g2, 0.5, sharded.local_layer_table(off, j0, j1), centre2, stream=side)
        side.synchronize()
        assert bool((centre2 == centre).all())
        for u, v in zip(x2, x):
            assert bool((u == v).all())
    finally:
        dist.destroy_process_group()
