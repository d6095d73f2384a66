"""GPU parity: the CUDA path, called through the C ABI, against the float64 oracle on the same
seeded inputs, element by element; plus the exact-arithmetic, determinism and edge-case checks."""
import numpy as np
import pytest

import gen
import oracle
from gpu_util import compare_with_oracle, gpu_step, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def grawa():
    import torch
    assert torch.cuda.is_available()
    import paper_2403_04206_b200 as g
    g.library()          # fails loudly if the CUDA library cannot be built or loaded
    return g


_inputs_cache = {}


def inputs(name):
    """Seeded inputs of a named benchmark workload (kept for the module: the big ones are costly)."""
    if name not in _inputs_cache:
        _inputs_cache.clear()           # hold one big workload at a time
        _inputs_cache[name] = gen.make_inputs(gen.CONFIGS[name])
    return _inputs_cache[name]


# ------------------------------------------------------------------ the five benchmark workloads, full size

@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
@pytest.mark.parametrize("name", ["toy10", "resnet20_cifar", "resnet18_imagenet"])
def test_parity_small_and_medium_workloads(grawa, name, variant):
    cfg = gen.CONFIGS[name]
    p, g = inputs(name)
    res = gpu_step(grawa, variant, p, g, cfg.pull, cfg.offsets())
    stats = compare_with_oracle(res, variant, p, g, cfg.pull, cfg.offsets())
    print(name, variant, stats)
    assert grawa.grawa_last_step_status() == 0


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
@pytest.mark.parametrize("name", ["vgg16", "vit_b16"])
def test_parity_large_workloads(grawa, name, variant):
    cfg = gen.CONFIGS[name]
    p, g = inputs(name)
    res = gpu_step(grawa, variant, p, g, cfg.pull, cfg.offsets())
    stats = compare_with_oracle(res, variant, p, g, cfg.pull, cfg.offsets())
    print(name, variant, stats)
    if name == "vit_b16" and variant == "mgrawa":
        # the worker with 100x larger gradients gets about 1/100 of a peer's weight
        assert 50 < res["beta"][1] / res["beta"][0] < 200


def test_parity_resnet18_table_with_32_workers_full_size(grawa):
    """The many-worker case the benchmark times (ResNet-18 layer table and value recipe, 32 workers):
    element by element against the oracle, per-layer and flat weights."""
    base = gen.CONFIGS["resnet18_imagenet"]
    cfg = gen.custom_config(np.diff(base.offsets()), 32, seed=base.seed, pull=base.pull, grad_recipe=base.grad_recipe,
                            log10_sigma=base.log10_sigma, loud_worker_factor=base.loud_worker_factor)
    _inputs_cache.clear()
    p, g = gen.make_inputs(cfg)
    for variant in ("lgrawa", "mgrawa"):
        res = gpu_step(grawa, variant, p, g, cfg.pull, cfg.offsets())
        compare_with_oracle(res, variant, p, g, cfg.pull, cfg.offsets())
        assert grawa.grawa_last_step_status() == 0
        del res


@pytest.mark.parametrize("pull", [0.3, 0.7])
@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
def test_parity_other_pull_strengths(grawa, variant, pull):
    cfg = gen.CONFIGS["resnet20_cifar"]
    p, g = inputs("resnet20_cifar")
    res = gpu_step(grawa, variant, p, g, pull, cfg.offsets())
    compare_with_oracle(res, variant, p, g, pull, cfg.offsets())


# ------------------------------------------------------------------ adversarial layer tables and worker counts

TABLES = [
    [1], [3], [5], [7], [4], [8192], [8193], [4096, 4096], [4095, 4097],
    [1, 3, 5, 7], [7, 5, 3, 1, 2, 6], [0, 5, 0, 0, 9, 0], [10, 1000, 10, 8192, 3, 20000, 1],
    [16384, 1, 16383, 2, 4094, 4098], [33000], [1023, 1025, 2047, 2049, 4095, 4097, 8191, 8193],
]


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
@pytest.mark.parametrize("sizes", TABLES, ids=lambda s: "-".join(map(str, s)))
def test_parity_adversarial_layer_tables(grawa, sizes, variant):
    cfg = gen.custom_config(sizes, 3, seed=11)
    p, g = gen.make_inputs(cfg)
    res = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets())
    compare_with_oracle(res, variant, p, g, 0.5, cfg.offsets())


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
@pytest.mark.parametrize("M", list(range(1, 18)) + [24, 33, 64])
def test_parity_worker_counts(grawa, M, variant):
    cfg = gen.custom_config([10, 5000, 3, 12000, 777], M, seed=100 + M, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    before = [a.copy() for a in p]
    res = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets())
    compare_with_oracle(res, variant, p, g, 0.5, cfg.offsets(), check_workers=(M > 1))
    if M == 1:   # identity: the worker is untouched, the centre is the worker
        assert np.array_equal(res["workers"][0].cpu().numpy(), before[0])
        assert np.array_equal(res["center"].cpu().numpy(), before[0])


def test_parity_without_layer_table_is_the_flat_norm(grawa):
    cfg = gen.custom_config([30000], 5, seed=5)
    p, g = gen.make_inputs(cfg)
    res = gpu_step(grawa, "mgrawa", p, g, 0.5, None)
    compare_with_oracle(res, "grawa", p, g, 0.5, None)


def test_parity_unaligned_base_pointers(grawa):
    """Workers that start 4 bytes into an allocation take the scalar kernels; results are the same."""
    import torch
    cfg = gen.custom_config([10, 5000, 3, 9000], 4, seed=21)
    p, g = gen.make_inputs(cfg)
    n = cfg.n
    xs = [torch.zeros(n + 1, device="cuda")[1:] for _ in range(4)]
    gs = [torch.zeros(n + 1, device="cuda")[1:] for _ in range(4)]
    for variant in ("mgrawa", "lgrawa"):
        for t, a in zip(xs + gs, p + g):
            t.copy_(torch.from_numpy(a))
        res = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets(), params_dev=xs, grads_dev=gs)
        compare_with_oracle(res, variant, p, g, 0.5, cfg.offsets())


# ------------------------------------------------------------------ exact arithmetic: indexing is bit-exact

def test_sumsq_bit_exact_on_integer_gradients(grawa):
    """Small-integer gradients make every partial sum exact in fp32 and fp64: the S table must be
    bit-identical to the oracle's, which exposes any off-by-one, gap or overlap between work items."""
    sizes = [10, 1000, 8192, 3, 20000, 1, 4097, 70000]
    rng = np.random.default_rng(3)
    off = np.concatenate([[0], np.cumsum(sizes)])
    g = [rng.integers(-3, 4, size=off[-1]).astype(np.float32) for _ in range(3)]
    p = [rng.normal(size=off[-1]).astype(np.float32) for _ in range(3)]
    res = gpu_step(grawa, "lgrawa", p, g, 0.5, off)
    assert np.array_equal(res["S"], oracle.sumsq(g, off))
    # a single 1 at every layer's first and last element
    for k in range(len(sizes)):
        for pos in {off[k], off[k + 1] - 1}:
            g1 = [np.zeros(off[-1], np.float32) for _ in range(2)]
            g1[0][pos] = 1.0
            g1[1][pos] = 2.0
            S = gpu_step(grawa, "lgrawa", p[:2], g1, 0.5, off)["S"]
            expect = np.zeros((len(sizes), 2)); expect[k] = [1, 4]
            assert np.array_equal(S, expect), (k, pos)


def test_centre_bit_exact_with_dyadic_weights(grawa):
    """Gradient norms 1, 1, 2, 4 per layer give weights with short binary expansions only when
    they are dyadic; use norms (1, 1, 1, 1) -> 1/4 each and (1, 1) -> 1/2: with integer parameters
    every product and sum is exact, so centre and workers must match the oracle bit for bit."""
    sizes = [5, 4096, 3, 9001]
    off = np.concatenate([[0], np.cumsum(sizes)])
    n = int(off[-1])
    rng = np.random.default_rng(4)
    for M in (2, 4, 8):
        g = []
        for m in range(M):
            gm = np.zeros(n, np.float32)
            for k in range(len(sizes)):
                gm[off[k] + (m % sizes[k])] = 1.0 if m % 2 == 0 else -1.0     # every layer norm is 1
            g.append(gm)
        p = [rng.integers(-1000, 1000, size=n).astype(np.float32) for _ in range(M)]
        for variant in ("mgrawa", "lgrawa"):
            res = gpu_step(grawa, variant, p, g, 0.5, off)
            ref = oracle.step(p, g, 0.5, variant, off)
            assert np.array_equal(res["beta"].astype(np.float64), ref["beta"])
            assert np.array_equal(res["center"].cpu().numpy().astype(np.float64), ref["center"])
            for m in range(M):
                assert np.array_equal(res["workers"][m].cpu().numpy().astype(np.float64), ref["workers"][m])


def test_layer_boundaries_select_the_right_weights(grawa):
    """LGRAWA with one-hot weights that alternate between workers from layer to layer: every
    element of the centre must be bit-equal to the worker that owns its layer."""
    sizes = [1, 2, 3, 4097, 5, 8191, 1, 8193, 7]
    off = np.concatenate([[0], np.cumsum(sizes)])
    n = int(off[-1])
    rng = np.random.default_rng(5)
    p = [rng.normal(size=n).astype(np.float32) for _ in range(3)]
    g = [rng.normal(size=n).astype(np.float32) for _ in range(3)]
    owner = np.zeros(n, dtype=np.int64)
    for k in range(len(sizes)):
        g[k % 3][off[k]:off[k + 1]] = 0.0       # zero gradient in layer k -> that worker takes weight 1
        owner[off[k]:off[k + 1]] = k % 3
    res = gpu_step(grawa, "lgrawa", p, g, 1.0, off)
    want = np.choose(owner, p)
    assert np.array_equal(res["center"].cpu().numpy(), want)
    for m in range(3):
        assert np.array_equal(res["workers"][m].cpu().numpy(), want)      # full pull


# ------------------------------------------------------------------ invariants on the GPU result itself

@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
def test_pull_extremes_are_bit_exact(grawa, variant):
    cfg = gen.CONFIGS["toy10"]
    p, g = inputs("toy10")
    r1 = gpu_step(grawa, variant, p, g, 1.0, cfg.offsets())
    c = r1["center"].cpu().numpy()
    for w in r1["workers"]:
        assert np.array_equal(w.cpu().numpy(), c)
    r0 = gpu_step(grawa, variant, p, g, 0.0, cfg.offsets())
    for w, a in zip(r0["workers"], p):
        assert np.array_equal(w.cpu().numpy(), a)
    assert np.array_equal(r0["center"].cpu().numpy(), c)


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
def test_run_to_run_bitwise_determinism(grawa, variant):
    cfg = gen.CONFIGS["resnet18_imagenet"]
    p, g = inputs("resnet18_imagenet")
    a = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets())
    b = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets())
    assert np.array_equal(a["S"], b["S"]) and np.array_equal(a["beta"], b["beta"])
    assert np.array_equal(a["center"].cpu().numpy(), b["center"].cpu().numpy())
    for u, v in zip(a["workers"], b["workers"]):
        assert bool((u == v).all())


def test_weights_sum_to_one_and_equal_norms_give_the_mean(grawa):
    import torch
    cfg = gen.custom_config([3000, 17, 9000], 6, seed=8)
    p, g = gen.make_inputs(cfg)
    res = gpu_step(grawa, "lgrawa", p, g, 0.5, cfg.offsets())
    assert np.allclose(res["beta"].sum(axis=1), 1.0, atol=3e-7)
    g_same = [g[0].copy() * (-1) ** m for m in range(6)]          # equal norms
    res = gpu_step(grawa, "mgrawa", p, g_same, 0.5, cfg.offsets())
    assert np.array_equal(res["beta"], np.full(6, np.float32(1 / 6)))
    mean = torch.stack(to_device(p)).double().mean(dim=0).cpu().numpy()
    assert np.abs(res["center"].cpu().numpy() - mean).max() <= 2e-6 * max(np.abs(a).max() for a in p)


def test_centre_invariant_to_worker_permutation(grawa):
    cfg = gen.custom_config([5000, 33, 7000], 5, seed=9)
    p, g = gen.make_inputs(cfg)
    ref = gpu_step(grawa, "lgrawa", p, g, 0.5, cfg.offsets())["center"].cpu().numpy()
    perm = [3, 0, 4, 2, 1]
    got = gpu_step(grawa, "lgrawa", [p[i] for i in perm], [g[i] for i in perm], 0.5, cfg.offsets())["center"].cpu().numpy()
    assert np.abs(got - ref).max() <= 2e-6 * max(np.abs(a).max() for a in p)


# ------------------------------------------------------------------ zero and non-finite scores

def test_zero_and_nonfinite_scores_follow_the_stated_policy(grawa):
    sizes = [100, 5000, 64]
    off = np.concatenate([[0], np.cumsum(sizes)])
    cfg = gen.custom_config(sizes, 4, seed=13)
    p, g = gen.make_inputs(cfg)
    g[1][off[1]:off[2]] = 0.0                       # worker 1 has zero gradient in layer 1
    g[2][:] = 0.0                                   # worker 2 has zero gradient everywhere
    res = gpu_step(grawa, "lgrawa", p, g, 0.5, off)
    compare_with_oracle(res, "lgrawa", p, g, 0.5, off)
    assert np.array_equal(res["beta"][1], [0, 0.5, 0.5, 0]) and np.array_equal(res["beta"][0], [0, 0, 1, 0])
    assert grawa.grawa_last_step_status() == 0
    res = gpu_step(grawa, "mgrawa", p, g, 0.5, off)
    assert np.array_equal(res["beta"], [0, 0, 1, 0])
    # NaN / Inf gradients: flagged, that worker gets weight 0, nothing traps
    g[0][off[1] + 7] = np.nan
    g[3][5] = np.inf
    for variant in ("lgrawa", "mgrawa"):
        res = gpu_step(grawa, variant, p, g, 0.5, off)
        ref_beta, flagged = oracle.weights(oracle.scores(oracle.sumsq(g, off), variant))
        assert flagged and grawa.grawa_last_step_status() == -3
        assert np.allclose(res["beta"], ref_beta, rtol=1e-5)
        assert np.isfinite(res["center"].cpu().numpy()).all()
    # a clean step afterwards clears the status
    g[0][off[1] + 7] = 0.5
    g[3][5] = 0.5
    gpu_step(grawa, "mgrawa", p, g, 0.5, off)
    assert grawa.grawa_last_step_status() == 0


def test_gradient_magnitudes_outside_the_supported_range_take_the_stated_rules(grawa):
    """The squares are taken in fp32: below |g| of about 1e-19 they are subnormal (fewer and fewer
    digits), below about 3.7e-23 exactly zero, so a layer of only such gradients sums to zero and takes
    the zero-score rule (where the float64 oracle still sees norms); a gradient above about 1.8e19
    squares to infinity and takes the non-finite rule.  The other layers are unaffected and match
    the oracle."""
    sizes = [3000, 5000, 7000]
    off = np.concatenate([[0], np.cumsum(sizes)])
    cfg = gen.custom_config(sizes, 4, seed=31, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    for m in range(4):
        g[m][off[1]:off[2]] *= np.float32(1e-25) * (m + 1)       # layer 1: tiny, different per worker
    res = gpu_step(grawa, "lgrawa", p, g, 0.5, off)
    ref_beta, _ = oracle.weights(oracle.scores(oracle.sumsq(g, off), "lgrawa"))
    assert np.all(res["S"][1] == 0) and np.array_equal(res["beta"][1], [0.25] * 4)     # zero-score rule, not the oracle's weights
    assert not np.allclose(ref_beta[1], 0.25, rtol=0.1)
    for k in (0, 2):
        assert np.abs(res["beta"][k] / ref_beta[k] - 1).max() <= 1e-5
    assert grawa.grawa_last_step_status() == 0
    g[3][off[2] + 5] = np.float32(3e19)                          # squares to +inf in fp32, finite in float64
    res = gpu_step(grawa, "lgrawa", p, g, 0.5, off)
    assert grawa.grawa_last_step_status() == -3
    assert res["beta"][2][3] == 0 and abs(res["beta"][2][:3].sum() - 1) < 1e-6
    assert np.isfinite(res["center"].cpu().numpy()).all()


# ------------------------------------------------------------------ optional arguments and the other entry points

def test_caller_workspace_and_no_centre(grawa):
    import torch
    cfg = gen.CONFIGS["resnet20_cifar"]
    p, g = inputs("resnet20_cifar")
    off = cfg.offsets()
    need = grawa.grawa_workspace_bytes(cfg.n, cfg.M, off)
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)                                   # scratch contents must not matter
    ref = gpu_step(grawa, "lgrawa", p, g, 0.5, off)
    res = gpu_step(grawa, "lgrawa", p, g, 0.5, off, workspace=ws[:need], want_center=False)
    assert res["center"] is None
    for u, v in zip(ref["workers"], res["workers"]):
        assert bool((u == v).all())
    with pytest.raises(grawa.GrawaError) as e:
        gpu_step(grawa, "lgrawa", p, g, 0.5, off, workspace=ws[:need - 256])
    assert e.value.status == -4
    with pytest.raises(grawa.GrawaError):
        gpu_step(grawa, "lgrawa", p, g, 0.5, off, workspace=ws[1:need + 1])       # misaligned


@pytest.mark.parametrize("tiles", [(1024, 1024), (4096, 16384), (65536, 2048)])
def test_tile_options_do_not_change_the_result(grawa, tiles):
    cfg = gen.CONFIGS["toy10"]
    p, g = inputs("toy10")
    old = grawa.grawa_get_option("sumsq_tile"), grawa.grawa_get_option("pull_tile")
    try:
        grawa.grawa_set_option("sumsq_tile", tiles[0])
        grawa.grawa_set_option("pull_tile", tiles[1])
        for variant in ("mgrawa", "lgrawa"):
            res = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets())
            compare_with_oracle(res, variant, p, g, 0.5, cfg.offsets())
    finally:
        grawa.grawa_set_option("sumsq_tile", old[0])
        grawa.grawa_set_option("pull_tile", old[1])


@pytest.mark.parametrize("M", [1, 3, 4, 9])
def test_prox_step_parity(grawa, M):
    import torch
    cfg = gen.custom_config([10, 5000, 3, 12001], M, seed=31)
    p, _ = gen.make_inputs(cfg)
    c = gen.make_inputs(gen.custom_config([cfg.n], 1, seed=32))[0][0]
    for a in (0.05 / 16, 0.01 / 32, 0.0, 1.0):
        x = to_device(p)
        grawa.grawa_prox_step(x, torch.from_numpy(c).cuda(), a)
        torch.cuda.synchronize()
        ref = oracle.prox(p, c, a)
        tol = 2e-6 * max(np.abs(q).max() for q in p + [c])
        for m in range(M):
            got = x[m].cpu().numpy()
            assert np.abs(got - ref[m]).max() <= tol
            if a == 0.0:
                assert np.array_equal(got, p[m])
            if a == 1.0:
                assert np.array_equal(got, c)


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
def test_host_buffer_entry_point(grawa, variant):
    import torch
    cfg = gen.CONFIGS["resnet20_cifar"]
    p, g = inputs("resnet20_cifar")
    off = cfg.offsets()
    hp = [torch.from_numpy(a.copy()).pin_memory() for a in p]
    hg = [torch.from_numpy(a.copy()).pin_memory() for a in g]
    hc = torch.empty(cfg.n, dtype=torch.float32).pin_memory()
    grawa.grawa_step_host(variant, hp, hg, 0.5, off, hc)
    dev = gpu_step(grawa, variant, p, g, 0.5, off)
    assert np.array_equal(hc.numpy(), dev["center"].cpu().numpy())
    for m in range(cfg.M):
        assert np.array_equal(hp[m].numpy(), dev["workers"][m].cpu().numpy())
        assert np.array_equal(hg[m].numpy(), g[m])
    # pageable numpy buffers work too
    np_p = [a.copy() for a in p]
    np_c = np.empty(cfg.n, np.float32)
    grawa.grawa_step_host(variant, np_p, g, 0.5, off, np_c)
    assert np.array_equal(np_c, hc.numpy())


def test_step_inside_a_cuda_graph(grawa):
    """After one eager call has built the plan, a step allocates nothing and can be captured."""
    import torch
    cfg = gen.CONFIGS["resnet20_cifar"]
    p, g = inputs("resnet20_cifar")
    off = cfg.offsets()
    stream = torch.cuda.Stream()
    x, gr = to_device(p), to_device(g)
    center = torch.empty(cfg.n, device="cuda")
    with torch.cuda.stream(stream):
        grawa.grawa_lgrawa_step(x, gr, 0.5, off, center)          # builds the plan for this stream
        stream.synchronize()
        for t, a in zip(x, p):
            t.copy_(torch.from_numpy(a))
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            grawa.grawa_lgrawa_step(x, gr, 0.5, off, center, stream=torch.cuda.current_stream())
    ref = gpu_step(grawa, "lgrawa", p, g, 0.5, off)
    for _ in range(5):           # every replay starts from clean sums (the two copies of the exact sums take turns)
        for t, a in zip(x, p):
            t.copy_(torch.from_numpy(a))
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert bool((center == ref["center"]).all())
        for u, v in zip(x, ref["workers"]):
            assert bool((u == v).all())


def test_captured_step_with_a_callers_workspace_and_status_word(grawa):
    """A caller's scratch buffer and status word inside a captured step: the part of the scratch that
    carries state is cleared by a node of the graph, so replays start clean whatever the buffer held,
    and the status word is rewritten by every replay."""
    import torch
    cfg = gen.custom_config([10, 50000, 0, 3, 120000, 777], 6, seed=77, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    ref = {v: gpu_step(grawa, v, p, g, 0.5, off) for v in ("lgrawa", "mgrawa")}
    need = grawa.grawa_workspace_bytes(cfg.n, cfg.M, off)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.Stream()
    for variant, fn in (("lgrawa", grawa.grawa_lgrawa_step), ("mgrawa", grawa.grawa_mgrawa_step)):
        x, gr = to_device(p), to_device(g)
        center = torch.empty(cfg.n, device="cuda")
        with torch.cuda.stream(stream):
            fn(x, gr, 0.5, off, center, workspace=ws, status_word=word)        # builds the plan for this stream
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                fn(x, gr, 0.5, off, center, workspace=ws, status_word=word, stream=torch.cuda.current_stream())
        for rep in range(4):
            for t, a in zip(x, p):
                t.copy_(torch.from_numpy(a))
            ws.fill_(0xFF if rep % 2 else 0x5A)          # whatever the caller did with its buffer in between
            word.fill_(9)
            if rep == 2:
                gr[1][off[1] + 3] = float("nan")         # this replay meets a non-finite score
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            if rep == 2:
                assert int(word.item()) == 1
                gr[1].copy_(torch.from_numpy(g[1]))
                continue
            assert int(word.item()) == 0
            assert bool((center == ref[variant]["center"]).all())
            for u, v in zip(x, ref[variant]["workers"]):
                assert bool((u == v).all())
        del graph


def test_prepared_step_makes_the_same_call(grawa):
    """The step with its arguments marshalled once gives the same bytes as the plain binding call,
    for fp32 and for 16-bit storage, and keeps doing so when called again."""
    import torch
    cfg = gen.CONFIGS["resnet20_cifar"]
    p, g = inputs("resnet20_cifar")
    off = cfg.offsets()
    for dt in (torch.float32, torch.bfloat16):
        xa = [torch.from_numpy(a).cuda().to(dt) for a in p]
        xb = [t.clone() for t in xa]
        gr = [torch.from_numpy(a).cuda().to(dt) for a in g]
        ca, cb = torch.zeros(cfg.n, dtype=dt, device="cuda"), torch.zeros(cfg.n, dtype=dt, device="cuda")
        word = torch.full((1,), 5, dtype=torch.int32, device="cuda")
        step = grawa.PreparedStep("lgrawa", xb, gr, 0.5, off, cb, status_word=word)
        for _ in range(3):
            grawa.grawa_step_typed("lgrawa", xa, gr, 0.5, off, ca)
            step()
            torch.cuda.synchronize()
            assert bool((ca == cb).all()) and all(bool((u == v).all()) for u, v in zip(xa, xb))
            assert int(word.item()) == 0


# ------------------------------------------------------------------ the bulk-copy centre+pull kernel

@pytest.fixture
def bulk_variant(grawa):
    old = grawa.grawa_get_option("pull_variant")
    grawa.grawa_set_option("pull_variant", 2)
    yield grawa
    grawa.grawa_set_option("pull_variant", old)
    grawa.grawa_set_option("bulk_tile", 0)


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
@pytest.mark.parametrize("name", ["toy10", "resnet20_cifar", "resnet18_imagenet"])
def test_bulk_variant_parity_on_workloads(bulk_variant, name, variant):
    cfg = gen.CONFIGS[name]
    p, g = inputs(name)
    res = gpu_step(bulk_variant, variant, p, g, cfg.pull, cfg.offsets())
    compare_with_oracle(res, variant, p, g, cfg.pull, cfg.offsets())
    assert bulk_variant.grawa_last_step_status() == 0


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
@pytest.mark.parametrize("sizes", [[1], [3], [7, 5, 3, 1, 2, 6], [0, 5, 0, 0, 9, 0], [10, 1000, 10, 8192, 3, 20000, 1],
                                   [1023, 1025, 2047, 2049, 4095, 4097, 8191, 8193], [33000]],
                         ids=lambda s: "-".join(map(str, s)))
def test_bulk_variant_parity_on_adversarial_tables(bulk_variant, sizes, variant):
    cfg = gen.custom_config(sizes, 3, seed=11)
    p, g = gen.make_inputs(cfg)
    for tile in (0, 256, 2048):
        bulk_variant.grawa_set_option("bulk_tile", tile)
        res = gpu_step(bulk_variant, variant, p, g, 0.5, cfg.offsets())
        compare_with_oracle(res, variant, p, g, 0.5, cfg.offsets())
        assert bulk_variant.grawa_last_step_status() == 0


@pytest.mark.parametrize("M", [2, 3, 5, 8, 13, 16, 17, 24, 33, 64])
def test_bulk_variant_parity_on_worker_counts(bulk_variant, M):
    cfg = gen.custom_config([10, 50000, 3, 120000, 777], M, seed=100 + M, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    for variant in ("mgrawa", "lgrawa"):
        res = gpu_step(bulk_variant, variant, p, g, 0.5, cfg.offsets())
        compare_with_oracle(res, variant, p, g, 0.5, cfg.offsets())
        assert bulk_variant.grawa_last_step_status() == 0


def test_bulk_and_register_variants_agree_bit_for_bit(grawa):
    """Same arithmetic in the same order: the two centre+pull kernels must give identical bytes."""
    cfg = gen.CONFIGS["resnet18_imagenet"]
    p, g = inputs("resnet18_imagenet")
    ref = gpu_step(grawa, "lgrawa", p, g, 0.5, cfg.offsets())
    old = grawa.grawa_get_option("pull_variant")
    try:
        grawa.grawa_set_option("pull_variant", 2)
        got = gpu_step(grawa, "lgrawa", p, g, 0.5, cfg.offsets())
    finally:
        grawa.grawa_set_option("pull_variant", old)
    assert bool((ref["center"] == got["center"]).all())
    for u, v in zip(ref["workers"], got["workers"]):
        assert bool((u == v).all())


def test_many_workers_take_the_shared_memory_kernel_by_default(grawa):
    """More than 16 workers: the default is the kernel with a run-time worker count that stages its
    columns through shared memory (any M up to 64); lambda 0.3 and a 33-element layer between two
    long ones exercise its edges."""
    cfg = gen.custom_config([100000, 33, 200001], 40, seed=77, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    res = gpu_step(grawa, "lgrawa", p, g, 0.3, cfg.offsets())
    compare_with_oracle(res, "lgrawa", p, g, 0.3, cfg.offsets())
    assert grawa.grawa_last_step_status() == 0


@pytest.mark.parametrize("M", [17, 31, 64])
def test_many_worker_kernel_matches_the_bulk_kernel_bit_for_bit_and_is_exact_at_the_pull_extremes(grawa, M):
    """The run-time-M shared-memory kernel takes the same fused multiply-add chain in the same order
    as the other centre+pull kernels: identical bytes; pull 1 puts every worker on the centre, pull 0
    leaves every worker untouched."""
    cfg = gen.custom_config([7, 5001, 0, 3, 12001, 777, 8, 9, 8192, 8193, 40000], M, seed=300 + M, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    ref = gpu_step(grawa, "lgrawa", p, g, 0.3, off)
    compare_with_oracle(ref, "lgrawa", p, g, 0.3, off)
    grawa.grawa_set_option("pull_variant", 2)
    try:
        got = gpu_step(grawa, "lgrawa", p, g, 0.3, off)
    finally:
        grawa.grawa_set_option("pull_variant", 0)
    assert bool((ref["center"] == got["center"]).all())
    for u, v in zip(ref["workers"], got["workers"]):
        assert bool((u == v).all())
    full = gpu_step(grawa, "mgrawa", p, g, 1.0, off)
    for w in full["workers"]:
        assert bool((w == full["center"]).all())
    none = gpu_step(grawa, "lgrawa", p, g, 0.0, off)
    for w, a in zip(none["workers"], p):
        assert np.array_equal(w.cpu().numpy(), a)


@pytest.mark.parametrize("case", range(40))
def test_parity_on_seeded_random_tables(grawa, case):
    """Random layer tables (empty, tiny, odd and long layers mixed), worker counts across every
    centre+pull kernel, pull strengths and variants, all drawn from the case number."""
    rng = np.random.default_rng(9000 + case)
    K = int(rng.integers(1, 14))
    kinds = rng.integers(0, 5, size=K)
    sizes = [int({0: 0, 1: rng.integers(1, 9), 2: rng.integers(9, 3000), 3: 4 * rng.integers(256, 9000),
                  4: rng.integers(20000, 90000)}[int(k)]) for k in kinds]
    if sum(sizes) == 0:
        sizes[-1] = 1234
    M = int(rng.choice([2, 3, 4, 5, 7, 8, 9, 12, 16, 17, 20, 29, 40, 64]))
    variant = ["mgrawa", "lgrawa", "grawa"][case % 3]
    pull = float(rng.choice([0.1, 0.3, 0.5, 0.7, 0.9]))
    cfg = gen.custom_config(sizes, M, seed=9000 + case, log10_sigma=(-3.0, 0.0))
    p, g = gen.make_inputs(cfg)
    res = gpu_step(grawa, variant, p, g, pull, cfg.offsets())
    compare_with_oracle(res, variant, p, g, pull, cfg.offsets())
    assert grawa.grawa_last_step_status() == 0


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
@pytest.mark.parametrize("M", [5, 64])
def test_parity_with_thousands_of_tiny_layers(grawa, M, variant):
    """3000 layers of 0..50 elements: every (layer, worker) row is its own item, the one-CTA
    finalisation walks long runs of layers per thread, most centre+pull items are ragged."""
    rng = np.random.default_rng(31)
    sizes = [int(v) for v in rng.integers(0, 51, size=3000)]
    cfg = gen.custom_config(sizes, M, seed=640 + M, log10_sigma=(-3.0, 0.0))
    p, g = gen.make_inputs(cfg)
    res = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets())
    compare_with_oracle(res, variant, p, g, 0.5, cfg.offsets())
    assert grawa.grawa_last_step_status() == 0
    again = gpu_step(grawa, variant, p, g, 0.5, cfg.offsets())            # tickets and digit rows left clean
    for key in ("S", "A", "beta"):
        assert np.array_equal(again[key], res[key]), key
    assert bool((again["center"] == res["center"]).all())


@pytest.mark.parametrize("M", [2, 3, 4, 7, 8, 9, 13, 16])
def test_32_byte_and_16_byte_accesses_agree_bit_for_bit(grawa, M):
    """Bases aligned to 32 bytes take 32-byte loads and stores, bases aligned to 16 bytes only (here
    every vector starts 16 bytes into its allocation) the 16-byte ones: same arithmetic, same bytes out,
    for the averaging step and for the proximity step; both against the oracle."""
    import torch
    cfg = gen.custom_config([7, 5001, 0, 3, 12001, 777, 8, 9, 8192, 8193, 40000], M, seed=700 + M, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()

    def shifted(arrs):
        out = []
        for a in arrs:
            t = torch.zeros(a.size + 4, device="cuda")[4:]
            assert t.data_ptr() % 32 == 16
            t.copy_(torch.from_numpy(a))
            out.append(t)
        return out
    for variant in ("lgrawa", "mgrawa"):
        wide = gpu_step(grawa, variant, p, g, 0.3, off)
        compare_with_oracle(wide, variant, p, g, 0.3, off)
        narrow = gpu_step(grawa, variant, p, g, 0.3, off, params_dev=shifted(p), grads_dev=shifted(g))
        compare_with_oracle(narrow, variant, p, g, 0.3, off)
        assert bool((wide["center"] == narrow["center"]).all())
        for u, v in zip(wide["workers"], narrow["workers"]):
            assert bool((u == v).all())
    xa, xb = to_device(p), shifted(p)
    ca, cb = to_device([g[0]])[0], shifted([g[0]])[0]
    grawa.grawa_prox_step(xa, ca, 0.05 / 16)
    grawa.grawa_prox_step(xb, cb, 0.05 / 16)
    torch.cuda.synchronize()
    for u, v in zip(xa, xb):
        assert bool((u == v).all())


def test_two_host_threads_on_their_own_streams_and_buffers(grawa):
    """Calls with different streams and disjoint buffers may run concurrently: two host threads, each
    with its own stream, problem shape and variant, forty steps each from fresh parameters; every
    result equals the one the same call gives alone, bit for bit."""
    import threading
    import torch
    jobs = [("lgrawa", gen.custom_config([7, 50001, 0, 3, 120001, 777], 5, seed=801, log10_sigma=(-2.0, 0.0))),
            ("mgrawa", gen.custom_config([4096, 64, 65536, 300001], 8, seed=802, log10_sigma=(-2.0, 0.0)))]
    data, alone = [], []
    for variant, cfg in jobs:
        p, g = gen.make_inputs(cfg)
        data.append((p, g))
        res = gpu_step(grawa, variant, p, g, 0.4, cfg.offsets())
        compare_with_oracle(res, variant, p, g, 0.4, cfg.offsets())
        alone.append(res)
    out, errors = [None, None], []

    def run(i):
        try:
            variant, cfg = jobs[i]
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                x0, g = to_device(data[i][0]), to_device(data[i][1])
                x = [t.clone() for t in x0]
                center = torch.empty(cfg.n, device="cuda")
                step = grawa.grawa_lgrawa_step if variant == "lgrawa" else grawa.grawa_mgrawa_step
                for _ in range(40):
                    for t, t0 in zip(x, x0):
                        t.copy_(t0)
                    step(x, g, 0.4, cfg.offsets(), center, stream=stream)
                stream.synchronize()
                assert grawa.grawa_last_step_status(stream) == 0
            out[i] = (x, center)
        except Exception as exc:                                  # surfaced in the main thread
            errors.append(exc)
    threads = [threading.Thread(target=run, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for i in range(2):
        x, center = out[i]
        assert bool((center == alone[i]["center"]).all())
        for u, v in zip(x, alone[i]["workers"]):
            assert bool((u == v).all())


# ------------------------------------------------------------------ repeated steps on one plan

@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
def test_repeated_steps_on_one_plan_leave_clean_counters(grawa, variant):
    """The two copies of the exact sums take turns and each is cleared while the other is in use;
    step after step must give the same bytes."""
    cfg = gen.custom_config([10, 50000, 0, 3, 120000, 777, 0], 7, seed=55, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    first = gpu_step(grawa, variant, p, g, 0.5, off)
    compare_with_oracle(first, variant, p, g, 0.5, off)
    for _ in range(4):
        again = gpu_step(grawa, variant, p, g, 0.5, off)
        for key in ("S", "A", "beta"):
            assert np.array_equal(again[key], first[key]), key
        assert bool((again["center"] == first["center"]).all())
        assert grawa.grawa_last_step_status() == 0


def test_parity_one_huge_layer_among_small_ones(grawa):
    """A layer of more than 1024 base tiles takes a larger tile (fewer partial sums); indexing of
    the neighbours and the exact-integer sums must be unaffected."""
    sizes = [7, 20_000_003, 5, 4096]
    off = np.concatenate([[0], np.cumsum(sizes)])
    rng = np.random.default_rng(8)
    g = [rng.integers(-2, 3, size=off[-1]).astype(np.float32) for _ in range(2)]
    p = [rng.normal(size=off[-1]).astype(np.float32) for _ in range(2)]
    res = gpu_step(grawa, "lgrawa", p, g, 0.5, off)
    assert np.array_equal(res["S"], oracle.sumsq(g, off))
    compare_with_oracle(res, "lgrawa", p, g, 0.5, off)


@pytest.mark.parametrize("M,sizes", [(1, [10, 5000, 3]), (3, [7, 5, 3, 1, 2, 6]), (5, [10, 3_000_001, 0, 3, 1_200_001, 777]),
                                     (20, [100001, 33, 200001])],
                         ids=["one-worker", "tiny", "chunked", "many-workers"])
def test_host_buffer_entry_point_on_ragged_problems(grawa, M, sizes):
    """The host-buffer call runs centre+pull chunk by chunk (several chunks for the large case);
    chunk cuts, unaligned layer edges and the many-worker kernel must give the device-buffer result."""
    cfg = gen.custom_config(sizes, M, seed=300 + M, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    for variant in ("mgrawa", "lgrawa"):
        hp = [a.copy() for a in p]
        hc = np.full(cfg.n, np.nan, np.float32)
        grawa.grawa_step_host(variant, hp, g, 0.5, off, hc)
        dev = gpu_step(grawa, variant, p, g, 0.5, off)
        assert np.array_equal(hc, dev["center"].cpu().numpy())
        for m in range(M):
            assert np.array_equal(hp[m], dev["workers"][m].cpu().numpy())
        compare_with_oracle(dev, variant, p, g, 0.5, off, check_workers=(M > 1))


def test_more_than_2_to_31_elements_per_worker(grawa):
    """Index arithmetic beyond 32 bits: 2^31 + 12345 elements per worker (34 GB on the device for two
    workers), one layer of 2^31 - 5 elements and a short one behind it.  Sums of squares are checked
    in full against the oracle, centre and workers on ranges at the start, across 2^31 and at the end."""
    import psutil
    import torch
    if psutil.virtual_memory().available < 100e9 or torch.cuda.mem_get_info()[0] < 60e9:
        pytest.skip("needs about 100 GB of host memory and 60 GB of device memory")
    n = (1 << 31) + 12345
    off = np.array([0, (1 << 31) - 5, n], dtype=np.int64)
    block = gen.make_inputs(gen.custom_config([1 << 20], 4, seed=404, log10_sigma=(-2.0, 0.0)))
    reps = n // (1 << 20) + 1
    p = [np.tile(block[0][m], reps)[:n] for m in range(2)]
    g = [np.tile(block[1][m + 2], reps)[:n] * np.float32(1 + m) for m in range(2)]
    g[1][-12345:] *= np.float32(5.0)                       # the short layer gets different weights
    res = gpu_step(grawa, "lgrawa", p, g, 0.5, off)
    S = oracle.sumsq(g, off)
    assert np.allclose(res["S"], S, rtol=1e-6, atol=0)
    beta, _ = oracle.weights(oracle.scores(S, "lgrawa"))
    assert np.abs(res["beta"] / beta - 1).max() <= 1e-5
    assert abs(beta[0, 0] - beta[1, 0]) > 0.1              # the two layers really differ
    tol = 2e-6 * max(float(np.abs(a).max()) for a in p)
    centre = res["center"]
    for j0, j1 in [(0, 1 << 20), ((1 << 31) - (1 << 19), (1 << 31) + 12345), (n - (1 << 18), n)]:
        c, w = oracle.center_pull(p, beta, 0.5, off, j0, j1)
        assert np.abs(centre[j0:j1].cpu().numpy() - c).max() <= tol
        for m in range(2):
            assert np.abs(res["workers"][m][j0:j1].cpu().numpy() - w[m]).max() <= tol
    assert grawa.grawa_last_step_status() == 0


def test_bounded_device_wait_times_out_and_the_context_stays_usable(grawa):
    """A wait that nothing will ever satisfy (a barrier nobody signals, inside the library's own
    self-test kernel) must give up after its time limit, report GRAWA_ERR_TIMEOUT through the status
    word, and leave the context healthy: the next step runs and is correct."""
    import time
    import torch
    t0 = time.perf_counter()
    grawa.grawa_selftest_bounded_wait(2_000_000)            # 2 ms limit
    assert grawa.grawa_last_step_status() == -5
    assert time.perf_counter() - t0 < 1.0
    assert "wait" in grawa.grawa_status_string(-5)
    with pytest.raises(grawa.GrawaError):
        grawa.grawa_selftest_bounded_wait(10)               # limit out of range: rejected on the host
    cfg = gen.custom_config([10, 5000, 3, 9000], 4, seed=21)
    p, g = gen.make_inputs(cfg)
    res = gpu_step(grawa, "lgrawa", p, g, 0.5, cfg.offsets())
    compare_with_oracle(res, "lgrawa", p, g, 0.5, cfg.offsets())
    assert grawa.grawa_last_step_status() == 0
    torch.cuda.synchronize()
