"""GPU parity of the step on 16-bit storage (bfloat16 / float16 parameters, gradients, centre).

The inputs are exactly representable in fp32, so the oracle runs on their fp32 images.  The GPU
rounds each result to the storage type once, so the bound is the fp32 bound of the parity contract
plus half a unit in the last place of the storage type at the oracle's value."""
import numpy as np
import pytest

import gen
import oracle
from gpu_util import TOL_BETA_REL, TOL_S_REL, TOL_X_ABS_FACTOR

pytestmark = pytest.mark.gpu

HALF_ULP = {"bfloat16": 2.0 ** -8, "float16": 2.0 ** -11}      # relative, normal range
TINY = {"bfloat16": 0.0, "float16": 2.0 ** -25}                # half the smallest fp16 subnormal step


@pytest.fixture(scope="module")
def grawa():
    import paper_2403_04206_b200 as g
    g.library()
    return g


def run_typed(grawa, dtype_name, variant, p32, g32, pull, off, want_center=True, offset_elems=0):
    """p32/g32: fp32 numpy inputs; they are rounded to the storage type first (that is the problem
    both sides then solve).  Returns GPU results as fp32 numpy plus the fp32 images of the inputs."""
    import torch
    dt = getattr(torch, dtype_name)

    def dev(a):
        t = torch.zeros(a.size + offset_elems, dtype=dt, device="cuda")
        t[offset_elems:] = torch.from_numpy(a).cuda().to(dt)
        return t[offset_elems:]
    x = [dev(a) for a in p32]
    g = [dev(a) for a in g32]
    p_img = [t.float().cpu().numpy() for t in x]
    g_img = [t.float().cpu().numpy() for t in g]
    M, n = len(x), p32[0].size
    K = len(off) - 1
    G = K if variant == "lgrawa" else 1
    beta = torch.empty(G * M, device="cuda")
    sumsq = torch.empty(K * M, dtype=torch.float64, device="cuda")
    center = torch.zeros(n, dtype=dt, device="cuda") if want_center else None
    grawa.grawa_step_typed(variant, x, g, pull, off, center, weights_out=beta, sumsq_out=sumsq)
    assert grawa.grawa_last_step_status() == 0
    return {"workers": [t.float().cpu().numpy() for t in x], "center": center.float().cpu().numpy() if want_center else None,
            "beta": beta.cpu().numpy(), "S": sumsq.cpu().numpy().reshape(K, M), "p_img": p_img, "g_img": g_img}


def check(res, dtype_name, variant, pull, off, check_workers=True):
    p, g = res["p_img"], res["g_img"]
    ref = oracle.step(p, g, pull, variant, off)
    assert np.allclose(res["S"], ref["S"], rtol=TOL_S_REL, atol=0)
    rb = ref["beta"].ravel()
    nz = rb != 0
    assert np.abs(res["beta"][nz] / rb[nz] - 1).max() <= TOL_BETA_REL
    base = TOL_X_ABS_FACTOR * max(float(np.abs(a).max()) for a in p)
    hu, tiny = HALF_ULP[dtype_name], TINY[dtype_name]
    if res["center"] is not None:
        assert np.all(np.abs(res["center"] - ref["center"]) <= base + hu * np.abs(ref["center"]) + tiny)
    if check_workers:
        for m in range(len(p)):
            assert np.all(np.abs(res["workers"][m] - ref["workers"][m]) <= base + hu * np.abs(ref["workers"][m]) + tiny)


@pytest.mark.parametrize("dtype_name", ["bfloat16", "float16"])
@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
@pytest.mark.parametrize("name", ["toy10", "resnet20_cifar", "resnet18_imagenet"])
def test_16bit_parity_on_workloads(grawa, name, variant, dtype_name):
    cfg = gen.CONFIGS[name]
    p, g = gen.make_inputs(cfg)
    res = run_typed(grawa, dtype_name, variant, p, g, cfg.pull, cfg.offsets())
    check(res, dtype_name, variant, cfg.pull, cfg.offsets())


@pytest.mark.parametrize("dtype_name", ["bfloat16", "float16"])
@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 8, 9, 16, 17, 33])
def test_16bit_parity_on_worker_counts_and_ragged_tables(grawa, M, dtype_name):
    cfg = gen.custom_config([7, 5001, 0, 3, 12001, 777, 8, 9, 8192, 8193], M, seed=200 + M, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    for variant in ("mgrawa", "lgrawa"):
        res = run_typed(grawa, dtype_name, variant, p, g, 0.3, cfg.offsets())
        check(res, dtype_name, variant, 0.3, cfg.offsets(), check_workers=(M > 1))
        if M == 1:
            assert np.array_equal(res["workers"][0], res["p_img"][0]) and np.array_equal(res["center"], res["p_img"][0])


@pytest.mark.parametrize("dtype_name", ["bfloat16", "float16"])
def test_16bit_unaligned_bases_and_no_centre(grawa, dtype_name):
    cfg = gen.custom_config([10, 5000, 3, 9000], 4, seed=21)
    p, g = gen.make_inputs(cfg)
    res = run_typed(grawa, dtype_name, "lgrawa", p, g, 0.5, cfg.offsets(), offset_elems=1)     # bases 2 bytes off
    check(res, dtype_name, "lgrawa", 0.5, cfg.offsets())
    res = run_typed(grawa, dtype_name, "mgrawa", p, g, 0.5, cfg.offsets(), want_center=False)
    check(res, dtype_name, "mgrawa", 0.5, cfg.offsets())


@pytest.mark.parametrize("dtype_name", ["bfloat16", "float16"])
def test_16bit_pull_extremes_are_bit_exact(grawa, dtype_name):
    cfg = gen.CONFIGS["toy10"]
    p, g = gen.make_inputs(cfg)
    r1 = run_typed(grawa, dtype_name, "lgrawa", p, g, 1.0, cfg.offsets())
    for w in r1["workers"]:
        assert np.array_equal(w, r1["center"])                   # full pull: every worker is the stored centre
    r0 = run_typed(grawa, dtype_name, "lgrawa", p, g, 0.0, cfg.offsets())
    for w, a in zip(r0["workers"], r0["p_img"]):
        assert np.array_equal(w, a)                              # no pull: untouched
    assert np.array_equal(r0["center"], r1["center"])


@pytest.mark.parametrize("dtype_name", ["bfloat16", "float16"])
@pytest.mark.parametrize("M", [5, 8, 12, 16])
def test_16bit_pull_extremes_are_bit_exact_on_the_staged_kernel(grawa, M, dtype_name):
    """5..16 workers take the kernel that stages its columns through shared memory: the same exact
    identities at pull 1 and pull 0, and the same bytes as the register kernel it replaces."""
    cfg = gen.custom_config([7, 5001, 0, 3, 12001, 777, 8, 9, 8192, 8193, 40000], M, seed=400 + M, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    r1 = run_typed(grawa, dtype_name, "lgrawa", p, g, 1.0, cfg.offsets())
    for w in r1["workers"]:
        assert np.array_equal(w, r1["center"])
    r0 = run_typed(grawa, dtype_name, "mgrawa", p, g, 0.0, cfg.offsets())
    for w, a in zip(r0["workers"], r0["p_img"]):
        assert np.array_equal(w, a)
    staged = run_typed(grawa, dtype_name, "lgrawa", p, g, 0.3, cfg.offsets())
    grawa.grawa_set_option("pull16_staged", 0)
    try:
        regs = run_typed(grawa, dtype_name, "lgrawa", p, g, 0.3, cfg.offsets())
    finally:
        grawa.grawa_set_option("pull16_staged", 1)
    assert np.array_equal(staged["center"], regs["center"])
    for u, v in zip(staged["workers"], regs["workers"]):
        assert np.array_equal(u, v)


def test_16bit_sumsq_bit_exact_on_integer_gradients(grawa):
    sizes = [10, 1000, 8192, 3, 20000, 1, 4097, 70000]
    rng = np.random.default_rng(3)
    off = np.concatenate([[0], np.cumsum(sizes)])
    g = [rng.integers(-3, 4, size=off[-1]).astype(np.float32) for _ in range(3)]
    p = [rng.normal(size=off[-1]).astype(np.float32) for _ in range(3)]
    for dtype_name in ("bfloat16", "float16"):
        res = run_typed(grawa, dtype_name, "lgrawa", p, g, 0.5, off)
        assert np.array_equal(res["S"], oracle.sumsq(g, off))


def test_typed_entry_with_float32_equals_the_plain_entry(grawa):
    import torch
    cfg = gen.CONFIGS["resnet20_cifar"]
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    xa = [torch.from_numpy(a).cuda() for a in p]
    xb = [torch.from_numpy(a).cuda() for a in p]
    gr = [torch.from_numpy(a).cuda() for a in g]
    ca, cb = torch.empty(cfg.n, device="cuda"), torch.empty(cfg.n, device="cuda")
    grawa.grawa_lgrawa_step(xa, gr, 0.5, off, ca)
    grawa.grawa_step_typed("lgrawa", xb, gr, 0.5, off, cb)
    torch.cuda.synchronize()
    assert bool((ca == cb).all()) and all(bool((u == v).all()) for u, v in zip(xa, xb))
    with pytest.raises(TypeError):
        grawa.grawa_step_typed("lgrawa", [t.double() for t in xa], gr, 0.5, off, ca)
    with pytest.raises(TypeError):
        grawa.grawa_step_typed("lgrawa", [t.half() for t in xa], gr, 0.5, off, ca)      # mixed dtypes


@pytest.mark.parametrize("dtype_name", ["bfloat16", "float16"])
@pytest.mark.parametrize("M", [17, 33, 64])
def test_16bit_many_worker_kernel_is_exact_at_the_pull_extremes_and_matches_the_scalar_kernel(grawa, M, dtype_name):
    """More than 16 workers take the run-time-M shared-memory kernel: exact identities at pull 1 and
    pull 0, and (from given norms, so that the weights are the same) the same bytes as the element-wise
    kernel that bases 2 bytes off alignment fall to."""
    cfg = gen.custom_config([7, 5001, 0, 3, 12001, 777, 8, 9, 8192, 8193, 40000], M, seed=500 + M, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    r1 = run_typed(grawa, dtype_name, "lgrawa", p, g, 1.0, cfg.offsets())
    for w in r1["workers"]:
        assert np.array_equal(w, r1["center"])
    r0 = run_typed(grawa, dtype_name, "mgrawa", p, g, 0.0, cfg.offsets())
    for w, a in zip(r0["workers"], r0["p_img"]):
        assert np.array_equal(w, a)
    vec = run_typed(grawa, dtype_name, "lgrawa", p, g, 0.3, cfg.offsets())
    check(vec, dtype_name, "lgrawa", 0.3, cfg.offsets())
    # same given norms, hence the same weights, through the vector kernel and (bases 2 bytes off) the element-wise one
    import torch
    dt = getattr(torch, dtype_name)
    K = len(cfg.offsets()) - 1
    norms = torch.from_numpy(np.random.default_rng(M).uniform(0.5, 2.0, size=(K, M))).cuda()
    got = []
    for shift in (0, 1):
        xs = []
        for a in p:
            t = torch.zeros(a.size + shift, dtype=dt, device="cuda")
            t[shift:] = torch.from_numpy(a).cuda().to(dt)
            xs.append(t[shift:])
        c = torch.zeros(xs[0].numel() + shift, dtype=dt, device="cuda")[shift:]
        grawa.grawa_step_from_layer_norms_typed("lgrawa", xs, norms, 0.3, cfg.offsets(), c)
        assert grawa.grawa_last_step_status() == 0
        got.append([c.float().cpu().numpy()] + [t.float().cpu().numpy() for t in xs])
    for u, v in zip(*got):
        assert np.array_equal(u, v)


def test_16bit_resnet18_table_with_32_workers_full_size(grawa):
    """The many-worker case the benchmark times on bfloat16 storage, element by element against the oracle."""
    base = gen.CONFIGS["resnet18_imagenet"]
    cfg = gen.custom_config(np.diff(base.offsets()), 32, seed=base.seed, pull=base.pull, grad_recipe=base.grad_recipe,
                            log10_sigma=base.log10_sigma, loud_worker_factor=base.loud_worker_factor)
    p, g = gen.make_inputs(cfg)
    res = run_typed(grawa, "bfloat16", "lgrawa", p, g, cfg.pull, cfg.offsets())
    del p, g
    check(res, "bfloat16", "lgrawa", cfg.pull, cfg.offsets())


@pytest.mark.parametrize("case", range(24))
def test_16bit_parity_on_seeded_random_tables(grawa, case):
    """The same kind of random tables on 16-bit storage, across the register, staged and run-time-M kernels."""
    rng = np.random.default_rng(7000 + case)
    K = int(rng.integers(1, 12))
    kinds = rng.integers(0, 5, size=K)
    sizes = [int({0: 0, 1: rng.integers(1, 17), 2: rng.integers(17, 3000), 3: 8 * rng.integers(256, 5000),
                  4: rng.integers(20000, 70000)}[int(k)]) for k in kinds]
    if sum(sizes) == 0:
        sizes[-1] = 4321
    M = int(rng.choice([2, 3, 4, 5, 8, 11, 16, 17, 25, 48, 64]))
    dtype_name = ["bfloat16", "float16"][case % 2]
    variant = ["lgrawa", "mgrawa", "grawa"][case % 3]
    pull = float(rng.choice([0.2, 0.5, 0.8]))
    cfg = gen.custom_config(sizes, M, seed=7000 + case, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    res = run_typed(grawa, dtype_name, variant, p, g, pull, cfg.offsets(), offset_elems=(8 if case % 4 == 3 else 0))
    check(res, dtype_name, variant, pull, cfg.offsets())


@pytest.mark.parametrize("dtype_name", ["bfloat16", "float16"])
@pytest.mark.parametrize("M", [2, 3, 4])
def test_16bit_32_byte_and_16_byte_columns_agree_bit_for_bit(grawa, M, dtype_name):
    """Up to 4 workers: bases aligned to 32 bytes take 32-byte columns, bases 16 bytes into their
    allocation the 16-byte ones; same arithmetic, same bytes out, both against the oracle."""
    cfg = gen.custom_config([7, 5001, 0, 3, 12001, 777, 8, 9, 8192, 8193, 40000, 16, 17], M, seed=900 + M, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    for variant in ("lgrawa", "mgrawa"):
        wide = run_typed(grawa, dtype_name, variant, p, g, 0.3, cfg.offsets())
        check(wide, dtype_name, variant, 0.3, cfg.offsets())
        narrow = run_typed(grawa, dtype_name, variant, p, g, 0.3, cfg.offsets(), offset_elems=8)
        check(narrow, dtype_name, variant, 0.3, cfg.offsets())
        assert np.array_equal(wide["center"], narrow["center"])
        for u, v in zip(wide["workers"], narrow["workers"]):
            assert np.array_equal(u, v)


@pytest.mark.parametrize("name", ["vgg16", "vit_b16"])
def test_16bit_parity_large_workloads_full_size(grawa, name):
    """bfloat16 LGRAWA on the two largest workloads at full size, element by element against the oracle
    run on the fp32 images of the rounded inputs (comparison in chunks, as for fp32 storage)."""
    import torch
    from gpu_util import compare_with_oracle
    cfg = gen.CONFIGS[name]
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    x, gr = [], []
    for m in range(cfg.M):                                      # round to storage; the oracle sees what the GPU sees
        t = torch.from_numpy(p[m]).cuda().bfloat16()
        p[m][:] = t.float().cpu().numpy()
        x.append(t)
        t = torch.from_numpy(g[m]).cuda().bfloat16()
        g[m][:] = t.float().cpu().numpy()
        gr.append(t)
    K, M = cfg.K, cfg.M
    beta = torch.empty(K * M, device="cuda")
    scores = torch.empty(K * M, dtype=torch.float64, device="cuda")
    sumsq = torch.empty(K * M, dtype=torch.float64, device="cuda")
    center = torch.zeros(cfg.n, dtype=torch.bfloat16, device="cuda")
    grawa.grawa_step_typed("lgrawa", x, gr, cfg.pull, off, center, weights_out=beta, scores_out=scores, sumsq_out=sumsq)
    assert grawa.grawa_last_step_status() == 0
    res = {"workers": x, "center": center, "beta": beta.cpu().numpy().reshape(K, M), "A": scores.cpu().numpy().reshape(K, M),
           "S": sumsq.cpu().numpy().reshape(K, M)}
    stats = compare_with_oracle(res, "lgrawa", p, g, cfg.pull, off, half_ulp=HALF_ULP["bfloat16"])
    print(name, "bfloat16 lgrawa", stats)
