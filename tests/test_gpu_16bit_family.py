"""GPU parity of the other entry points on 16-bit storage: the proximity step, per-layer norms and sums
of squares, the step from given norms / sums (Local variants, element-range shards) and the host-buffer
step.  Inputs are rounded to the storage type first; the oracle runs on their fp32 images; the bound on
stored values is the fp32 bound of the parity contract plus half a unit in the last place of the
storage type at the oracle's value.  Also: the caller-owned status word of the options."""
import numpy as np
import pytest

import gen
import oracle
from gpu_util import TOL_BETA_REL, TOL_S_REL, TOL_X_ABS_FACTOR

pytestmark = pytest.mark.gpu

HALF_ULP = {"bfloat16": 2.0 ** -8, "float16": 2.0 ** -11}
TINY = {"bfloat16": 0.0, "float16": 2.0 ** -25}
DTYPES = ["bfloat16", "float16"]


@pytest.fixture(scope="module")
def grawa():
    import paper_2403_04206_b200 as g
    g.library()
    return g


def to_dev(arrs, dtype_name):
    import torch
    dt = getattr(torch, dtype_name)
    return [torch.from_numpy(a).cuda().to(dt) for a in arrs]


def images(tensors):
    return [t.float().cpu().numpy() for t in tensors]


def close16(got, want, base, dtype_name):
    return np.all(np.abs(got - want) <= base + HALF_ULP[dtype_name] * np.abs(want) + TINY[dtype_name])


@pytest.mark.parametrize("dtype_name", DTYPES)
@pytest.mark.parametrize("M", [1, 3, 4, 9])
def test_prox_step_typed_parity(grawa, M, dtype_name):
    import torch
    rng = np.random.default_rng(40 + M)
    n = 100_003
    x = to_dev([rng.normal(size=n).astype(np.float32) for _ in range(M)], dtype_name)
    c = to_dev([rng.normal(size=n).astype(np.float32)], dtype_name)[0]
    x_img, c_img = images(x), images([c])[0]
    a = 0.05 / 16
    grawa.grawa_prox_step_typed(x, c, a)
    torch.cuda.synchronize()
    ref = oracle.prox(x_img, c_img, a)
    base = TOL_X_ABS_FACTOR * max(float(np.abs(v).max()) for v in x_img)
    for got, want in zip(images(x), ref):
        assert close16(got, want, base, dtype_name)
    # the extremes are exact: a = 0 leaves the bits alone, a = 1 copies the centre
    before = [t.clone() for t in x]
    grawa.grawa_prox_step_typed(x, c, 0.0)
    torch.cuda.synchronize()
    assert all(bool((u.view(torch.int16) == v.view(torch.int16)).all()) for u, v in zip(x, before))
    grawa.grawa_prox_step_typed(x, c, 1.0)
    torch.cuda.synchronize()
    assert all(bool((u.view(torch.int16) == c.view(torch.int16)).all()) for u in x)


@pytest.mark.parametrize("dtype_name", DTYPES)
def test_prox_step_typed_unaligned_and_float32(grawa, dtype_name):
    import torch
    rng = np.random.default_rng(7)
    n = 10_001
    dt = getattr(torch, dtype_name)
    store = [torch.zeros(n + 3, dtype=dt, device="cuda") for _ in range(3)]
    x = [s[1 + i:1 + i + n] for i, s in enumerate(store)]                 # bases 2, 4, 6 bytes off
    for t in x:
        t.copy_(torch.from_numpy(rng.normal(size=n).astype(np.float32)).cuda().to(dt))
    c = to_dev([rng.normal(size=n).astype(np.float32)], dtype_name)[0]
    x_img, c_img = images(x), images([c])[0]
    grawa.grawa_prox_step_typed(x, c, 0.25)
    torch.cuda.synchronize()
    ref = oracle.prox(x_img, c_img, 0.25)
    base = TOL_X_ABS_FACTOR * max(float(np.abs(v).max()) for v in x_img)
    for got, want in zip(images(x), ref):
        assert close16(got, want, base, dtype_name)
    # float32 through the typed call is the plain call
    a32 = [torch.from_numpy(v).cuda() for v in x_img]
    b32 = [t.clone() for t in a32]
    c32 = torch.from_numpy(c_img).cuda()
    grawa.grawa_prox_step_typed(a32, c32, 0.25)
    grawa.grawa_prox_step(b32, c32, 0.25)
    torch.cuda.synchronize()
    assert all(bool((u == v).all()) for u, v in zip(a32, b32))


@pytest.mark.parametrize("dtype_name", DTYPES)
def test_layer_norms_and_sumsq_typed(grawa, dtype_name):
    import torch
    cfg = gen.custom_config([7, 5001, 0, 3, 120001, 777, 8, 8193], 5, seed=300, log10_sigma=(-2.0, 0.0))
    _, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    gd = to_dev(g, dtype_name)
    g_img = images(gd)
    S = oracle.sumsq(g_img, off)
    out = torch.full((cfg.K, cfg.M), -1.0, dtype=torch.float64, device="cuda")
    grawa.grawa_layer_sumsq_typed(gd, off, out)
    torch.cuda.synchronize()
    assert np.allclose(out.cpu().numpy(), S, rtol=TOL_S_REL, atol=0)
    norms = torch.full((cfg.K,), -1.0, dtype=torch.float64, device="cuda")
    grawa.grawa_layer_norms_typed(gd[2], off, norms)
    torch.cuda.synchronize()
    assert np.allclose(norms.cpu().numpy(), np.sqrt(S[:, 2]), rtol=TOL_S_REL, atol=0)
    # exact on integer-valued gradients
    gi = [np.random.default_rng(m).integers(-3, 4, size=cfg.n).astype(np.float32) for m in range(cfg.M)]
    grawa.grawa_layer_sumsq_typed(to_dev(gi, dtype_name), off, out)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), oracle.sumsq(gi, off))


@pytest.mark.parametrize("dtype_name", DTYPES)
@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
def test_step_from_layer_norms_and_sums_typed(grawa, variant, dtype_name):
    import torch
    cfg = gen.custom_config([10, 50000, 0, 3, 120001, 777], 5, seed=92, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    K, M = cfg.K, cfg.M
    G = K if variant == "lgrawa" else 1
    rng = np.random.default_rng(5)
    # given norms (the running estimates of the Local variants)
    norms = 10.0 ** rng.uniform(-2, 1, size=(K, M))
    x = to_dev(p, dtype_name)
    p_img = images(x)
    center = torch.zeros(cfg.n, dtype=x[0].dtype, device="cuda")
    beta = torch.empty(G * M, device="cuda")
    grawa.grawa_step_from_layer_norms_typed(variant, x, torch.from_numpy(norms).cuda(), 0.4, off, center, weights_out=beta)
    torch.cuda.synchronize()
    ref_beta, _ = oracle.weights(oracle.scores_from_norms(norms, variant))
    assert np.abs(beta.cpu().numpy() / ref_beta.ravel() - 1).max() <= TOL_BETA_REL
    c_ref, w_ref = oracle.center_pull(p_img, ref_beta, 0.4, off)
    base = TOL_X_ABS_FACTOR * max(float(np.abs(a).max()) for a in p_img)
    assert close16(center.float().cpu().numpy(), c_ref, base, dtype_name)
    for got, want in zip(images(x), w_ref):
        assert close16(got, want, base, dtype_name)
    # given sums of squares in three parts (element-range shards), added in part order
    gd = to_dev(g, dtype_name)
    S = oracle.sumsq(images(gd), off)
    parts = rng.dirichlet([1.0, 1.0, 1.0], size=(K, M)).transpose(2, 0, 1) * S[None]      # [3, K, M], sums to S
    x = to_dev(p, dtype_name)
    grawa.grawa_step_from_layer_sums_typed(variant, x, torch.from_numpy(np.ascontiguousarray(parts)).cuda(), 3, 0.4, off,
                                           center, weights_out=beta)
    torch.cuda.synchronize()
    ref_beta, _ = oracle.weights(oracle.scores(parts[0] + parts[1] + parts[2], variant))
    nz = ref_beta.ravel() != 0
    assert np.abs(beta.cpu().numpy()[nz] / ref_beta.ravel()[nz] - 1).max() <= TOL_BETA_REL
    c_ref, w_ref = oracle.center_pull(p_img, ref_beta, 0.4, off)
    assert close16(center.float().cpu().numpy(), c_ref, base, dtype_name)
    for got, want in zip(images(x), w_ref):
        assert close16(got, want, base, dtype_name)


@pytest.mark.parametrize("dtype_name", DTYPES)
@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
def test_host_buffer_step_typed_equals_the_device_step(grawa, variant, dtype_name):
    import torch
    cfg = gen.custom_config([10, 3_000_001, 0, 3, 1_200_001, 777], 5, seed=93, log10_sigma=(-2.0, 0.0))
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    dt = getattr(torch, dtype_name)
    hp = [torch.from_numpy(a).to(dt).pin_memory() for a in p]
    hg = [torch.from_numpy(a).to(dt).pin_memory() for a in g]
    hc = torch.zeros(cfg.n, dtype=dt).pin_memory()
    x, gr = [t.cuda() for t in hp], [t.cuda() for t in hg]
    center = torch.zeros(cfg.n, dtype=dt, device="cuda")
    grawa.grawa_step_typed(variant, x, gr, 0.5, off, center)
    grawa.grawa_step_host_typed(variant, hp, hg, 0.5, off, hc)
    torch.cuda.synchronize()
    assert bool((hc.view(torch.int16) == center.cpu().view(torch.int16)).all())
    for u, v in zip(hp, x):
        assert bool((u.view(torch.int16) == v.cpu().view(torch.int16)).all())


def test_caller_owned_status_word(grawa):
    """A device int named in the options receives the step's status without a host synchronisation
    of the library's own: 0 after a clean step, bit 0 after a step that met a non-finite score."""
    import torch
    cfg = gen.custom_config([100, 5000, 64], 4, seed=13)
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    word = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    for variant, fn in (("lgrawa", grawa.grawa_lgrawa_step), ("mgrawa", grawa.grawa_mgrawa_step)):
        x = [torch.from_numpy(a).cuda() for a in p]
        fn(x, [torch.from_numpy(a).cuda() for a in g], 0.5, off, None, status_word=word)
        torch.cuda.synchronize()
        assert int(word.item()) == 0
        bad = [a.copy() for a in g]
        bad[1][off[1] + 3] = np.nan
        fn(x, [torch.from_numpy(a).cuda() for a in bad], 0.5, off, None, status_word=word)
        torch.cuda.synchronize()
        assert int(word.item()) == 1 and grawa.grawa_last_step_status() == -3
        word.fill_(77)
