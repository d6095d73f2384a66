"""GPU parity of the Local-variant building blocks: per-layer norms of one worker, the running
norm estimate, and the averaging step driven by given layer norms instead of gradients."""
import numpy as np
import pytest

import gen
import oracle
from gpu_util import TOL_BETA_REL, TOL_S_REL, TOL_X_ABS_FACTOR, gpu_step, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def grawa():
    import paper_2403_04206_b200 as g
    g.library()
    return g


@pytest.mark.parametrize("sizes", [[10, 5000, 0, 3, 120001, 777], [1], [8192, 8193], [20_000_003, 5]],
                         ids=lambda s: "-".join(map(str, s)))
def test_layer_norms_of_one_worker(grawa, sizes):
    import torch
    cfg = gen.custom_config(sizes, 1, seed=61, log10_sigma=(-2.0, 0.0))
    _, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    out = torch.full((cfg.K,), -1.0, dtype=torch.float64, device="cuda")
    grawa.grawa_layer_norms(torch.from_numpy(g[0]).cuda(), off, out)
    torch.cuda.synchronize()
    want = np.sqrt(oracle.sumsq(g, off))[:, 0]
    got = out.cpu().numpy()
    assert np.array_equal(got[want == 0], want[want == 0])
    nz = want != 0
    assert np.abs(got[nz] / want[nz] - 1).max() <= TOL_S_REL
    # without a layer table: the flat norm
    flat = torch.zeros(1, dtype=torch.float64, device="cuda")
    grawa.grawa_layer_norms(torch.from_numpy(g[0]).cuda(), None, flat)
    torch.cuda.synchronize()
    assert abs(flat.item() / np.sqrt(oracle.sumsq(g)[0, 0]) - 1) <= TOL_S_REL


def test_norm_ema_matches_the_oracle_step_by_step(grawa):
    import torch
    K, gamma = 300, 0.9
    rng = np.random.default_rng(5)
    mvg_ref = np.zeros(K)
    mvg = torch.zeros(K, dtype=torch.float64, device="cuda")
    est = torch.zeros(K, dtype=torch.float64, device="cuda")
    for t in range(1, 7):
        cur = rng.uniform(0.1, 3.0, size=K)
        est_ref = oracle.norm_ema(mvg_ref, cur, gamma, t)
        grawa.grawa_norm_ema(mvg, torch.from_numpy(cur).cuda(), gamma, t, est)
        torch.cuda.synchronize()
        assert np.allclose(mvg.cpu().numpy(), mvg_ref, rtol=1e-14, atol=0)
        assert np.allclose(est.cpu().numpy(), est_ref, rtol=1e-14, atol=0)
    with pytest.raises(grawa.GrawaError):
        grawa.grawa_norm_ema(mvg, est, 1.0, 1, est)          # gamma must be below 1
    with pytest.raises(grawa.GrawaError):
        grawa.grawa_norm_ema(mvg, est, 0.5, 0, est)          # t counts from 1


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
@pytest.mark.parametrize("M", [1, 4, 16, 20])
def test_step_from_layer_norms_parity(grawa, variant, M):
    import torch
    cfg = gen.custom_config([10, 50000, 0, 3, 120001, 777], M, seed=70 + M, log10_sigma=(-2.0, 0.0))
    p, _ = gen.make_inputs(cfg)
    off = cfg.offsets()
    rng = np.random.default_rng(M)
    norms = 10.0 ** rng.uniform(-3, 1, size=(cfg.K, M))
    norms[2] = 0.0                                            # the empty layer
    x = to_device(p)
    center = torch.empty(cfg.n, device="cuda")
    G = cfg.K if variant == "lgrawa" else 1
    beta = torch.empty(G * M, device="cuda")
    grawa.grawa_step_from_layer_norms(variant, x, torch.from_numpy(norms).cuda(), 0.5, off, center, weights_out=beta)
    assert grawa.grawa_last_step_status() == 0
    A = oracle.scores_from_norms(norms, variant)
    beta_ref, _ = oracle.weights(A)
    got_beta = beta.cpu().numpy().reshape(beta_ref.shape)
    assert np.abs(got_beta / beta_ref - 1).max() <= TOL_BETA_REL
    c_ref, w_ref = oracle.center_pull(p, beta_ref, 0.5, off, want_workers=(M > 1))
    tol = TOL_X_ABS_FACTOR * max(float(np.abs(a).max()) for a in p)
    assert np.abs(center.cpu().numpy() - c_ref).max() <= tol
    if M > 1:
        for m in range(M):
            assert np.abs(x[m].cpu().numpy() - w_ref[m]).max() <= tol
    else:
        assert np.array_equal(x[0].cpu().numpy(), p[0])


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa", "grawa"])
@pytest.mark.parametrize("M", [3, 64])
def test_step_from_layer_norms_with_thousands_of_layers(grawa, variant, M):
    """3000 layers: the finalisation runs as several CTAs (rows shared out and a last CTA that adds the
    terms; with per-layer weights a warp per layer and status words cleared in front of the launch).
    Twice in a row, the second time with a non-finite norm: the status says so and the next step is clean."""
    import torch
    rng = np.random.default_rng(M)
    sizes = [int(v) for v in rng.integers(0, 41, size=3000)]
    cfg = gen.custom_config(sizes, M, seed=170 + M, log10_sigma=(-2.0, 0.0))
    p, _ = gen.make_inputs(cfg)
    off = cfg.offsets()
    norms = 10.0 ** rng.uniform(-3, 1, size=(cfg.K, M))
    norms[np.diff(off) == 0] = 0.0
    A = oracle.scores_from_norms(norms, variant)
    beta_ref, _ = oracle.weights(A)
    G = cfg.K if variant == "lgrawa" else 1
    tol = TOL_X_ABS_FACTOR * max(float(np.abs(a).max()) for a in p)
    word = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    for trial in range(3):
        given = norms.copy()
        if trial == 1:
            given[1234, 1] = np.inf
        x = to_device(p)
        center = torch.empty(cfg.n, device="cuda")
        beta = torch.empty(G * M, device="cuda")
        grawa.grawa_step_from_layer_norms(variant, x, torch.from_numpy(given).cuda(), 0.5, off, center, weights_out=beta,
                                          status_word=word)
        status = grawa.grawa_last_step_status()
        if trial == 1:
            assert status == -3 and word.item() != 0            # GRAWA_ERR_NONFINITE
            continue
        assert status == 0 and word.item() == 0
        got_beta = beta.cpu().numpy().reshape(beta_ref.shape)
        nz = beta_ref != 0
        assert np.abs(got_beta[nz] / beta_ref[nz] - 1).max() <= TOL_BETA_REL
        c_ref, w_ref = oracle.center_pull(p, beta_ref, 0.5, off, want_workers=True)
        assert np.abs(center.cpu().numpy() - c_ref).max() <= tol
        for m in range(M):
            assert np.abs(x[m].cpu().numpy() - w_ref[m]).max() <= tol


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
def test_norms_then_step_equals_the_gradient_step_bit_for_bit(grawa, variant):
    """Layer norms taken worker by worker and fed back give exactly the step that reads the gradients."""
    import torch
    cfg = gen.CONFIGS["resnet20_cifar"]
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    ref = gpu_step(grawa, variant, p, g, 0.5, off)
    norms = torch.zeros(cfg.K, cfg.M, dtype=torch.float64, device="cuda")
    col = torch.zeros(cfg.K, dtype=torch.float64, device="cuda")
    for m in range(cfg.M):
        grawa.grawa_layer_norms(ref["grads"][m], off, col)
        norms[:, m] = col
    x = to_device(p)
    center = torch.empty(cfg.n, device="cuda")
    grawa.grawa_step_from_layer_norms(variant, x, norms, 0.5, off, center)
    torch.cuda.synchronize()
    assert bool((center == ref["center"]).all())
    for u, v in zip(x, ref["workers"]):
        assert bool((u == v).all())


def test_from_norms_argument_checks(grawa):
    import torch
    x = [torch.zeros(100, device="cuda") for _ in range(2)]
    with pytest.raises(grawa.GrawaError):
        grawa.grawa_step_from_layer_norms("lgrawa", x, None, 0.5, [0, 50, 100])     # no norms
    with pytest.raises(grawa.GrawaError):
        grawa.grawa_step_from_layer_norms(5, x, torch.ones(4, dtype=torch.float64, device="cuda"), 0.5, [0, 50, 100])
