"""Pins of the CPU oracle against what the paper and the mathematics fix:
hand cases (tests/golden/hand_cases.txt), closed forms, invariants, special cases
that reduce to library routines, and an independent vectorised statement.
None of these tests touches the CUDA library.
"""
import itertools
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.txt")


def load_cases():
    cases, cur = {}, None
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if not line:
            continue
        if line.startswith("[case"):
            cur = cases.setdefault(line[5:-1].strip(), {})
            continue
        key, val = line.split(":")
        layers = [np.array([float(t) for t in part.split()]) for part in val.split("|")]
        cur[key.strip()] = layers if len(layers) > 1 else layers[0]
    return cases


CASES = load_cases()
rng = np.random.default_rng(1234)


def f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


# ---------------------------------------------------------------- hand cases

def test_hand_case_two_workers_two_layers():
    c = CASES["two_workers_two_layers"]
    g = [f32(np.concatenate(c["g1"])), f32(np.concatenate(c["g2"]))]
    off = np.array([0, 2, 4])
    S = oracle.sumsq(g, off)
    assert np.array_equal(S[0], c["sumsq_layer1"]) and np.array_equal(S[1], c["sumsq_layer2"])
    A_m = oracle.scores(S, "mgrawa")
    assert np.array_equal(A_m, c["mgrawa_scores"])
    assert np.allclose(oracle.weights(A_m)[0], c["mgrawa_beta"], rtol=0, atol=1e-15)
    A_g = oracle.scores(S, "grawa")
    assert np.allclose(A_g ** 2, c["grawa_scores_squared"], rtol=1e-15)
    assert np.allclose(oracle.weights(A_g)[0], c["grawa_beta"], rtol=0, atol=5e-9)
    beta_l = oracle.weights(oracle.scores(S, "lgrawa"))[0]
    assert np.allclose(beta_l[0], c["lgrawa_beta_layer1"], rtol=0, atol=1e-15)
    assert np.allclose(beta_l[1], c["lgrawa_beta_layer2"], rtol=0, atol=1e-15)
    # the three variants really differ on this case
    assert abs(oracle.weights(A_g)[0][0] - 0.6) > 1e-3 and abs(beta_l[1][0] - 0.6) > 1e-2


def test_hand_case_centre_and_pull():
    c = CASES["centre_and_pull"]
    r = oracle.step([f32(c["x1"]), f32(c["x2"])], [f32(c["g1"]), f32(c["g2"])], float(c["pull"][0]), "mgrawa")
    assert np.allclose(r["beta"], c["beta"], atol=1e-15)
    assert np.allclose(r["center"], c["centre"], atol=1e-14)
    assert np.allclose(r["workers"][0], c["x1_new"], atol=1e-14)
    assert np.allclose(r["workers"][1], c["x2_new"], atol=1e-14)


def test_hand_case_three_workers():
    c = CASES["three_workers"]
    beta, flagged = oracle.weights(c["scores"])
    assert not flagged and np.allclose(beta, c["beta"], atol=1e-16)


# ---------------------------------------------------------------- weights

@pytest.mark.parametrize("M", [1, 2, 3, 4, 8])
def test_weights_equal_product_form(M):
    """Eq. 2's closed form beta_m = Theta/||.||, Theta = prod / sum_i (prod/||.||_i)."""
    A = rng.uniform(0.1, 10.0, size=M)
    prod = np.prod(A)
    theta = prod / sum(prod / A[i] for i in range(M))
    beta, _ = oracle.weights(A)
    assert np.allclose(beta, theta / A, rtol=1e-13)
    # consequence used in the convergence proof: beta_i <= 1  =>  Theta <= every norm
    assert theta <= A.min() * (1 + 1e-15)


def test_weights_two_workers_closed_form():
    A = np.array([0.37, 4.2])
    beta, _ = oracle.weights(A)
    assert np.allclose(beta, [A[1] / A.sum(), A[0] / A.sum()], rtol=1e-15)


@pytest.mark.parametrize("M", [2, 5, 12, 16, 64])
def test_weights_sum_to_one_and_in_unit_interval(M):
    A = 10.0 ** rng.uniform(-4, 2, size=(7, M))
    beta, _ = oracle.weights(A)
    assert np.allclose(beta.sum(axis=1), 1.0, atol=1e-15)
    assert np.all(beta >= 0) and np.all(beta <= 1)
    assert abs(beta.sum() - 7) < 1e-13           # LGRAWA: sum over layers and workers = K
    # inverse proportionality: beta_a / beta_b = A_b / A_a
    assert np.allclose(beta[:, 0] / beta[:, 1], A[:, 1] / A[:, 0], rtol=1e-13)
    # ordering: smaller score, larger weight
    assert np.array_equal(np.argsort(A[0]), np.argsort(-beta[0]))


def test_weights_scale_invariant_and_permutation_equivariant():
    A = rng.uniform(0.5, 3.0, size=6)
    beta, _ = oracle.weights(A)
    assert np.allclose(oracle.weights(A * 128.0)[0], beta, rtol=1e-15)   # N-sample sum vs mean does not matter
    p = rng.permutation(6)
    assert np.array_equal(oracle.weights(A[p])[0], beta[p])


def test_weights_zero_score_policy():
    assert np.array_equal(oracle.weights(np.array([2.0, 0.0, 5.0]))[0], [0, 1, 0])
    assert np.array_equal(oracle.weights(np.array([0.0, 0.0, 5.0, 1.0]))[0], [0.5, 0.5, 0, 0])
    assert np.array_equal(oracle.weights(np.zeros(4))[0], [0.25] * 4)
    # limit reading: a tiny score behaves like the zero one
    assert np.allclose(oracle.weights(np.array([2.0, 1e-300, 5.0]))[0], [0, 1, 0], atol=1e-299)


def test_weights_nonfinite_policy():
    beta, flagged = oracle.weights(np.array([1.0, np.nan, 1.0, np.inf]))
    assert flagged and np.array_equal(beta, [0.5, 0, 0.5, 0])
    beta, flagged = oracle.weights(np.array([np.nan, np.inf]))
    assert flagged and np.array_equal(beta, [0.5, 0.5])
    beta, flagged = oracle.weights(np.array([[1.0, 3.0], [np.nan, 2.0]]))
    assert flagged and np.allclose(beta, [[0.75, 0.25], [0, 1]])
    assert not oracle.weights(np.array([1.0, 2.0]))[1]


# ---------------------------------------------------------------- scores / sum of squares

def test_sumsq_against_library_norm():
    sizes = [5, 0, 17, 1, 300]
    off = np.concatenate([[0], np.cumsum(sizes)])
    g = [f32(rng.normal(size=off[-1])) for _ in range(3)]
    S = oracle.sumsq(g, off)
    for k in range(len(sizes)):
        for m in range(3):
            seg = g[m][off[k]:off[k + 1]].astype(np.float64)
            assert math.isclose(S[k, m], np.linalg.norm(seg) ** 2, rel_tol=1e-13, abs_tol=0)
    assert np.all(S[1] == 0)
    A_l = oracle.scores(S, "lgrawa")
    A_m = oracle.scores(S, "mgrawa")
    A_g = oracle.scores(S, "grawa")
    for m in range(3):
        norms = [np.linalg.norm(g[m][off[k]:off[k + 1]].astype(np.float64)) for k in range(len(sizes))]
        assert np.allclose(A_l[:, m], norms, rtol=1e-13)
        assert math.isclose(A_m[m], sum(norms), rel_tol=1e-13)
        assert math.isclose(A_g[m], np.linalg.norm(g[m].astype(np.float64)), rel_tol=1e-13)
        # triangle inequality: the sum of layer norms dominates the flat norm (motivation of MGRAWA)
        assert A_m[m] > A_g[m]


def test_sumsq_indexing_is_exact():
    """A single 1 placed at a layer's first/last element must land in that layer and only there."""
    sizes = [3, 1, 0, 6, 2, 5]
    off = np.concatenate([[0], np.cumsum(sizes)])
    n, K = off[-1], len(sizes)
    for k in range(K):
        for pos in {off[k], off[k + 1] - 1} if sizes[k] else set():
            g = np.zeros(n, dtype=np.float32)
            g[pos] = 1.0
            S = oracle.sumsq([g, 2 * g], off)
            expect = np.zeros((K, 2)); expect[k] = [1, 4]
            assert np.array_equal(S, expect)
    # layer-constant integer gradients: S = n_k c_k^2 exactly
    g = np.concatenate([np.full(s, k + 1, dtype=np.float32) for k, s in enumerate(sizes)])
    assert np.array_equal(oracle.sumsq([g], off)[:, 0], [s * (k + 1) ** 2 for k, s in enumerate(sizes)])


def test_variants_coincide_for_one_layer_and_differ_otherwise():
    g = [f32(rng.normal(size=50) * s) for s in (0.1, 1.0, 3.0)]
    x = [f32(rng.normal(size=50)) for _ in range(3)]
    one = [oracle.step(x, g, 0.3, v) for v in ("grawa", "mgrawa", "lgrawa")]
    assert np.array_equal(one[0]["center"], one[1]["center"]) and np.array_equal(one[0]["center"], one[2]["center"])
    assert np.array_equal(one[1]["beta"], one[2]["beta"][0])
    off = np.array([0, 10, 50])
    g[0][:10] *= 40.0                      # worker 0 is loud in layer 0 only
    many = [oracle.step(x, g, 0.3, v, off) for v in ("grawa", "mgrawa", "lgrawa")]
    assert not np.allclose(many[0]["beta"], many[1]["beta"], rtol=1e-3)
    assert not np.allclose(many[1]["center"], many[2]["center"], rtol=1e-3)


# ---------------------------------------------------------------- centre and pull

def _random_problem(M, sizes, scale=None):
    off = np.concatenate([[0], np.cumsum(sizes)])
    n = off[-1]
    x = [f32(rng.normal(size=n)) for _ in range(M)]
    g = [f32(rng.normal(size=n) * (scale[m] if scale is not None else 1.0)) for m in range(M)]
    return x, g, off


def numpy_statement(x, g, off, pull, variant):
    """Second, independent few-line float64 statement of the five steps."""
    X, G = np.stack(x).astype(np.float64), np.stack(g).astype(np.float64)
    K = len(off) - 1
    lay = np.repeat(np.arange(K), np.diff(off))                       # layer of each element
    onehot = (lay[None, :] == np.arange(K)[:, None]).astype(np.float64)  # [K, n]
    S = onehot @ (G * G).T                                            # [K, M]
    if variant == "lgrawa":
        A = np.sqrt(S)
        beta = (1 / A) / (1 / A).sum(axis=1, keepdims=True)
        B = beta[lay].T                                               # [M, n]
    else:
        A = np.sqrt(S).sum(axis=0) if variant == "mgrawa" else np.sqrt(S.sum(axis=0))
        beta = (1 / A) / (1 / A).sum()
        B = np.repeat(beta[:, None], X.shape[1], axis=1)
    c = (B * X).sum(axis=0)
    return S, beta, c, (1 - pull) * X + pull * c[None, :]


@pytest.mark.parametrize("variant", ["grawa", "mgrawa", "lgrawa"])
@pytest.mark.parametrize("M,sizes", [(2, [4]), (3, [1, 7, 2]), (5, [6, 3, 11, 1, 9]), (16, [13, 8])])
def test_step_against_independent_numpy_statement(variant, M, sizes):
    x, g, off = _random_problem(M, sizes, scale=10.0 ** rng.uniform(-2, 1, size=M))
    r = oracle.step(x, g, 0.7, variant, off)
    S, beta, c, xn = numpy_statement(x, g, off, 0.7, variant)
    assert np.allclose(r["S"], S, rtol=1e-13)
    assert np.allclose(r["beta"], beta, rtol=1e-12)
    assert np.allclose(r["center"], c, rtol=1e-12, atol=1e-14)
    assert np.allclose(np.stack(r["workers"]), xn, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("variant", ["grawa", "mgrawa", "lgrawa"])
@pytest.mark.parametrize("sizes", [[4, 0, 9, 2, 0], [0, 0, 3, 0, 5], [0, 7], [3, 0, 0, 0, 1, 0], [2, 0, 2, 0, 2]])
def test_empty_layers_against_independent_numpy_statement(variant, sizes):
    """Layer tables with zero-size layers (first, last, several in a row): the element -> layer
    lookup must skip them.  Every layer gets its own per-worker gradient scales, so the weights of
    neighbouring layers differ by orders of magnitude and a lookup that lands one row off (the empty
    layer's row, or the previous non-empty one) moves the centre far outside the tolerance."""
    M = 5
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    n, K = int(off[-1]), len(sizes)
    x = [f32(rng.normal(size=n) + 3.0 * m) for m in range(M)]
    g = [f32(rng.normal(size=n)) for _ in range(M)]
    for k in range(K):
        scales = 10.0 ** np.roll(np.array([-2.0, -1.0, 0.0, 1.0, 2.0]), k)  # which worker is quiet rotates with k
        for m in range(M):
            g[m][off[k]:off[k + 1]] *= np.float32(scales[m])
    r = oracle.step(x, g, 0.6, variant, off)
    with np.errstate(divide="ignore", invalid="ignore"):
        S, beta, c, xn = numpy_statement(x, g, off, 0.6, variant)
    full = np.diff(off) > 0
    assert np.allclose(r["S"][full], S[full], rtol=1e-13) and np.all(r["S"][~full] == 0)
    if variant == "lgrawa":
        assert np.allclose(r["beta"][full], beta[full], rtol=1e-12)
        b = r["beta"][full]
        for a in range(len(b) - 1):
            assert np.abs(b[a] - b[a + 1]).max() > 0.3   # consecutive non-empty layers have very different weights
    else:
        assert np.allclose(r["beta"], beta, rtol=1e-12)
    assert np.allclose(r["center"], c, rtol=1e-12, atol=1e-14)
    assert np.allclose(np.stack(r["workers"]), xn, rtol=1e-12, atol=1e-14)
    # the ranged call, started at every element (so the lookup begins in front of, on and after
    # each run of empty layers), against the numpy statement rather than the oracle's own whole call
    for j0 in range(n):
        cj, wj = oracle.center_pull(x, r["beta"], 0.6, off, j0, n)
        assert np.allclose(cj, c[j0:], rtol=1e-12, atol=1e-14)
        assert np.allclose(np.stack(wj), xn[:, j0:], rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("variant", ["mgrawa", "lgrawa"])
def test_equal_norms_give_the_plain_mean(variant):
    """Equal gradient norms -> uniform weights -> the centre is the arithmetic mean of the workers."""
    M, sizes = 5, [7, 12, 3]
    x, _, off = _random_problem(M, sizes)
    base = f32(rng.normal(size=off[-1]))
    # same magnitudes, different signs/orderings per layer: norms equal, gradients not
    g = []
    for m in range(M):
        gm = base.copy()
        for k in range(len(sizes)):
            seg = gm[off[k]:off[k + 1]]
            seg[:] = np.roll(seg, m) * (-1) ** m
        g.append(gm)
    r = oracle.step(x, g, 0.5, variant, off)
    assert np.allclose(r["beta"], 1.0 / M, rtol=1e-14)
    assert np.allclose(r["center"], np.mean(np.stack(x).astype(np.float64), axis=0), rtol=1e-13, atol=1e-15)


def test_zero_gradient_worker_becomes_the_centre():
    x, g, off = _random_problem(4, [9, 5])
    g[2][:] = 0
    for v in ("grawa", "mgrawa", "lgrawa"):
        r = oracle.step(x, g, 0.5, v, off)
        assert np.array_equal(r["center"], x[2].astype(np.float64))


@pytest.mark.parametrize("variant", ["grawa", "mgrawa", "lgrawa"])
def test_centre_invariant_to_worker_permutation(variant):
    x, g, off = _random_problem(6, [5, 14, 2], scale=10.0 ** rng.uniform(-2, 1, size=6))
    ref = oracle.step(x, g, 0.5, variant, off)
    for _ in range(3):
        p = rng.permutation(6)
        r = oracle.step([x[i] for i in p], [g[i] for i in p], 0.5, variant, off)
        assert np.allclose(r["center"], ref["center"], rtol=1e-12, atol=1e-15)
        for a, i in enumerate(p):
            assert np.allclose(r["workers"][a], ref["workers"][i], rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("variant", ["grawa", "mgrawa", "lgrawa"])
def test_pull_strength_extremes_and_single_worker(variant):
    x, g, off = _random_problem(4, [3, 8, 5], scale=[0.1, 1, 2, 5])
    r1 = oracle.step(x, g, 1.0, variant, off)
    for w in r1["workers"]:
        assert np.array_equal(w, r1["center"])                     # full pull: every worker is the centre
    r0 = oracle.step(x, g, 0.0, variant, off)
    for w, xi in zip(r0["workers"], x):
        assert np.array_equal(w, xi.astype(np.float64))             # no pull: untouched
    assert np.array_equal(r0["center"], r1["center"])
    rs = oracle.step(x[:1], g[:1], 0.4, variant, off)               # M = 1: identity
    assert np.array_equal(rs["beta"].ravel(), np.ones(rs["beta"].size))
    assert np.array_equal(rs["center"], x[0].astype(np.float64))
    assert np.allclose(rs["workers"][0], x[0].astype(np.float64), rtol=1e-16)


@pytest.mark.parametrize("lam", [0.3, 0.5, 0.7])
def test_pull_identities(lam):
    x, g, off = _random_problem(5, [6, 1, 10], scale=[0.3, 1, 1, 4, 9])
    r = oracle.step(x, g, lam, "lgrawa", off)
    X = np.stack(x).astype(np.float64)
    W = np.stack(r["workers"])
    c = r["center"]
    assert np.all(c >= X.min(axis=0) - 1e-15) and np.all(c <= X.max(axis=0) + 1e-15)   # convex combination
    assert np.allclose(W[0] - W[3], (1 - lam) * (X[0] - X[3]), rtol=1e-12, atol=1e-15)  # spread shrinks by 1-lambda
    lay = np.repeat(np.arange(3), np.diff(off))
    assert np.allclose((r["beta"][lay].T * W).sum(axis=0), c, rtol=1e-12, atol=1e-15)   # weighted mean is a fixed point
    assert np.allclose(W, (1 - lam) * X + lam * c[None, :], rtol=1e-14, atol=1e-16)


def test_centre_uses_pre_pull_values_range_api():
    """The ranged call returns the same numbers as the whole-vector call (layer lookup from any j0)."""
    x, g, off = _random_problem(3, [4, 0, 9, 2, 0], scale=[1, 2, 3])
    r = oracle.step(x, g, 0.5, "lgrawa", off)
    for j0, j1 in [(0, 15), (3, 6), (4, 13), (13, 15), (7, 7)]:
        c, w = oracle.center_pull(x, r["beta"], 0.5, off, j0, j1)
        assert np.array_equal(c, r["center"][j0:j1])
        for m in range(3):
            assert np.array_equal(w[m], r["workers"][m][j0:j1])


def test_loud_worker_gets_proportionally_small_weight():
    g0 = f32(rng.normal(size=1000))
    g = [100 * g0, g0.copy(), g0.copy()]
    beta = oracle.weights(oracle.scores(oracle.sumsq(g), "mgrawa"))[0]
    assert np.allclose(beta[1] / beta[0], 100.0, rtol=1e-6) and np.allclose(beta.sum(), 1)


# ---------------------------------------------------------------- proximity step, running norms

def test_prox_closed_form():
    x = [f32(rng.normal(size=33)) for _ in range(3)]
    c = f32(rng.normal(size=33))
    out = oracle.prox(x, c, 0.05 / 16)
    for m in range(3):
        assert np.allclose(out[m], x[m] + (0.05 / 16) * (c.astype(np.float64) - x[m]), rtol=1e-13, atol=1e-16)
    assert np.array_equal(oracle.prox(x, c, 0.0)[1], x[1].astype(np.float64))
    assert np.array_equal(oracle.prox(x, c, 1.0)[2], c.astype(np.float64))


def test_norm_ema_constant_input_closed_form():
    """With a constant input c the moving value is (1-gamma^t) c, so the literal estimate is gamma c for every t."""
    gamma, c = 0.9, np.array([2.0, 0.5, 7.0])
    mvg = np.zeros(3)
    for t in range(1, 8):
        est = oracle.norm_ema(mvg, c, gamma, t)
        assert np.allclose(mvg, (1 - gamma ** t) * c, rtol=1e-13)
        assert np.allclose(est, gamma * c, rtol=1e-13)


def test_scores_from_norms_match_scores_from_sums():
    """Given the exact layer norms, the from-norms scores are the from-gradients scores."""
    sizes = [5, 17, 1, 300]
    off = np.concatenate([[0], np.cumsum(sizes)])
    g = [f32(rng.normal(size=off[-1]) * s) for s in (0.1, 1.0, 7.0)]
    S = oracle.sumsq(g, off)
    N = np.sqrt(S)
    assert np.array_equal(oracle.scores_from_norms(N, "lgrawa"), oracle.scores(S, "lgrawa"))
    assert np.array_equal(oracle.scores_from_norms(N, "mgrawa"), oracle.scores(S, "mgrawa"))
    assert np.allclose(oracle.scores_from_norms(N, "grawa"), oracle.scores(S, "grawa"), rtol=1e-14)
    # hand case: norms (3, 4) and (6, 8) over two layers -> MGRAWA (7, 14), GRAWA (5, 10), LGRAWA as given
    N = np.array([[3.0, 6.0], [4.0, 8.0]])
    assert np.array_equal(oracle.scores_from_norms(N, "mgrawa"), [7, 14])
    assert np.array_equal(oracle.scores_from_norms(N, "grawa"), [5, 10])
    assert np.array_equal(oracle.scores_from_norms(N, "lgrawa"), N)


def test_norm_ema_bias_correction_cancels_in_the_weights():
    """All workers share t, so the literal estimate (with its leading gamma) gives the same weights
    as the plain moving value: beta only sees ratios."""
    gamma = 0.8
    cur = rng.uniform(0.5, 2.0, size=(4, 3))            # 4 steps, 3 workers, one layer
    mvg = np.zeros((3, 1))
    for t in range(1, 5):
        est = np.stack([oracle.norm_ema(mvg[m], cur[t - 1, m:m + 1], gamma, t) for m in range(3)])
    beta_est = oracle.weights(est[:, 0])[0]
    beta_mvg = oracle.weights(mvg[:, 0])[0]
    assert np.allclose(beta_est, beta_mvg, rtol=1e-13)


# ---------------------------------------------------------------- property-based checks

from hypothesis import given, settings, strategies as st


@settings(max_examples=60, deadline=None)
@given(st.lists(st.floats(min_value=1e-6, max_value=1e6, allow_nan=False, allow_infinity=False), min_size=1, max_size=16))
def test_weights_properties_hold_for_any_positive_scores(scores):
    A = np.array(scores)
    beta, flagged = oracle.weights(A)
    assert not flagged
    assert abs(beta.sum() - 1.0) <= 1e-13 and np.all(beta > 0) and np.all(beta <= 1)
    assert np.allclose(beta * A, (beta * A)[0], rtol=1e-12)            # beta_m A_m is the same for all m (= Theta)
    assert (beta * A)[0] <= A.min() * (1 + 1e-12)                      # Theta <= every norm


@settings(max_examples=25, deadline=None)
@given(st.integers(min_value=1, max_value=6), st.lists(st.integers(min_value=0, max_value=9), min_size=1, max_size=5),
       st.floats(min_value=0.0, max_value=1.0), st.integers(min_value=0, max_value=10_000))
def test_step_invariants_on_random_small_problems(M, sizes, lam, seed):
    n = sum(sizes)
    if n == 0:
        return
    r = np.random.default_rng(seed)
    off = np.concatenate([[0], np.cumsum(sizes)])
    x = [f32(r.normal(size=n)) for _ in range(M)]
    g = [f32(r.normal(size=n) * 10.0 ** r.uniform(-2, 1)) for _ in range(M)]
    for variant in ("grawa", "mgrawa", "lgrawa"):
        out = oracle.step(x, g, lam, variant, off)
        X = np.stack(x).astype(np.float64)
        c = out["center"]
        assert np.all(c >= X.min(axis=0) - 1e-12) and np.all(c <= X.max(axis=0) + 1e-12)
        W = np.stack(out["workers"])
        assert np.allclose(W, (1 - lam) * X + lam * c[None, :], rtol=1e-13, atol=1e-15)
        b = out["beta"]
        assert np.allclose(b.sum(axis=-1), 1.0, atol=1e-13)
