"""Helpers of the GPU parity tests: run the CUDA path through the binding, run the oracle on the
same host inputs, compare chunk by chunk."""
import numpy as np

import oracle

# Tolerances of the parity contract: weights to 1e-5 relative, parameters and centre to
# 2e-6 * max|x| absolute (max over the input parameters), sums of squares to 1e-6 relative.
TOL_BETA_REL = 1e-5
TOL_X_ABS_FACTOR = 2e-6
TOL_S_REL = 1e-6
CHUNK = 1 << 18


def to_device(arrs):
    import torch
    return [torch.from_numpy(a).cuda() for a in arrs]


def gpu_step(grawa, variant, params_np, grads_np, pull, off=None, want_center=True, workspace=None,
             params_dev=None, grads_dev=None):
    """One step on the GPU.  Returns device tensors: workers (list), center, beta, scores, sumsq."""
    import torch
    M, n = len(params_np), params_np[0].size
    x = params_dev if params_dev is not None else to_device(params_np)
    g = grads_dev if grads_dev is not None else to_device(grads_np)
    K = (len(off) - 1) if off is not None else 1
    G = K if variant == "lgrawa" else 1
    beta = torch.full((G * M,), -1.0, dtype=torch.float32, device="cuda")
    scores = torch.full((G * M,), -1.0, dtype=torch.float64, device="cuda")
    sumsq = torch.full((K * M,), -1.0, dtype=torch.float64, device="cuda")
    center = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda") if want_center else None
    fn = {"mgrawa": grawa.grawa_mgrawa_step, "lgrawa": grawa.grawa_lgrawa_step, "grawa": grawa.grawa_grawa_step}[variant]
    fn(x, g, pull, off, center, weights_out=beta, scores_out=scores, sumsq_out=sumsq, workspace=workspace)
    torch.cuda.synchronize()
    shape = (K, M) if variant == "lgrawa" else (M,)
    return {"workers": x, "center": center, "beta": beta.cpu().numpy().reshape(shape),
            "A": scores.cpu().numpy().reshape(shape), "S": sumsq.cpu().numpy().reshape(K, M), "grads": g}


def _host(t):
    """A device tensor as a float32 numpy array (16-bit storage types are widened exactly)."""
    import torch
    return (t if t.dtype == torch.float32 else t.float()).cpu().numpy()


def compare_with_oracle(res, variant, params_np, grads_np, pull, off=None, check_workers=True, half_ulp=0.0, tiny=0.0):
    """Element-by-element comparison of a GPU result with the oracle on the same inputs.  For results
    stored in a 16-bit type, `half_ulp` (relative) and `tiny` (absolute) add the one rounding of the
    store to the fp32 bound."""
    M, n = len(params_np), params_np[0].size
    S = oracle.sumsq(grads_np, off)
    A = oracle.scores(S, variant)
    beta, _ = oracle.weights(A)
    # sums of squares and scores
    assert np.allclose(res["S"], S, rtol=TOL_S_REL, atol=0), np.abs(res["S"] / np.where(S == 0, 1, S) - 1).max()
    assert np.allclose(res["A"], A, rtol=TOL_S_REL, atol=0)
    # weights: relative error on every weight (exact zeros must be exact zeros)
    nz = beta != 0
    assert np.array_equal(res["beta"][~nz], beta[~nz])
    rel = np.abs(res["beta"][nz].astype(np.float64) - beta[nz]) / beta[nz]
    assert rel.size == 0 or rel.max() <= TOL_BETA_REL, rel.max()
    # centre and pulled workers, chunked
    xmax = max(float(np.abs(p).max()) for p in params_np) if n else 0.0
    tol = TOL_X_ABS_FACTOR * xmax
    worst = 0.0
    workers_host = [_host(w) for w in res["workers"]] if check_workers else None
    center_host = _host(res["center"]) if res["center"] is not None else None
    bufs = (np.zeros(CHUNK), [np.zeros(CHUNK) for _ in range(M)])      # reused: fresh pages are slow
    for j0 in range(0, n, CHUNK):
        j1 = min(n, j0 + CHUNK)
        c, w = oracle.center_pull(params_np, beta, pull, off, j0, j1, want_workers=check_workers, out=bufs)
        if center_host is not None:
            worst = max(worst, float((np.abs(center_host[j0:j1] - c) - half_ulp * np.abs(c) - tiny).max()))
        if check_workers:
            for m in range(M):
                worst = max(worst, float((np.abs(workers_host[m][j0:j1] - w[m]) - half_ulp * np.abs(w[m]) - tiny).max()))
    assert worst <= tol, (worst, tol)
    return {"beta_rel": float(rel.max()) if rel.size else 0.0, "x_abs_over_max": worst / xmax if xmax else 0.0}
