"""ctypes front end of the float64 CPU oracle in ``grawa_oracle.c``.

TEST INFRASTRUCTURE ONLY: the oracle defines what the averaging update must
compute (it is written from the paper's equations) and is what the CUDA library
is compared against.  It is never on a product path; only tests, the smoke check
and the benchmark's CPU-baseline leg import this package.  It shares no code with
the CUDA library and does not import it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "grawa_oracle.c")
_LIB = os.path.join(_HERE, "libgrawa_oracle.so")

GRAWA, MGRAWA, LGRAWA = 0, 1, 2
VARIANTS = {"grawa": GRAWA, "mgrawa": MGRAWA, "lgrawa": LGRAWA}


def build(force: bool = False) -> str:
    """Compile the oracle (plain gcc -O2, single thread, strict IEEE) when missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i64, ci, dbl = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_double
        lib.grawa_oracle_sumsq.argtypes = [vp, ci, vp, ci, vp]
        lib.grawa_oracle_sumsq.restype = None
        lib.grawa_oracle_scores.argtypes = [vp, ci, ci, ci, vp]
        lib.grawa_oracle_scores.restype = None
        lib.grawa_oracle_scores_from_norms.argtypes = [vp, ci, ci, ci, vp]
        lib.grawa_oracle_scores_from_norms.restype = None
        lib.grawa_oracle_weights.argtypes = [vp, ci, ci, vp]
        lib.grawa_oracle_weights.restype = ci
        lib.grawa_oracle_center_pull.argtypes = [vp, ci, vp, ci, vp, ci, i64, i64, dbl, vp, vp]
        lib.grawa_oracle_center_pull.restype = None
        lib.grawa_oracle_prox.argtypes = [vp, ci, vp, i64, dbl, vp]
        lib.grawa_oracle_prox.restype = None
        lib.grawa_oracle_norm_ema.argtypes = [vp, vp, ci, dbl, i64, vp]
        lib.grawa_oracle_norm_ema.restype = None
        _lib = lib
    return _lib


def _f32_list(arrs):
    out = []
    for a in arrs:
        a = np.asarray(a)
        if a.dtype != np.float32 or not a.flags["C_CONTIGUOUS"]:
            a = np.ascontiguousarray(a, dtype=np.float32)
        out.append(a)
    return out


def _ptr_array(arrs):
    return (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def _offsets(off, n):
    if off is None:
        return np.array([0, n], dtype=np.int64)
    off = np.ascontiguousarray(off, dtype=np.int64)
    assert off[0] == 0 and off[-1] == n and np.all(np.diff(off) >= 0), "bad layer offsets"
    return off


def sumsq(grads, layer_offsets=None) -> np.ndarray:
    """Step 1: S[k, m] = sum of squares of worker m's gradient over layer k (Eq. 3 / Eq. 5)."""
    g = _f32_list(grads)
    off = _offsets(layer_offsets, g[0].size)
    K, M = off.size - 1, len(g)
    S = np.zeros((K, M), dtype=np.float64)
    _load().grawa_oracle_sumsq(_ptr_array(g), M, off.ctypes.data, K, S.ctypes.data)
    return S


def scores(S, variant) -> np.ndarray:
    """Step 2: LGRAWA sqrt(S) [K, M] (Eq. 5-6); MGRAWA sum_k sqrt(S) [M] (Eq. 3); GRAWA sqrt(sum_k S) [M] (Eq. 2)."""
    v = VARIANTS[variant] if isinstance(variant, str) else variant
    S = np.ascontiguousarray(S, dtype=np.float64)
    K, M = S.shape
    A = np.zeros((K, M) if v == LGRAWA else (M,), dtype=np.float64)
    _load().grawa_oracle_scores(S.ctypes.data, K, M, v, A.ctypes.data)
    return A


def scores_from_norms(norms, variant) -> np.ndarray:
    """Step 2 from given per-layer norms [K, M] (the running estimates of the Local variants)."""
    v = VARIANTS[variant] if isinstance(variant, str) else variant
    N = np.ascontiguousarray(norms, dtype=np.float64)
    K, M = N.shape
    A = np.zeros((K, M) if v == LGRAWA else (M,), dtype=np.float64)
    _load().grawa_oracle_scores_from_norms(N.ctypes.data, K, M, v, A.ctypes.data)
    return A


def weights(A):
    """Step 3: inverse-score weights normalised to 1 over the last axis (Eq. 2, 4, 7).
    Returns (beta, flagged) where flagged tells that a non-finite score was met."""
    A = np.ascontiguousarray(A, dtype=np.float64)
    groups = 1 if A.ndim == 1 else A.shape[0]
    M = A.shape[-1]
    beta = np.zeros_like(A)
    flagged = _load().grawa_oracle_weights(A.ctypes.data, groups, M, beta.ctypes.data)
    return beta, bool(flagged)


def center_pull(params, beta, pull, layer_offsets=None, j0=0, j1=None, want_workers=True, out=None):
    """Steps 4-5 on [j0, j1): x_C = sum_m beta_m x_m, then x_m <- (1-pull) x_m + pull x_C.
    ``beta`` is [K, M] (per layer, Eq. 7) or [M].  Returns (center, workers) in float64.
    ``out``: optional (center_buffer, [worker_buffers]) of float64 arrays with at least j1-j0
    elements that are reused instead of allocating fresh outputs (views of them are returned)."""
    x = _f32_list(params)
    n, M = x[0].size, len(x)
    j1 = n if j1 is None else j1
    beta = np.ascontiguousarray(beta, dtype=np.float64)
    per_layer = beta.ndim == 2
    off = _offsets(layer_offsets, n)
    K = off.size - 1
    if per_layer:
        assert beta.shape == (K, M)
    else:
        assert beta.shape == (M,)
    if out is not None:
        center = out[0][:j1 - j0]
        outs = [b[:j1 - j0] for b in out[1]] if want_workers else None
        assert center.dtype == np.float64 and center.flags["C_CONTIGUOUS"] and center.size == j1 - j0
    else:
        center = np.zeros(j1 - j0, dtype=np.float64)
        outs = [np.zeros(j1 - j0, dtype=np.float64) for _ in range(M)] if want_workers else None
    _load().grawa_oracle_center_pull(_ptr_array(x), M, beta.ctypes.data, int(per_layer),
                                     off.ctypes.data, K, j0, j1, float(pull), center.ctypes.data,
                                     _ptr_array(outs) if want_workers else None)
    return center, outs


def step(params, grads, pull, variant, layer_offsets=None):
    """The whole update.  Returns a dict with S, A, beta, center, workers (float64) and flagged."""
    S = sumsq(grads, layer_offsets)
    A = scores(S, variant)
    beta, flagged = weights(A)
    center, outs = center_pull(params, beta, pull, layer_offsets)
    return {"S": S, "A": A, "beta": beta, "center": center, "workers": outs, "flagged": flagged}


def prox(params, center, mu_over_tau):
    """Proximity step of the local phase: x_m <- (1 - mu/tau) x_m + (mu/tau) x_C (the "Prox." update of Algorithm 1)."""
    x = _f32_list(params)
    c = _f32_list([center])[0]
    outs = [np.zeros(c.size, dtype=np.float64) for _ in x]
    _load().grawa_oracle_prox(_ptr_array(x), len(x), c.ctypes.data, c.size, float(mu_over_tau), _ptr_array(outs))
    return outs


def norm_ema(g_mvg, g_cur, gamma, t):
    """Local-GRAWA running norm: updates g_mvg in place, returns g_est (appendix algorithm, taken literally)."""
    assert g_mvg.dtype == np.float64 and g_mvg.flags["C_CONTIGUOUS"]
    g_cur = np.ascontiguousarray(g_cur, dtype=np.float64)
    est = np.zeros_like(g_mvg)
    _load().grawa_oracle_norm_ema(g_mvg.ctypes.data, g_cur.ctypes.data, g_mvg.size, float(gamma), int(t), est.ctypes.data)
    return est
