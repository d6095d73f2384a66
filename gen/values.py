"""Value recipes of the five benchmark workloads and the ctypes loader of the
counter-based generator in ``synth.c``.

Everything here is seeded and synthetic: the layer tables stand in for the CNN
and transformer workloads of the paper's experiments (whose datasets and trained
weights are not needed to exercise the averaging update).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from math import sqrt

import numpy as np

from .layer_tables import TABLES, layer_offsets

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "synth.c")
_LIB = os.path.join(_HERE, "libsynth.so")

# Philox key word 1 ("purpose") values: separate, non-overlapping streams.
_P_BASE, _P_WORKER, _P_GRAD, _P_SIGMA = 1, 2, 3, 4


def build(force: bool = False) -> str:
    """Compile ``synth.c`` into ``libsynth.so`` next to it (gcc, OpenMP) when missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        f32p, i64, dbl, u32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_double, ctypes.c_uint32
        lib.synth_fill_normal.argtypes = [f32p, f32p, i64, dbl, dbl, u32, u32, u32, u32]
        lib.synth_fill_student_t3.argtypes = [f32p, i64, dbl, u32, u32, u32, u32]
        lib.synth_fill_uniform.argtypes = [ctypes.c_void_p, i64, u32, u32, u32, u32]
        lib.synth_scale.argtypes = [f32p, i64, dbl]
        lib.synth_philox_block.argtypes = [ctypes.c_void_p] * 3
        for f in (lib.synth_fill_normal, lib.synth_fill_student_t3, lib.synth_fill_uniform,
                  lib.synth_scale, lib.synth_philox_block):
            f.restype = None
        _lib = lib
    return _lib


def philox_block(counter, key):
    """One raw Philox4x32-10 block (for the known-answer test)."""
    c = np.asarray(counter, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    _load().synth_philox_block(c.ctypes.data, k.ctypes.data, out.ctypes.data)
    return out


def _ptr(a: np.ndarray) -> int:
    assert a.dtype == np.float32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def _normal(out, base, mean, std, seed, purpose, worker, layer):
    _load().synth_fill_normal(_ptr(out), _ptr(base) if base is not None else None, out.size,
                              float(mean), float(std), seed, purpose, worker, layer)


def _uniform(n, seed, purpose, worker, layer=0):
    out = np.zeros(n, dtype=np.float64)
    _load().synth_fill_uniform(out.ctypes.data, n, seed, purpose, worker, layer)
    return out


@dataclass(frozen=True)
class WorkloadConfig:
    """One benchmark workload: a layer table, M workers and the value recipe."""
    name: str
    table: str                 # key of gen.TABLES, or "custom"
    M: int
    pull: float
    seed: int
    param_recipe: str          # "iid" | "kaiming" | "transformer"
    grad_recipe: str           # "normal" | "student_t3"
    log10_sigma: tuple         # (lo, hi) of the log-uniform per-(worker, layer) gradient scale
    loud_worker_factor: float = 1.0   # worker 0's gradients are multiplied by this
    sizes: tuple = field(default=())  # only for table == "custom"

    def layers(self):
        if self.table == "custom":
            return [(f"layer{i}", (int(s),), "weight", 0) for i, s in enumerate(self.sizes)]
        return TABLES[self.table]()

    def offsets(self) -> np.ndarray:
        return layer_offsets(self.layers())

    @property
    def n(self) -> int:
        return int(self.offsets()[-1])

    @property
    def K(self) -> int:
        return len(self.layers())

    def algorithmic_bytes(self) -> int:
        """Gradients read once, parameters read once and written once, centre written once."""
        return (3 * self.M + 1) * 4 * self.n


CONFIGS = {
    "toy10": WorkloadConfig("toy10", "toy10", 4, 0.5, 0, "iid", "normal", (-3.0, -1.0)),
    "resnet20_cifar": WorkloadConfig("resnet20_cifar", "resnet20_cifar", 8, 0.5, 1, "kaiming", "normal", (-4.0, -1.0)),
    "resnet18_imagenet": WorkloadConfig("resnet18_imagenet", "resnet18_imagenet", 8, 0.5, 2, "kaiming", "student_t3", (-4.0, -1.0)),
    "vgg16": WorkloadConfig("vgg16", "vgg16", 4, 0.5, 3, "kaiming", "normal", (-4.0, -1.0)),
    "vit_b16": WorkloadConfig("vit_b16", "vit_b16", 16, 0.5, 4, "transformer", "normal", (-3.0, -1.0), 100.0),
}
CONFIG_ORDER = ["toy10", "resnet20_cifar", "resnet18_imagenet", "vgg16", "vit_b16"]


def custom_config(sizes, M, seed=0, pull=0.5, param_recipe="iid", grad_recipe="normal",
                  log10_sigma=(-3.0, -1.0), loud_worker_factor=1.0, name="custom") -> WorkloadConfig:
    """A workload over an arbitrary list of layer sizes (zero-sized layers allowed)."""
    return WorkloadConfig(name, "custom", int(M), float(pull), int(seed), param_recipe, grad_recipe,
                          tuple(log10_sigma), float(loud_worker_factor), tuple(int(s) for s in sizes))


def make_inputs(cfg: WorkloadConfig, params_out=None, grads_out=None, workers=None):
    """Fill (or allocate) the M parameter vectors and M gradient vectors of ``cfg``.

    ``params_out`` / ``grads_out``: optional lists of M C-contiguous float32 numpy
    arrays of n elements (for example views of pinned buffers) that are filled in
    place.  ``workers`` restricts the work to a subset of worker indices (others
    are left untouched); a worker's values never depend on which subset is asked for.
    Returns ``(params, grads)`` as lists of numpy arrays.
    """
    layers = cfg.layers()
    off = cfg.offsets()
    n, M, seed = int(off[-1]), cfg.M, cfg.seed
    if params_out is None:
        params_out = [np.empty(n, dtype=np.float32) for _ in range(M)]
    if grads_out is None:
        grads_out = [np.empty(n, dtype=np.float32) for _ in range(M)]
    workers = range(M) if workers is None else workers
    lo, hi = cfg.log10_sigma

    base = None
    if cfg.param_recipe in ("kaiming", "transformer"):
        base = np.empty(n, dtype=np.float32)
        for k, (_, _, kind, fan_in) in enumerate(layers):
            seg = base[off[k]:off[k + 1]]
            if seg.size == 0:
                continue
            if kind in ("weight", "embed"):
                std = sqrt(2.0 / fan_in) if (cfg.param_recipe == "kaiming" and fan_in) else 0.02
                _normal(seg, None, 0.0, std, seed, _P_BASE, 0, k)
            else:
                seg[:] = 0.0  # gains/shifts are drawn per worker below

    for m in workers:
        x, g = params_out[m], grads_out[m]
        assert x.size == n and g.size == n
        u = _uniform(max(len(layers), 1), seed, _P_SIGMA, m)
        for k, (_, _, kind, fan_in) in enumerate(layers):
            xs, gs = x[off[k]:off[k + 1]], g[off[k]:off[k + 1]]
            if xs.size == 0:
                continue
            # parameters
            if cfg.param_recipe == "iid":
                _normal(xs, None, 0.0, 0.05, seed, _P_WORKER, m, k)
            elif kind in ("weight", "embed"):
                std = sqrt(2.0 / fan_in) if (cfg.param_recipe == "kaiming" and fan_in) else 0.02
                _normal(xs, base[off[k]:off[k + 1]], 0.0, 0.1 * std, seed, _P_WORKER, m, k)
            elif kind == "scale":
                _normal(xs, None, 1.0, 0.02, seed, _P_WORKER, m, k)
            else:
                _normal(xs, None, 0.0, 0.02, seed, _P_WORKER, m, k)
            # gradients
            sigma = 10.0 ** (lo + (hi - lo) * u[k])
            if m == 0:
                sigma *= cfg.loud_worker_factor
            if cfg.grad_recipe == "student_t3":
                _load().synth_fill_student_t3(_ptr(gs), gs.size, sigma, seed, _P_GRAD, m, k)
            else:
                _normal(gs, None, 0.0, sigma, seed, _P_GRAD, m, k)
    return params_out, grads_out
