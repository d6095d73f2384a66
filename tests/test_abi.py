"""The C-ABI library builds, loads and exports every symbol include/grawa.h declares, and its
host-side validation rejects bad arguments before anything is enqueued (no GPU needed)."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2403_04206_b200 as grawa
from paper_2403_04206_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "grawa.h")


def declared_functions():
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    return sorted(set(re.findall(r"\b(grawa_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = grawa.library()
    names = declared_functions()
    assert {"grawa_mgrawa_step", "grawa_lgrawa_step", "grawa_grawa_step", "grawa_step_host",
            "grawa_prox_step", "grawa_workspace_bytes", "grawa_last_step_status"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in grawa.h but not exported"
        assert hasattr(grawa, name), f"{name} has no Python binding of the same name"


def test_version_and_strings():
    assert grawa.grawa_version() >= 100
    assert grawa.grawa_status_string(0) == "ok"
    assert "invalid" in grawa.grawa_status_string(-1)
    assert grawa.grawa_status_string(-3) and grawa.grawa_status_string(-99)


def test_workspace_bytes_grows_with_layers_and_workers_and_rejects_bad_tables():
    small = grawa.grawa_workspace_bytes(1000, 4, [0, 10, 1000])
    more_layers = grawa.grawa_workspace_bytes(1000, 4, [0, 10, 20, 30, 40, 1000])
    more_workers = grawa.grawa_workspace_bytes(1000, 16, [0, 10, 1000])
    assert 0 < small < more_layers and small < more_workers and small % 256 == 0
    # the scratch holds per-(layer, worker) tables only: it does not grow with the vector
    assert grawa.grawa_workspace_bytes(10_000_000, 4, [0, 10, 10_000_000]) == small
    assert grawa.grawa_workspace_bytes(1000, 4) > 0
    assert grawa.grawa_workspace_bytes(1000, 0) == 0
    assert grawa.grawa_workspace_bytes(1000, 65) == 0
    assert grawa.grawa_workspace_bytes(1000, 4, [0, 20, 10, 1000]) == 0     # decreasing
    assert grawa.grawa_workspace_bytes(1000, 4, [1, 10, 1000]) == 0         # does not start at 0
    assert grawa.grawa_workspace_bytes(1000, 4, [0, 10, 999]) == 0          # does not end at n


def _host_call(name, params, grads, n, M, pull, off, center):
    """Raw call with fake (never dereferenced) device addresses; stream 0.  Only used with
    arguments the host validation must reject, so nothing is enqueued."""
    lib = grawa.library()
    P = (ctypes.c_void_p * max(1, len(params)))(*params) if params is not None else None
    G = (ctypes.c_void_p * max(1, len(grads)))(*grads) if grads is not None else None
    o = np.asarray(off, dtype=np.int64) if off is not None else None
    return getattr(lib, name)(P, G, n, M, ctypes.c_float(pull), o.ctypes.data if o is not None else None,
                              (o.size - 1) if o is not None else 0, center, None, None)


@pytest.mark.parametrize("name", ["grawa_mgrawa_step", "grawa_lgrawa_step", "grawa_grawa_step"])
def test_host_validation_rejects_before_launch(name):
    n, B = 1000, 1 << 20
    ok_p, ok_g = [0x10000000 + i * B for i in range(4)], [0x20000000 + i * B for i in range(4)]
    bad = lambda **kw: _host_call(name, kw.get("p", ok_p), kw.get("g", ok_g), kw.get("n", n), kw.get("M", 4),
                                  kw.get("pull", 0.5), kw.get("off", [0, 10, n]), kw.get("c", 0x30000000))
    assert bad(pull=1.5) == -1 and bad(pull=-0.1) == -1 and bad(pull=float("nan")) == -1
    assert bad(M=0) == -1 and bad(M=65) == -1 and bad(n=-1) == -1
    assert bad(off=[0, 20, 10, n]) == -1 and bad(off=[0, 10, n + 1]) == -1 and bad(off=[5, 10, n]) == -1
    assert bad(p=None) == -1 and bad(g=None) == -1
    assert bad(p=[ok_p[0], 0, ok_p[2], ok_p[3]]) == -1                      # NULL worker
    assert bad(p=[ok_p[0], ok_p[0] + 16, ok_p[2], ok_p[3]]) == -1           # two workers overlap
    assert bad(c=ok_p[1] + 400) == -1                                       # centre overlaps a worker
    assert bad(g=[ok_p[0]] + ok_g[1:]) == -1                                # gradient aliases a parameter
    assert bad(p=[ok_p[0] + 2] + ok_p[1:]) == -1                            # not 4-byte aligned
    # n = 0 is a no-op that succeeds without touching the device
    assert _host_call(name, ok_p, ok_g, 0, 4, 0.5, [0, 0], 0) == 0


def test_prox_and_host_step_validation():
    lib = grawa.library()
    P = (ctypes.c_void_p * 2)(0x10000000, 0x10100000)
    assert lib.grawa_prox_step(P, 0x30000000, 100, 2, ctypes.c_float(1.5), None) == -1
    assert lib.grawa_prox_step(P, None, 100, 2, ctypes.c_float(0.1), None) == -1
    assert lib.grawa_prox_step(P, 0x30000000, 0, 2, ctypes.c_float(0.1), None) == 0
    assert lib.grawa_step_host(7, P, P, 100, 2, ctypes.c_float(0.5), None, 0, None, None) == -1
    with pytest.raises(grawa.GrawaError):
        grawa.grawa_step_host("mgrawa", [np.zeros(4, np.float32)], [np.zeros(4, np.float32)], 2.0, stream=0)


def test_options_roundtrip_and_range():
    assert grawa.grawa_get_option("no_such_option") == -1
    old = grawa.grawa_get_option("pull_variant")
    grawa.grawa_set_option("pull_variant", old)
    with pytest.raises(grawa.GrawaError):
        grawa.grawa_set_option("pull_variant", 9)
    with pytest.raises(grawa.GrawaError):
        grawa.grawa_set_option("sumsq_tile", 1000)     # not a multiple of 1024
    with pytest.raises(grawa.GrawaError):
        grawa.grawa_set_option("no_such_option", 1)
    assert grawa.grawa_get_option("sumsq_tile") % 1024 == 0


def test_binding_type_checks():
    with pytest.raises(TypeError):
        grawa.grawa_step_host("mgrawa", [np.zeros(4, np.float64)], [np.zeros(4, np.float32)], 0.5, stream=0)
    with pytest.raises(ValueError):
        binding._addr(np.zeros((4, 4), np.float32)[:, 0])
