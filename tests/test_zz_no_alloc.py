"""The allocation-free entry point grawa_sumsq_static against the ordinary step's sums of squares
and against the CPU oracle.

Some users of this library cannot let it allocate: their device memory is already owned by a
framework's pool, so a cudaMalloc from inside the library fails or fragments it, or they sit in
a latency-bound loop where the device-wide synchronisation of an allocation is not acceptable.
grawa_sumsq_static serves them from a scratch array compiled into the library.  This test calls
it through the C ABI twice in a row (second call smaller than the first, so left-over scratch
contents would show) and compares with what grawa_grawa_step reports for the same gradients and
with the oracle's float64 sums, and checks the claim the entry point exists for: the device's free
memory is the same after its calls as before them.
Collected last on purpose: a failure here leaves every other test already run.
"""
import ctypes

import numpy as np
import pytest

import gen
import oracle

TOL_S_REL = 1e-6          # the tolerance the parity tests use for sums of squares


def test_too_large_and_bad_arguments_are_rejected_on_the_host():
    import paper_2403_04206_b200 as grawa
    lib = grawa.library()
    G = (ctypes.c_void_p * 4)(0x10000000, 0x20000000, 0x30000000, 0x40000000)
    limit_tiles = 131072 // 4
    assert lib.grawa_sumsq_static(G, limit_tiles * 16384 + 1, 4, 0x50000000, None) == -6
    assert "scratch" in grawa.grawa_status_string(-6)
    assert lib.grawa_sumsq_static(None, 100, 4, 0x50000000, None) == -1
    assert lib.grawa_sumsq_static(G, 100, 4, None, None) == -1
    assert lib.grawa_sumsq_static(G, 100, 0, 0x50000000, None) == -1
    assert lib.grawa_sumsq_static(G, -1, 4, 0x50000000, None) == -1


@pytest.mark.gpu
def test_static_scratch_sums_match_the_step_entry_point_twice_in_a_row():
    import torch
    import paper_2403_04206_b200 as grawa

    def reference(p, g):
        x = [torch.from_numpy(a).cuda() for a in p]
        gr = [torch.from_numpy(a).cuda() for a in g]
        out = torch.zeros(len(g), dtype=torch.float64, device="cuda")
        grawa.grawa_grawa_step(x, gr, 0.0, None, None, sumsq_out=out)     # pull 0: workers untouched
        torch.cuda.synchronize()
        return out.cpu().numpy(), gr

    # one small call first: the driver loads a kernel's code on its first launch, which is not an
    # allocation by this library but would show in the free-memory comparison below
    warm = torch.zeros(1, dtype=torch.float64, device="cuda")
    grawa.grawa_sumsq_static([torch.ones(64, device="cuda")], warm)
    torch.cuda.synchronize()
    assert float(warm.item()) == 64.0
    big = gen.custom_config([3_000_001], 5, seed=41, log10_sigma=(-3.0, 0.0))
    small = gen.custom_config([70_003], 3, seed=42, log10_sigma=(-3.0, 0.0))
    for cfg in (big, small):                      # two calls in a row on the shared scratch
        p, g = gen.make_inputs(cfg)
        want, gr = reference(p, g)
        got = torch.full((cfg.M,), -1.0, dtype=torch.float64, device="cuda")
        again = torch.full((cfg.M,), -1.0, dtype=torch.float64, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]          # what the driver has left, torch's pool included
        grawa.grawa_sumsq_static(gr, got)
        grawa.grawa_sumsq_static(gr, again)       # same inputs: same bytes
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before  # neither call took device memory from anybody
        got = got.cpu().numpy()
        assert np.all(want > 0)
        assert np.abs(got / want - 1).max() <= TOL_S_REL, (got, want)
        exact = oracle.sumsq(g)[0]                           # the definition, in float64
        assert np.abs(got / exact - 1).max() <= TOL_S_REL, (got, exact)
        assert np.array_equal(again.cpu().numpy(), got)
    # n = 0 writes zeros
    z = torch.full((2,), -1.0, dtype=torch.float64, device="cuda")
    grawa.grawa_sumsq_static([torch.empty(0, device="cuda"), torch.empty(0, device="cuda")], z, n=0)
    torch.cuda.synchronize()
    assert np.array_equal(z.cpu().numpy(), [0.0, 0.0])
