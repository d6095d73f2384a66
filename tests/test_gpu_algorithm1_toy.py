"""Algorithm 1 (MGRAWA) end to end on the paper's toy problem, the Vincent function
f(x, y) = -sin(10 ln x) - sin(10 ln y): four workers started from the corners the paper lists run
SGD with learning rate 0.01, take the proximity step every iteration and the distributed update
every tau = 4 iterations (the gradient at the current point stands for the accumulated gradient).
The library drives the proximity and averaging steps on the GPU; the oracle runs the same loop in
float64.  The paper prints no numbers for this example (only figures) and does not state its pull
strength, so this is a wiring check of the two entry points in the algorithm's order, not a pin."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu

STARTS = [(0.25, 0.25), (0.25, 10.0), (10.0, 0.25), (10.0, 10.0)]
ETA, TAU, MU, LAM, ITERS = 0.01, 4, 0.05, 0.5, 24


def grad(p):
    return -10.0 * np.cos(10.0 * np.log(p)) / p


def test_algorithm_1_loop_matches_the_oracle_loop():
    import torch
    import paper_2403_04206_b200 as grawa
    # float64 loop with the oracle
    xs = [np.array(s, dtype=np.float64) for s in STARTS]
    xc = np.mean(xs, axis=0)
    # GPU loop with the library (fp32 storage)
    xg = [torch.tensor(s, dtype=torch.float32, device="cuda") for s in STARTS]
    cg = torch.tensor(np.mean(STARTS, axis=0), dtype=torch.float32, device="cuda")
    for t in range(1, ITERS + 1):
        # local SGD step (the caller's part of the algorithm)
        xs = [x - ETA * grad(x) for x in xs]
        for x in xg:
            p = x.double()
            x.copy_((p - ETA * (-10.0 * torch.cos(10.0 * torch.log(p)) / p)).float())
        # proximity step
        xs = [np.asarray(o) for o in oracle.prox([x.astype(np.float32) for x in xs], xc.astype(np.float32), MU / TAU)]
        grawa.grawa_prox_step(xg, cg, MU / TAU)
        if t % TAU == 0:
            g_or = [grad(x).astype(np.float32) for x in xs]
            out = oracle.step([x.astype(np.float32) for x in xs], g_or, LAM, "mgrawa")
            xs, xc = [np.asarray(w) for w in out["workers"]], np.asarray(out["center"])
            gg = [(-10.0 * torch.cos(10.0 * torch.log(x.double())) / x.double()).float() for x in xg]
            grawa.grawa_mgrawa_step(xg, gg, LAM, None, cg)
            assert grawa.grawa_last_step_status() == 0
    torch.cuda.synchronize()
    got = np.stack([x.cpu().numpy() for x in xg])
    want = np.stack(xs)
    # fp32 storage against a float64 loop that re-rounds its state to fp32 at every library call
    assert np.abs(got - want).max() <= 5e-4 * np.abs(want).max(), (got, want)
    assert np.abs(cg.cpu().numpy() - xc).max() <= 5e-4 * np.abs(want).max()
    # the pull did its job: the workers are closer together than the starting corners
    assert np.ptp(got, axis=0).max() < np.ptp(np.array(STARTS), axis=0).max()
