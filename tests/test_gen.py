"""The seeded input generator: published Philox known answers, layer-table totals,
reproducibility, and the statistical shape the workload recipes promise."""
import numpy as np
import pytest

import gen
from gen.values import CONFIG_ORDER


def test_philox_known_answers():
    """Known-answer vectors published with the Philox4x32-10 definition."""
    kat = [
        ([0, 0, 0, 0], [0, 0], [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]),
        ([0xffffffff] * 4, [0xffffffff] * 2, [0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd]),
        ([0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344], [0xa4093822, 0x299f31d0],
         [0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1]),
    ]
    for ctr, key, out in kat:
        assert [int(v) for v in gen.philox_block(ctr, key)] == out


def test_layer_table_totals():
    want = {"toy10": (10, 726346), "resnet20_cifar": (59, 269722), "resnet18_imagenet": (62, 11689512),
            "vgg16": (32, 138357544), "vit_b16": (152, 86567656)}
    for name in CONFIG_ORDER:
        cfg = gen.CONFIGS[name]
        assert (cfg.K, cfg.n) == want[name]
        off = cfg.offsets()
        assert off[0] == 0 and np.all(np.diff(off) > 0)
    assert max(gen.layer_sizes(gen.TABLES["vgg16"]())) == 25088 * 4096
    assert [gen.CONFIGS[c].M for c in CONFIG_ORDER] == [4, 8, 8, 4, 16]


def test_values_reproducible_and_worker_independent():
    cfg = gen.CONFIGS["resnet20_cifar"]
    p1, g1 = gen.make_inputs(cfg)
    p2, g2 = gen.make_inputs(cfg)
    for a, b in zip(p1 + g1, p2 + g2):
        assert np.array_equal(a, b)
    # a worker's values do not depend on which subset of workers is generated
    n = cfg.n
    ps = [np.zeros(n, np.float32) for _ in range(cfg.M)]
    gs = [np.zeros(n, np.float32) for _ in range(cfg.M)]
    gen.make_inputs(cfg, ps, gs, workers=[5])
    assert np.array_equal(ps[5], p1[5]) and np.array_equal(gs[5], g1[5]) and not ps[4].any()
    # workers differ from each other, but share the common base (drift is 10 % of the base std)
    off = cfg.offsets()
    w0, w1 = p1[0][off[3]:off[4]], p1[1][off[3]:off[4]]
    assert not np.array_equal(w0, w1) and np.corrcoef(w0, w1)[0, 1] > 0.95


def test_value_distributions():
    cfg = gen.CONFIGS["toy10"]
    p, g = gen.make_inputs(cfg)
    off = cfg.offsets()
    assert abs(p[0].std() - 0.05) < 5e-4 and abs(p[0].mean()) < 5e-4
    for m in range(cfg.M):
        for k in (2, 4, 6):
            s = g[m][off[k]:off[k + 1]].std()
            assert 0.9e-3 < s < 1.1e-1
    # kurtosis of the normal fill is 3 within sampling error
    z = p[1][off[4]:off[5]] / 0.05
    assert abs((z ** 4).mean() - 3.0) < 0.1
    cfg5 = gen.custom_config([20000, 30000], 3, seed=9, grad_recipe="student_t3", loud_worker_factor=100.0)
    _, g5 = gen.make_inputs(cfg5)
    assert np.abs(g5[1]).max() / g5[1].std() > 8          # heavy tails
    cfgn = gen.custom_config([20000, 30000], 3, seed=9, loud_worker_factor=100.0)
    _, gn = gen.make_inputs(cfgn)
    cfg1 = gen.custom_config([20000, 30000], 3, seed=9)
    _, g1 = gen.make_inputs(cfg1)
    assert np.allclose(gn[0], 100 * g1[0], rtol=1e-6) and np.array_equal(gn[1], g1[1])


def test_custom_config_allows_empty_layers():
    cfg = gen.custom_config([5, 0, 3, 0], 2, seed=3)
    p, g = gen.make_inputs(cfg)
    assert cfg.n == 8 and cfg.K == 4 and p[0].size == 8 and np.all(np.isfinite(g[1]))
