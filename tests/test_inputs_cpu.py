"""Seeded input generator: counter-based addressing, determinism and distribution (CPU only)."""
import math

import numpy as np
import torch

from paper_1811_10792_b200 import inputs


def test_any_column_range_can_be_regenerated():
    full = inputs.normal(5, 3000, seed=11, stream=inputs.STREAM_GRAD, step=7, std=0.1)
    part = inputs.normal(5, 200, seed=11, stream=inputs.STREAM_GRAD, step=7, std=0.1, col_offset=1234)
    assert torch.equal(part, full[:, 1234:1434])
    padded = inputs.normal(5, 3000, seed=11, stream=inputs.STREAM_GRAD, step=7, std=0.1, ld=3072)
    assert padded.stride(0) == 3072 and torch.equal(padded, full)


def test_streams_steps_seeds_and_rows_are_independent():
    base = inputs.normal(4, 512, seed=1, stream=2, step=0, std=1.0)
    for kw in (dict(seed=2, stream=2, step=0), dict(seed=1, stream=3, step=0), dict(seed=1, stream=2, step=1)):
        other = inputs.normal(4, 512, std=1.0, **kw)
        assert not torch.equal(base, other)
        assert abs(float((base * other).mean())) < 0.1
    assert not torch.equal(base[0], base[1])


def test_distribution_moments():
    x = inputs.normal(8, 200_000, seed=5, stream=1, step=3, std=0.1).double().numpy()
    assert abs(x.mean()) < 1e-3 and abs(x.std() - 0.1) < 1e-3
    z = x / 0.1
    assert abs((z ** 3).mean()) < 0.02 and abs((z ** 4).mean() - 3.0) < 0.05
    assert np.isfinite(x).all()


def test_workload_recipes():
    w = inputs.WORKLOADS["resnet50"]
    assert (w.n, w.d, w.K, w.peers, w.momentum, w.weight_decay, w.tau) == (32, 25_557_032, 20, 1, 0.9, 1e-4, 0)
    x0 = inputs.initial_x(w.scaled(1000))
    assert torch.equal(x0[0], x0[31]) and abs(float(x0.std()) - 0.1) < 0.02          # identical rows, variance 0.01
    t = inputs.WORKLOADS["transformer"]
    assert (t.n, t.d, t.peers, t.momentum, t.lr) == (16, 61_000_000, 2, 0.0, 1e-3)
    assert math.isclose(t.x0_std ** 2, 0.02) and math.isclose(t.grad_std ** 2, 1e-3)
    x0 = inputs.initial_x(t.scaled(1000))
    assert not torch.equal(x0[0], x0[1])
    o = inputs.WORKLOADS["resnet50_osgp1"]
    assert o.tau == 1 and o.weight_decay == 0.0
    s = inputs.sweep_workload(64, 10_000)
    assert (s.graph, s.max_outdeg, s.num_steps, s.K) == ("random", 4, 10, 10)
    g = torch.empty(4, 100)
    assert torch.equal(inputs.gradient(s.scaled(100), 3, g.clone()), inputs.gradient(s.scaled(100), 3, g.clone()))
