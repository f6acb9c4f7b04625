"""Many steps in a row with the per-step conservation bracket on (option check_steps: the column sums of X plus ring
after every step against those of the half step, Sec. 2, 1^T P = 1^T): a lost update, a tile taken twice, a slot of the
delay ring consumed late or a weight committed by the wrong CTA shows as a drift bit in the device status word.  Every
kernel family and launch mode runs at a size that fills the device for several tiles per CTA."""
import dataclasses

import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def binding():
    from paper_1811_10792_b200 import build
    build.build()
    from paper_1811_10792_b200 import binding as b
    return b


@pytest.fixture(scope="module")
def inputs():
    from paper_1811_10792_b200 import inputs as i
    return i


CASES = {
    # name: (workload, d, ld alignment in floats, options, expected kernel family, expected lockstep cluster)
    "pipelined": ("resnet50", 2_000_008, 256, {}, 3, 0),
    "register_staged": ("resnet50", 2_000_008, 256, {"variant": 1}, 1, 0),
    "lockstep_pairs_dense_pitch": ("resnet50", 2_000_008, 1, {}, 1, 2),
    "delay_ring_lockstep": ("resnet50_osgp1", 2_000_008, 256, {}, 1, 2),
    "delay_two_dense_pitch": ("resnet50_osgp1", 2_000_008, 1, {"tau": 2}, 1, 2),
    "plain_sgd_pipelined": ("transformer", 4_000_000, 256, {}, 3, 0),
    "adam": ("transformer_adam", 4_000_000, 256, {}, 1, 0),
    "peeled": ("resnet50", 2_000_009, 1, {}, 5, 0),
    "peeled_delay_ring": ("resnet50_osgp1", 2_000_007, 1, {}, 5, 0),
    "fused_diagnostics": ("resnet50", 2_000_008, 256, {"diagnostics": 1}, 1, 0),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_three_hundred_checked_steps(binding, inputs, name):
    wname, d, ld_align, options, want_variant, want_lockstep = CASES[name]
    options = dict(options)
    w = dataclasses.replace(inputs.WORKLOADS[wname], d=d)
    if "tau" in options:
        w = dataclasses.replace(w, tau=options.pop("tau"))
    n = w.n
    ld = (d + ld_align - 1) // ld_align * ld_align
    def matrix():
        return torch.zeros((n, ld), device=DEV)[:, :d]
    X = matrix()
    X.copy_(inputs.initial_x(w, device=DEV))
    adam = w.optimizer == "adam"
    M, V, Z, W = matrix(), (matrix() if adam else None), matrix(), torch.ones(n, device=DEV)
    G = [inputs.gradient(w, k, matrix()) for k in range(3)]
    with binding.Sgp(n, d, binding.graph_desc(w), tau=w.tau, ld=ld) as h:
        for key, val in options.items():
            h.set_option(key, val)
        h.set_option("check_steps", 1)
        for k in range(300):
            if adam:
                h.step_adam(X, W, M, V, G[k % 3], Z, k, k + 1, 1e-3, 0.9, 0.98, 1e-8, 0.0)
            else:
                h.step(X, W, M if w.momentum else None, G[k % 3], Z, k, 1e-3, w.momentum, w.weight_decay, w.nesterov)
        torch.cuda.synchronize()
        assert h.device_status() == 0
        assert h.get_option("last_variant") == want_variant and h.get_option("last_lockstep") == want_lockstep
        stats = h.check(X, W)
        assert stats["code"] == binding.SGP_OK and stats["nonfinite"] == 0 and abs(stats["sum_w"] - n) < 1e-4 * n


@pytest.mark.parametrize("tau,period", [(0, 1), (1, 1), (2, 1), (3, 2)])
def test_two_hundred_steps_one_node_per_gpu_equal_the_stacked_step(binding, inputs, tau, period):
    """The message slots of the one-node-per-GPU mode are reused every tau + 2 steps: after 200 steps on a random
    digraph (weights away from 1) the loopback ranks still hold the stacked step's bits."""
    from test_rowshard_gpu import _run_both
    w = dataclasses.replace(inputs.sweep_workload(12, 20_004), tau=tau, weight_decay=1e-4, lr=0.01)
    _x0, _grads, got, stacked = _run_both(binding, inputs, w, 200, send_period=period)
    for name in ("X", "Z", "M", "W"):
        assert torch.equal(got[name], stacked[name]), name
    assert float(got["W"].max() - got["W"].min()) > 1e-3
