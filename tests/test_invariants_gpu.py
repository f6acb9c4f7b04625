"""sgp_check / sgp_colsum: the invariants of column-stochastic mixing, checked per column on the GPU.

Sec. 2: every column of P^(k) sums to one, so the mix conserves sum_i w_i and, coordinate by coordinate,
sum_i x_i -- counting the messages in transit of the delay model (the virtual nodes).  All failures here are
injected on the host side (a corrupted element, a zero weight, a NaN, a withheld tile request): nothing
faults, traps or hangs."""
import dataclasses

import numpy as np
import pytest
import torch

from gpu_runner import DEV
from parity_util import assert_close, graph_desc, oracle_P_of_k

pytestmark = pytest.mark.gpu


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


def _state(inputs, w):
    X = inputs.initial_x(w, device=DEV).contiguous()
    return X, torch.ones(w.n, device=DEV), torch.zeros_like(X), torch.empty_like(X), torch.empty_like(X)


def _expected_colsum(h, w, X, G, M_after, col_before_all, col_before_x):
    """Column sums X' + ring' must have: sum_i h_i + ring, h = x - lr * s, linear in the column sums."""
    col_g = h.colsum(G)
    s = col_g + w.weight_decay * col_before_x
    if w.momentum != 0.0:
        col_m = h.colsum(M_after)
        s = w.momentum * col_m + s if w.nesterov else col_m
    return (col_before_all - w.lr * s).contiguous()


@pytest.mark.parametrize("tau", [0, 1, 3])
@pytest.mark.parametrize("n,d", [(16, 40_037), (64, 9_001), (256, 1_029)])
def test_clean_run_conserves_every_column(binding, inputs, n, d, tau):
    from oracle import sgp as osgp
    w = dataclasses.replace(inputs.sweep_workload(n, d), tau=tau, weight_decay=1e-3)
    X, W, M, Z, G = _state(inputs, w)
    x0 = X.cpu().numpy().astype(np.float64)
    grads = []
    with binding.Sgp(n, d, graph_desc(w, binding), tau=tau) as h:
        for k in range(5):
            inputs.gradient(w, k, G)
            grads.append(G.cpu().numpy().astype(np.float64))
            before_all, before_x = h.colsum(X, include_ring=True), h.colsum(X)
            h.step(X, W, M, G, Z, k, w.lr, w.momentum, w.weight_decay, True)
            ref = _expected_colsum(h, w, X, G, M, before_all, before_x)
            stats = h.check(X, W, colsum_ref=ref)
            assert stats["code"] == binding.SGP_OK and stats["status"] == 0
            assert stats["max_colsum_rel_drift"] <= 2e-6 and stats["nonfinite"] == 0
            assert stats["sum_w_drift"] <= 1e-5 * n and stats["min_w"] > 0
        after = h.colsum(X, include_ring=True).cpu().numpy()
    st = osgp.sgp_run(x0, 5, oracle_P_of_k(w), lambda k, z: grads[k], w.lr, momentum=w.momentum, nesterov=True,
                      weight_decay=w.weight_decay, tau=tau)
    mass, sum_w = osgp.total_mass(st)
    assert_close("column mass", after, mass)
    assert abs(stats["sum_w"] - sum_w) <= 1e-5 * n
    assert abs(stats["total"] - mass.sum()) <= 1e-6 * np.abs(st.x).sum()


def test_one_corrupted_column_is_reported(binding, inputs):
    w = dataclasses.replace(inputs.sweep_workload(32, 70_001), tau=1, grad_std=0.0, momentum=0.0)
    n, d = w.n, w.d
    X, W, _, Z, G = _state(inputs, w)
    G.zero_()
    with binding.Sgp(n, d, graph_desc(w, binding), tau=1) as h:
        ref = h.colsum(X, include_ring=True).clone()                     # zero gradients: the sums must not move
        for k in range(4):
            h.step(X, W, None, G, Z, k, w.lr, 0.0, 0.0, True)
        ok = h.check(X, W, colsum_ref=ref)
        assert ok["code"] == binding.SGP_OK and ok["max_colsum_rel_drift"] <= 2e-6
        # a sign error confined to two columns: the grand total is unchanged, the per-column check is not fooled
        X[5, 12_345] += 0.5
        X[9, 54_321] -= 0.5
        bad = h.check(X, W, colsum_ref=ref, raise_on_error=False)
        assert bad["code"] == binding.SGP_ERR_INVARIANT
        assert abs(bad["max_colsum_drift"] - 0.5) < 1e-3 and bad["max_colsum_rel_drift"] > 1e-2
        assert abs(bad["total"] - ok["total"]) <= 1e-7 * abs(ok["total"]) + 1e-6
        assert int(bad["status"]) & binding.SGP_STATUS_COLUMN_SUM
        assert h.device_status() & binding.SGP_STATUS_COLUMN_SUM
        h.reset()
        assert h.device_status() == 0


def test_zero_weight_is_an_error_code_and_never_an_inf(binding, inputs):
    w = inputs.sweep_workload(8, 3_000)
    n, d = w.n, w.d
    X, W, M, Z, G = _state(inputs, w)
    inputs.gradient(w, 0, G)
    with binding.Sgp(n, d, graph_desc(w, binding)) as h:
        W[3] = 0.0
        res = h.check(X, W, raise_on_error=False)
        assert res["code"] == binding.SGP_ERR_ZERO_WEIGHT and res["min_w"] == 0.0
        assert int(res["status"]) & binding.SGP_STATUS_ZERO_WEIGHT
        h.reset()
        # every weight zero: the mixed weights are zero too; z is written as 0, not inf or NaN
        W.zero_()
        h.step(X, W, M, G, Z, 0, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
        assert torch.isfinite(Z).all().item() and torch.count_nonzero(Z).item() == 0
        assert h.device_status() & binding.SGP_STATUS_ZERO_WEIGHT
        with pytest.raises(binding.SgpError) as e:                       # the handle refuses to go on until reset
            h.step(X, W, M, G, Z, 1, w.lr, w.momentum, 0.0, True)
        assert e.value.code == binding.SGP_ERR_ZERO_WEIGHT
        Zd = torch.empty_like(X)
        h.debias(X, W, Zd)
        torch.cuda.synchronize()
        assert torch.count_nonzero(Zd).item() == 0
        h.reset()
        W.fill_(1.0)
        h.step(X, W, M, G, Z, 1, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
        assert h.device_status() == 0 and torch.isfinite(Z).all().item()
        W[0] = float("nan")
        res = h.check(X, W, raise_on_error=False)
        assert res["code"] == binding.SGP_ERR_ZERO_WEIGHT and res["min_w"] == -1.0


def test_non_finite_entries_are_counted(binding, inputs):
    w = dataclasses.replace(inputs.sweep_workload(4, 10_000), tau=2)
    n, d = w.n, w.d
    X, W, M, Z, G = _state(inputs, w)
    inputs.gradient(w, 0, G)
    with binding.Sgp(n, d, graph_desc(w, binding), tau=2) as h:
        h.step(X, W, M, G, Z, 0, w.lr, w.momentum, 0.0, True)
        assert h.check(X, W)["nonfinite"] == 0
        X[2, 77] = float("inf")
        X[0, 9_999] = float("nan")
        res = h.check(X, W, raise_on_error=False)
        assert res["code"] == binding.SGP_ERR_INVARIANT and res["nonfinite"] == 2
        assert int(res["status"]) & binding.SGP_STATUS_NONFINITE


@pytest.mark.parametrize("optimizer,tau,variant", [("nesterov", 0, 1), ("nesterov", 2, 1), ("heavy", 1, 1),
                                                   ("sgd", 0, 3), ("nesterov", 0, 3), ("adam", 1, 1)])
def test_check_steps_option_brackets_every_step(binding, inputs, optimizer, tau, variant):
    """Debug mode: sum_i x_i' plus ring against sum_i h_i plus ring, on the device, every step."""
    w = dataclasses.replace(inputs.WORKLOADS["resnet50"].scaled(256 * 301 + 12, K=4), tau=tau)
    n, d = w.n, w.d
    X, W, M, Z, G = _state(inputs, w)
    V2 = torch.zeros_like(X)
    with binding.Sgp(n, d, graph_desc(w, binding), tau=tau) as h:
        h.set_option("variant", variant)
        h.set_option("check_steps", 1)
        for k in range(4):
            inputs.gradient(w, k, G)
            if optimizer == "adam":
                h.step_adam(X, W, M, V2, G, Z, k, k + 1, 1e-2, 0.9, 0.98, 1e-8, 1e-3)
            elif optimizer == "sgd":
                h.step(X, W, None, G, Z, k, w.lr, 0.0, w.weight_decay, True)
            else:
                h.step(X, W, M, G, Z, k, w.lr, 0.9, w.weight_decay, optimizer == "nesterov")
        assert h.device_status() == 0
        assert h.get_option("check_steps") == 1


def test_check_steps_sees_a_tile_that_was_never_mixed(binding, inputs):
    """Host-side injection: one tile request of the pipelined kernel is withheld (bounded wait, no hang), so
    those columns keep x instead of the mixed half step and the bracketed check reports the drift."""
    w = inputs.WORKLOADS["resnet50"].scaled(256 * 600, K=1)
    n, d = w.n, w.d
    X, W, M, Z, G = _state(inputs, w)
    inputs.gradient(w, 0, G)
    with binding.Sgp(n, d, graph_desc(w, binding)) as h:
        h.set_option("variant", 3)
        h.set_option("wait_limit_ms", 200)
        h.set_option("inject_stall", 1)
        h.set_option("check_steps", 1)
        h.step(X, W, M, G, Z, 0, w.lr, w.momentum, w.weight_decay, True)
        status = h.device_status()
        assert status & binding.SGP_STATUS_WAIT_TILE and status & binding.SGP_STATUS_COLUMN_SUM
        with pytest.raises(binding.SgpError) as e:
            h.step(X, W, M, G, Z, 1, w.lr, w.momentum, w.weight_decay, True)
        assert e.value.code == binding.SGP_ERR_DEVICE
        h.reset()
        h.set_option("inject_stall", 0)
        X2, W2, M2, Z2, _ = _state(inputs, w)
        h.step(X2, W2, M2, G, Z2, 0, w.lr, w.momentum, w.weight_decay, True)
        assert h.device_status() == 0
