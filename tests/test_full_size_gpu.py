"""Parity at the full workload sizes, in the launch configuration the benchmark times.

The float64 oracle cannot run 8e8 .. 6.4e9 elements in seconds, but every column of the SGP recursion
evolves independently of every other column, so the oracle is run on sampled column windows (first
tile, an unaligned window in the middle, the ragged last tile) fed with the very fp32 bits the GPU
consumed, and compared element by element there.  Whole-array invariants (sum of weights, no
non-finite value, conserved column sums) cover the rest."""
import dataclasses

import numpy as np
import pytest
import torch

from parity_util import assert_close, graph_desc, run_oracle

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


def _windows(d):
    mid = (d // 2) | 1                                   # odd start: not vector aligned
    return [(0, min(d, 4096)), (mid, min(d, mid + 3001)), (max(0, d - 2056), d)]


def _run_full(binding, inputs, w, K, ld_align=256):
    """ld_align = 256 is the benchmark's layout (rows start on 1 KB boundaries); 1 is the dense layout."""
    n, d = w.n, w.d
    ld = (d + ld_align - 1) // ld_align * ld_align
    need = 4 * n * d * (4 + w.tau) + (2 << 30)
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < need:
        pytest.skip(f"needs {need / 2**30:.0f} GiB of device memory, {free_b / 2**30:.0f} GiB free")
    def matrix(fill):
        return torch.full((n, ld), fill, dtype=torch.float32, device=DEV)[:, :d]
    X = matrix(0.0)
    X.copy_(inputs.initial_x(w, device=DEV))
    M = matrix(0.0) if w.momentum != 0.0 else None
    Z = matrix(float("nan"))
    G = matrix(0.0)
    W = torch.ones(n, device=DEV)
    wins = _windows(d)
    x0 = [X[:, a:b].cpu().numpy().copy() for a, b in wins]
    grads = [[] for _ in wins]
    with binding.Sgp(n, d, graph_desc(w, binding), tau=w.tau, ld=ld) as h:
        for k in range(K):
            inputs.gradient(w, k, G)
            for i, (a, b) in enumerate(wins):
                grads[i].append(G[:, a:b].cpu().numpy().copy())
            if k == K - 1:
                # per-column conservation over ALL d columns for the last step (Sec. 2: 1^T P = 1^T): what the
                # columns of X plus ring must sum to follows from column sums of X, G and the new momentum
                before_all, before_x = h.colsum(X, include_ring=True), h.colsum(X)
            h.step(X, W, M, G, Z, k, w.lr, w.momentum, w.weight_decay, w.nesterov)
        s = h.colsum(G) + w.weight_decay * before_x
        if M is not None:
            s = w.momentum * h.colsum(M) + s if w.nesterov else h.colsum(M)
        ref = (before_all - w.lr * s).contiguous()
        del before_all, before_x, s
        torch.cuda.synchronize()
        assert h.device_status() == 0
        stats = h.check(X, W, colsum_ref=ref)
        sum_w, min_w, nonfinite = stats["sum_w"], stats["min_w"], stats["nonfinite"]
        del ref
    assert stats["code"] == 0 and stats["max_colsum_rel_drift"] <= 2e-6, stats
    assert abs(sum_w - n) <= 1e-4 * n and min_w > 0 and nonfinite == 0
    assert torch.isfinite(Z).all().item()
    for i, (a, b) in enumerate(wins):
        ww = w.scaled(b - a, K=K)
        st = run_oracle(ww, x0[i], grads[i], K=K)
        assert_close(f"X[{a}:{b}]", X[:, a:b].cpu().numpy(), st.x)
        assert_close(f"Z[{a}:{b}]", Z[:, a:b].cpu().numpy(), st.z)
        if M is not None:
            assert_close(f"M[{a}:{b}]", M[:, a:b].cpu().numpy(), st.u)
        assert_close("W", W.cpu().numpy(), st.w)
    del X, M, Z, G
    torch.cuda.empty_cache()


@pytest.mark.parametrize("ld_align", [256, 1])
def test_resnet50_full_size(binding, inputs, ld_align):
    _run_full(binding, inputs, inputs.WORKLOADS["resnet50"], K=20 if ld_align == 256 else 3, ld_align=ld_align)


@pytest.mark.parametrize("name,d", [("resnet50", 25_557_033), ("resnet50_osgp1", 25_557_031), ("transformer", 61_000_001)])
def test_rows_off_the_16_byte_grid_full_size(binding, inputs, name, d):
    """Dense pitch with d not a multiple of 4: rows start at every distance from a 16-byte boundary and the step runs
    the peeled kernel; same sampled windows and whole-array invariants (with the per-column conservation check over
    all d columns) as the aligned layouts."""
    _run_full(binding, inputs, dataclasses.replace(inputs.WORKLOADS[name], d=d), K=3, ld_align=1)


def test_transformer_full_size(binding, inputs):
    _run_full(binding, inputs, inputs.WORKLOADS["transformer"], K=20)


def test_resnet50_overlap_full_size(binding, inputs):
    _run_full(binding, inputs, inputs.WORKLOADS["resnet50_osgp1"], K=20)


@pytest.mark.parametrize("n,d", [(256, 10_000_000), (64, 100_000_000)])
def test_sweep_largest_points(binding, inputs, n, d):
    """More than 2^31 elements per array: 64-bit offsets everywhere."""
    _run_full(binding, inputs, inputs.sweep_workload(n, d), K=2)


def test_transformer_adam_full_size(binding, inputs):
    """Adam-SGP at the Transformer size, K = 5 steps, sampled windows."""
    from oracle import sgp as osgp
    from parity_util import oracle_P_of_k
    w = inputs.WORKLOADS["transformer_adam"]
    n, d, K = w.n, w.d, 5
    X, ld = binding.empty_matrix(n, d, device=DEV)
    X.copy_(inputs.initial_x(w, device=DEV))
    M1, _ = binding.empty_matrix(n, d, device=DEV, fill=0.0)
    M2, _ = binding.empty_matrix(n, d, device=DEV, fill=0.0)
    Z, _ = binding.empty_matrix(n, d, device=DEV, fill=float("nan"))
    G, _ = binding.empty_matrix(n, d, device=DEV)
    W = torch.ones(n, device=DEV)
    wins = _windows(d)
    x0 = [X[:, a:b].cpu().numpy().copy() for a, b in wins]
    grads = [[] for _ in wins]
    with binding.Sgp(n, d, graph_desc(w, binding), ld=ld) as h:
        for k in range(K):
            inputs.gradient(w, k, G)
            for i, (a, b) in enumerate(wins):
                grads[i].append(G[:, a:b].cpu().numpy().copy())
            if k == K - 1:
                h.set_option("check_steps", 1)     # the last step is bracketed by the per-column conservation check
            h.step_adam(X, W, M1, M2, G, Z, k, k + 1, w.lr, w.beta1, w.beta2, w.adam_eps, 0.0)
        torch.cuda.synchronize()
        assert h.device_status() == 0
    for i, (a, b) in enumerate(wins):
        st = osgp.sgp_run(x0[i].astype(np.float64), K, oracle_P_of_k(w), lambda k, z: grads[i][k].astype(np.float64),
                          w.lr, adam=(w.beta1, w.beta2, w.adam_eps))
        assert_close(f"X[{a}:{b}]", X[:, a:b].cpu().numpy(), st.x)
        assert_close(f"Z[{a}:{b}]", Z[:, a:b].cpu().numpy(), st.z)
        assert_close(f"M1[{a}:{b}]", M1[:, a:b].cpu().numpy(), st.u)
        assert_close(f"M2[{a}:{b}]", M2[:, a:b].cpu().numpy(), st.v)
    del X, M1, M2, Z, G
    torch.cuda.empty_cache()


def test_tau_full_size_mass_conservation(binding, inputs):
    """With zero gradients the total mass (state + ring) of every column is conserved by the delayed mix."""
    w = dataclasses.replace(inputs.sweep_workload(64, 3_000_001), tau=2, grad_std=0.0, momentum=0.0)
    n, d = w.n, w.d
    X = inputs.initial_x(w, device=DEV).contiguous()
    Z = torch.empty_like(X)
    G = torch.zeros_like(X)
    W = torch.ones(n, device=DEV)
    with binding.Sgp(n, d, graph_desc(w, binding), tau=2) as h:
        ref = h.colsum(X, include_ring=True).clone()
        for k in range(7):
            h.step(X, W, None, G, Z, k, w.lr, 0.0, 0.0, True)
        stats = h.check(X, W, colsum_ref=ref)
    assert stats["code"] == 0 and stats["max_colsum_rel_drift"] <= 2e-6, stats
    assert abs(stats["sum_w"] - n) <= 1e-4 * n and stats["nonfinite"] == 0


@pytest.mark.parametrize("name", ["resnet50", "resnet50_osgp1"])
def test_fused_diagnostics_full_size(binding, inputs, name):
    """The diagnostics of the full-size launch (every CTA accumulates hundreds of tiles in fp32 slots) against the same
    quantities formed from the arrays with float64 torch arithmetic on the device: properties that hold at any size.
    Parameter deviation (Sec. 6.1): || h_i - mean_j h_j || with h = x - lr (m u' + g + wd x) rebuilt from the state
    before the step and the momentum after it; consensus distance: || z_i - xbar ||, xbar = (colsum(X') + ring') / n."""
    w = inputs.WORKLOADS[name]
    n, d = w.n, w.d
    X, ld = binding.empty_matrix(n, d, device=DEV)
    X.copy_(inputs.initial_x(w, device=DEV))
    M, _ = binding.empty_matrix(n, d, device=DEV, fill=0.0)
    Z, _ = binding.empty_matrix(n, d, device=DEV, fill=float("nan"))
    G, _ = binding.empty_matrix(n, d, device=DEV)
    W = torch.ones(n, device=DEV)
    with binding.Sgp(n, d, binding.graph_desc(w), tau=w.tau, ld=ld) as h:
        for k in range(3):
            inputs.gradient(w, k, G)
            X += 0.01 * torch.arange(n, device=DEV, dtype=torch.float32)[:, None] if k == 0 else 0.0   # nodes differ
            if k == 2:
                h.set_option("diagnostics", 1)
                X_before = X.clone()
            h.step(X, W, M, G, Z, k, w.lr, w.momentum, w.weight_decay, True)
        dev, cons, summary = h.diagnostics()
        colsum_after = h.colsum(X, include_ring=True)
        assert h.device_status() == 0
    lr, m, wd = (float(np.float32(v)) for v in (w.lr, w.momentum, w.weight_decay))
    want_dev = torch.zeros(n, dtype=torch.float64, device=DEV)
    want_cons = torch.zeros(n, dtype=torch.float64, device=DEV)
    step = 1 << 21
    for c0 in range(0, d, step):
        c1 = min(d, c0 + step)
        xb, g, mu = X_before[:, c0:c1].double(), G[:, c0:c1].double(), M[:, c0:c1].double()
        hh = xb - lr * (m * mu + g + wd * xb)
        want_dev += ((hh - hh.mean(dim=0, keepdim=True)) ** 2).sum(dim=1)
        xbar = colsum_after[c0:c1] / n
        want_cons += ((Z[:, c0:c1].double() - xbar[None, :]) ** 2).sum(dim=1)
    want_dev, want_cons = want_dev.sqrt().cpu().numpy(), want_cons.sqrt().cpu().numpy()
    assert np.abs(dev - want_dev).max() <= 2e-5 * want_dev.max(), (dev[:4], want_dev[:4])
    assert np.abs(cons - want_cons).max() <= 2e-5 * max(want_cons.max(), want_dev.max()), (cons[:4], want_cons[:4])
    assert abs(summary["param_dev_max"] - want_dev.max()) <= 2e-5 * want_dev.max()
    assert want_dev.min() > 0
    del X, M, Z, G, X_before
    torch.cuda.empty_cache()
