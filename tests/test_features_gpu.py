"""GPU parity of the schedule features and the fused diagnostics against the float64 oracle:
the undirected bipartite exponential graph (App. A), Alg. 2's send period (line 5), the biased-OSGP ablation
(Sec. 6.1 / Table 4) and the parameter deviation / consensus distance computed inside the step (Sec. 6.1 Fig. 2;
consensus lemma of the supplement)."""
import dataclasses

import numpy as np
import pytest
import torch

from gpu_runner import DEV, compare_with_oracle, run_gpu
from parity_util import REL_TOL, assert_close, graph_desc, oracle_P_of_k

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


# ---------------------------------------------------------------- App. A: undirected bipartite exponential graph
@pytest.mark.parametrize("n,d", [(2, 515), (8, 4_100), (16, 2_051), (32, 8_200), (64, 1_030)])
@pytest.mark.parametrize("variant", [1, 3])
def test_bipartite_exponential_graph(binding, inputs, n, d, variant):
    w = dataclasses.replace(inputs.WORKLOADS["resnet50"].scaled(d, K=7), n=n, graph="bipartite", x0_shared=False)
    out = run_gpu(binding, inputs, w, options={"variant": variant})
    compare_with_oracle(w, out)
    assert np.array_equal(out["W"], np.ones(n, dtype=np.float32))        # symmetric doubly stochastic: w == 1, z == x
    assert np.array_equal(out["Z"], out["X"])


def test_bipartite_graph_needs_even_n(binding):
    with pytest.raises(binding.SgpError) as e:
        binding.Sgp(7, 100, binding.GraphDesc.bipartite_exp())
    assert e.value.code == binding.SGP_ERR_ARG


# ---------------------------------------------------------------- Alg. 2 line 5: transmit every s-th step only
@pytest.mark.parametrize("tau,s", [(0, 2), (0, 3), (2, 2), (3, 3), (1, 2), (3, 2)])
@pytest.mark.parametrize("graph,variant", [("exp", 1), ("exp", 3), ("random", 1)])
def test_send_period(binding, inputs, tau, s, graph, variant):
    if graph == "exp":
        w = dataclasses.replace(inputs.WORKLOADS["resnet50"].scaled(256 * 11 + 4, K=11), n=8, tau=tau, x0_shared=False)
    else:
        w = dataclasses.replace(inputs.sweep_workload(16, 3_001), tau=tau, K=11)
    out = run_gpu(binding, inputs, w, options={"variant": variant, "send_period": s})
    compare_with_oracle(w, out, send_period=s)
    if tau > 0:
        assert np.ptp(out["W"]) > 1e-3 or abs(out["W"][0] - 1.0) > 1e-3


def test_send_period_idle_step_keeps_the_half_step(binding, inputs):
    """tau = 0, s = 2: on an odd step nobody transmits, so X' = X - lr * G exactly (identity mixing matrix)."""
    w = inputs.sweep_workload(16, 5_000)
    n, d = w.n, w.d
    X = inputs.initial_x(w, device=DEV).contiguous()
    W = torch.ones(n, device=DEV); Z = torch.empty_like(X); G = torch.empty_like(X)
    inputs.gradient(w, 1, G)
    want = (X.double() - float(np.float32(w.lr)) * G.double()).cpu().numpy()
    with binding.Sgp(n, d, graph_desc(w, binding)) as h:
        h.set_option("send_period", 2)
        h.step(X, W, None, G, Z, 1, w.lr, 0.0, 0.0, True)
        torch.cuda.synchronize()
        with pytest.raises(binding.SgpError):
            h.set_option("send_period", 0)
    assert_close("X", X.cpu().numpy(), want, tol=1e-6)
    assert torch.equal(Z, X) and torch.equal(W, torch.ones_like(W))


# ---------------------------------------------------------------- Table 4: biased OSGP (push-sum weight not used)
@pytest.mark.parametrize("tau,variant", [(1, 1), (1, 3), (2, 1)])
def test_biased_osgp(binding, inputs, tau, variant):
    w = dataclasses.replace(inputs.WORKLOADS["resnet50_osgp1"].scaled(256 * 9 + 8, K=9), n=8, tau=tau)
    out = run_gpu(binding, inputs, w, options={"variant": variant}, flags=binding.SGP_FLAG_BIASED)
    compare_with_oracle(w, out, biased=True)
    assert np.array_equal(out["Z"], out["X"])                           # z is the numerator itself
    assert abs(out["W"][0] - 1.0) > 0.2                                  # while w has drifted towards 2/3 (tau = 1)
    unbiased = run_gpu(binding, inputs, w, options={"variant": variant})
    assert not np.allclose(unbiased["Z"], out["Z"], rtol=1e-3, atol=1e-6)


def test_biased_standalone_debias(binding, inputs):
    w = inputs.sweep_workload(4, 1_000)
    X = inputs.initial_x(w, device=DEV).contiguous()
    W = torch.tensor([0.5, 2.0, 1.0, 0.25], device=DEV)
    Z = torch.empty_like(X)
    with binding.Sgp(4, 1_000, graph_desc(w, binding), flags=binding.SGP_FLAG_BIASED) as h:
        h.debias(X, W, Z)
        torch.cuda.synchronize()
    assert torch.equal(Z, X)
    with pytest.raises(binding.SgpError):
        binding.Sgp(4, 1_000, graph_desc(w, binding), flags=2)


# ---------------------------------------------------------------- diagnostics fused into the step
def _oracle_diagnostics(w, out, K, P_of_k=None):
    from oracle import sgp as osgp
    x0 = out["x0"].astype(np.float64)
    st = osgp.init_state(x0, w.tau)
    P_of_k = oracle_P_of_k(w) if P_of_k is None else P_of_k
    res = []
    for k in range(K):
        osgp.sgp_step(st, out["grads"][k].astype(np.float64), P_of_k(k), w.lr, w.momentum, w.nesterov, w.weight_decay)
        res.append((osgp.param_deviation(st.h), osgp.consensus_distance(st)))
    return res


DIAG_TOL = 2e-5      # norms over d terms accumulated in fp32 per warp group, fp64 above


@pytest.mark.parametrize("case", [
    dict(n=8, d=4_100, tau=0, graph="exp", variant=1),
    dict(n=8, d=4_100, tau=0, graph="exp", variant=3),
    dict(n=32, d=256 * 40 + 8, tau=0, graph="exp", variant=0),
    dict(n=32, d=256 * 40 + 8, tau=1, graph="exp", variant=1),
    dict(n=32, d=256 * 12, tau=1, graph="exp", variant=3),
    dict(n=16, d=9_001, tau=2, graph="random", variant=1),
    dict(n=16, d=9_001, tau=3, graph="random", variant=3),
    dict(n=64, d=3_000, tau=0, graph="random", variant=1),
    dict(n=256, d=1_029, tau=0, graph="random", variant=1),
    dict(n=256, d=1_029, tau=1, graph="random", variant=1),
    dict(n=7, d=2_000, tau=0, graph="complete", variant=1),
    dict(n=32, d=256 * 9, tau=0, graph="complete", variant=3),
    dict(n=5, d=1_001, tau=1, graph="random", variant=1, ld_extra=3),          # scalar path
])
def test_fused_diagnostics_match_oracle(binding, inputs, case):
    n, d, tau = case["n"], case["d"], case["tau"]
    if case["graph"] == "exp":
        w = dataclasses.replace(inputs.WORKLOADS["resnet50"].scaled(d, K=5), n=n, tau=tau, x0_shared=False)
    else:
        w = dataclasses.replace(inputs.sweep_workload(n, d), tau=tau, K=5, graph=case["graph"], weight_decay=1e-3)
    out = run_gpu(binding, inputs, w, options={"variant": case["variant"]}, want_diagnostics=True,
                  ld=d + case.get("ld_extra", 0))
    compare_with_oracle(w, out)                                          # the step itself is unchanged by the flag
    want = _oracle_diagnostics(w, out, w.K)
    for k, ((dev, cons, summary), (odev, ocons)) in enumerate(zip(out["diagnostics"], want)):
        assert_close(f"param_dev[{k}]", dev, odev, tol=DIAG_TOL)
        scale = max(np.abs(ocons).max(), 1e-6 * np.sqrt(d))
        assert np.abs(cons - ocons).max() <= DIAG_TOL * max(scale, np.abs(odev).max()), (k, cons, ocons)
        assert abs(summary["param_dev_mean"] - odev.mean()) <= DIAG_TOL * odev.max()
        assert abs(summary["param_dev_min"] - odev.min()) <= DIAG_TOL * odev.max()
        assert abs(summary["param_dev_max"] - odev.max()) <= DIAG_TOL * odev.max()
    assert np.max(want[-1][0]) > 0                                        # the nodes really differ


def test_diagnostics_results_identical_with_and_without_flag(binding, inputs):
    w = dataclasses.replace(inputs.WORKLOADS["resnet50"].scaled(256 * 33, K=3), tau=1)
    a = run_gpu(binding, inputs, w, want_diagnostics=True)
    b = run_gpu(binding, inputs, w)
    for name in ("X", "Z", "M", "W"):
        assert np.array_equal(a[name], b[name]), name


def test_diagnostics_need_a_step(binding, inputs):
    w = inputs.sweep_workload(4, 1_000)
    with binding.Sgp(4, 1_000, graph_desc(w, binding)) as h:
        with pytest.raises(binding.SgpError) as e:
            h.diagnostics()
        assert e.value.code == binding.SGP_ERR_STATE
