"""GPU parity: the fused CUDA step (through the C ABI) against the float64 oracle, element by element,
on the same seeded inputs.  Sizes span several column tiles and a ragged tail; the w != 1 cases
(irregular graphs, delayed messages) are included because regular graphs cannot detect a broken
weight path."""
import dataclasses
from fractions import Fraction

import numpy as np
import pytest
import torch

from conftest import read_golden
from parity_util import REL_TOL, assert_close, graph_desc, oracle_P_of_k, run_oracle

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


from gpu_runner import compare_with_oracle as _compare, run_gpu as _run_gpu


# ------------------------------------------------------------------ the five workload configurations, oracle-sized
def test_config1_tiny_closed_loop(binding, inputs):
    """n=8, d=4096, K=100, one-peer graph, Nesterov; g = z - c + noise computed from each side's OWN z."""
    from oracle import sgp as osgp
    w = inputs.WORKLOADS["tiny"]
    n, d, K = w.n, w.d, w.K
    c = inputs.normal(n, d, seed=w.seed, stream=inputs.STREAM_TARGET, step=0, std=1.0, device=DEV)
    noise = [inputs.normal(n, d, seed=w.seed, stream=inputs.STREAM_NOISE, step=k, std=0.1, device=DEV) for k in range(K)]
    X = torch.zeros((n, d), device=DEV)
    W = torch.ones(n, device=DEV)
    M = torch.zeros_like(X)
    Z = X.clone()
    with binding.Sgp(n, d, binding.GraphDesc.exp_peers(1)) as h:
        for k in range(K):
            G = Z - c + noise[k]                      # harness arithmetic (gradient oracle), not the SGP path
            h.step(X, W, M, G, Z, k, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
    c64 = c.cpu().numpy().astype(np.float64)
    nz = [t.cpu().numpy().astype(np.float64) for t in noise]
    st = osgp.sgp_run(np.zeros((n, d)), K, oracle_P_of_k(w), lambda k, z: z - c64 + nz[k], w.lr, momentum=w.momentum,
                      nesterov=True)
    assert_close("X", X.cpu().numpy(), st.x)
    assert_close("Z", Z.cpu().numpy(), st.z)
    assert_close("M", M.cpu().numpy(), st.u)
    assert np.array_equal(W.cpu().numpy(), np.ones(n, dtype=np.float32))
    # the run really optimises: consensus around mean(c)
    assert np.abs(st.z.mean(axis=0) - c64.mean(axis=0)).max() < 0.2


@pytest.mark.parametrize("d", [8200, 128 * 37, 1000])
def test_config2_resnet_recipe_scaled(binding, inputs, d):
    w = inputs.WORKLOADS["resnet50"].scaled(d)
    out = _run_gpu(binding, inputs, w)
    st = _compare(w, out)
    assert np.array_equal(out["W"], np.ones(w.n, dtype=np.float32))      # regular graph


@pytest.mark.parametrize("d", [256 * 9 + 12, 5000])
def test_config3_transformer_recipe_scaled(binding, inputs, d):
    w = inputs.WORKLOADS["transformer"].scaled(d)
    out = _run_gpu(binding, inputs, w)
    _compare(w, out)
    assert np.all(np.isnan(out["M"]) | (out["M"] == 0))                  # plain SGD never touches M


@pytest.mark.parametrize("tau", [1, 2, 3])
def test_config4_overlap_scaled(binding, inputs, tau):
    import dataclasses
    w = dataclasses.replace(inputs.WORKLOADS["resnet50_osgp1"].scaled(4104, K=20), tau=tau)
    out = _run_gpu(binding, inputs, w)
    st = _compare(w, out)
    assert abs(out["W"][0] - 1.0) > 0.2                                  # mass in transit: w != 1


@pytest.mark.parametrize("n", [4, 16, 64, 256])
@pytest.mark.parametrize("d", [10_000, 1029])
def test_config5_sweep_points(binding, inputs, n, d):
    w = inputs.sweep_workload(n, d)
    out = _run_gpu(binding, inputs, w)
    _compare(w, out)
    assert np.ptp(out["W"]) > 1e-3                                       # irregular graph: weights differ


@pytest.mark.parametrize("tau", [0, 2])
def test_random_graph_with_delay_and_weight_decay(binding, inputs, tau):
    import dataclasses
    w = dataclasses.replace(inputs.sweep_workload(16, 3000), tau=tau, weight_decay=1e-2, K=13)
    out = _run_gpu(binding, inputs, w)
    _compare(w, out)


# ------------------------------------------------------------------ degenerate and ragged shapes
@pytest.mark.parametrize("n", [1, 2, 3, 5, 8])
@pytest.mark.parametrize("d", [1, 3, 4, 5, 127, 128, 129])
def test_small_shapes(binding, inputs, n, d):
    w = inputs.Workload("small", n=n, d=d, K=5, graph="exp", peers=1, lr=0.1, momentum=0.9, weight_decay=1e-3)
    out = _run_gpu(binding, inputs, w)
    _compare(w, out)


@pytest.mark.parametrize("ld_extra,offset", [(0, 0), (4, 0), (3, 0), (0, 1), (8, 4)])
def test_pitch_and_alignment_paths(binding, inputs, ld_extra, offset):
    """ld > d, ld not a multiple of 4 and pointers off 16-byte alignment: vector and scalar paths, same numbers."""
    w = inputs.sweep_workload(16, 2052)
    out = _run_gpu(binding, inputs, w, ld=w.d + ld_extra, offset=offset)
    _compare(w, out)


def test_without_z_and_heavy_ball(binding, inputs):
    import dataclasses
    w = dataclasses.replace(inputs.sweep_workload(16, 2500), nesterov=False)
    out = _run_gpu(binding, inputs, w, write_z=False)
    _compare(w, out, write_z=False)
    assert np.all(np.isnan(out["Z"]))                                    # Z = NULL: never written


def test_complete_graph_is_parallel_sgd(binding, inputs):
    """All-to-all mixing with n = 256 (table read from global memory in place); identical init => AllReduce SGD."""
    w = inputs.Workload("complete", n=256, d=520, K=4, graph="complete", lr=0.1, momentum=0.0, x0_shared=True)
    out = _run_gpu(binding, inputs, w)
    _compare(w, out)
    want = out["x0"][0].astype(np.float64)
    for g in out["grads"]:
        want = want - w.lr * g.astype(np.float64).mean(axis=0)
    assert_close("Z vs parallel SGD", out["Z"], np.broadcast_to(want, out["Z"].shape))


def test_custom_four_node_graph_weights_converge(binding, inputs):
    """The paper's worked 4-node matrix as a custom schedule: w -> (8,16,16,12)/13 and z -> average."""
    rows = read_golden("four_node_update_equations.txt")
    recv = [int(r[0]) for r in rows]; send = [int(r[1]) for r in rows]; wt = [float(Fraction(r[2])) for r in rows]
    g = binding.GraphDesc.custom(1, [0] * len(rows), send, recv, wt)
    from oracle import schedule as osched
    P = osched.custom_mixing_matrix(4, send, recv, np.asarray(wt, dtype=np.float32))
    w = inputs.Workload("four", n=4, d=300, K=60, graph="custom", lr=0.0, momentum=0.0, grad_std=0.0)
    out = _run_gpu(binding, inputs, w, graph=g)
    _compare(w, out, P_of_k=lambda k: P)
    assert np.allclose(out["W"], np.array([8, 16, 16, 12]) / 13.0, rtol=1e-5)
    assert np.allclose(out["Z"], np.broadcast_to(out["x0"].astype(np.float64).mean(axis=0), out["Z"].shape),
                       rtol=0, atol=2e-6)


def test_one_peer_consensus_on_gpu(binding, inputs):
    """Zero gradients, n = 32: after log2(n) = 5 fused steps every node holds the average (fp32 rounding only)."""
    w = inputs.Workload("consensus", n=32, d=1000, K=5, graph="exp", peers=1, lr=0.1, momentum=0.9, grad_std=0.0)
    out = _run_gpu(binding, inputs, w)
    mean = out["x0"].astype(np.float64).mean(axis=0)
    assert np.abs(out["Z"] - mean).max() <= 4e-7 * np.abs(out["x0"]).max()


def test_tile_and_grid_options_do_not_change_results(binding, inputs):
    w = inputs.sweep_workload(16, 5000)
    base = _run_gpu(binding, inputs, w)
    for opts in ({"tile_cols": 32}, {"tile_cols": 1024}, {"ctas_per_sm": 1}, {"ctas_per_sm": 4}):
        other = _run_gpu(binding, inputs, w, options=opts)
        for name in ("X", "W", "M", "Z"):
            assert np.array_equal(base[name], other[name], equal_nan=True), (opts, name)


def test_standalone_debias(binding, inputs):
    from oracle import sgp as osgp
    for n, d, ld, off in ((5, 1027, 1027, 0), (16, 4096, 4100, 0), (3, 10, 12, 1)):
        buf = torch.randn(n * ld + off + 4, device=DEV)
        X = buf[off:off + n * ld].view(n, ld)[:, :d]
        W = torch.rand(n, device=DEV) + 0.5
        zb = torch.full((n * ld + off + 4,), float("nan"), device=DEV)
        Z = zb[off:off + n * ld].view(n, ld)[:, :d]
        with binding.Sgp(n, d, binding.GraphDesc.exp_peers(1), ld=ld) as h:
            h.debias(X, W, Z)
            torch.cuda.synchronize()
        assert_close("Z", Z.cpu().numpy(), osgp.debias(X.cpu().numpy(), W.cpu().numpy()))
        assert torch.isnan(zb).sum().item() == zb.numel() - n * d


def test_ring_export_import_resumes_bit_exactly(binding, inputs):
    import dataclasses
    w = dataclasses.replace(inputs.sweep_workload(8, 1500), tau=2, K=9)
    n, d = w.n, w.d
    def fresh():
        return (inputs.initial_x(w, device=DEV).contiguous(), torch.ones(n, device=DEV), torch.zeros((n, d), device=DEV),
                torch.empty((n, d), device=DEV))
    G = torch.empty((n, d), device=DEV)
    X, W, M, Z = fresh()
    with binding.Sgp(n, d, graph_desc(w, binding), tau=2) as h:
        for k in range(9):
            h.step(X, W, M, inputs.gradient(w, k, G), Z, k, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
    X2, W2, M2, Z2 = fresh()
    rx = torch.empty((2, n, d), device=DEV); rw = torch.empty((2, n), device=DEV)
    with binding.Sgp(n, d, graph_desc(w, binding), tau=2) as h:
        for k in range(4):
            h.step(X2, W2, M2, inputs.gradient(w, k, G), Z2, k, w.lr, w.momentum, 0.0, True)
        h.ring_export(rx, rw)
        torch.cuda.synchronize()
    with binding.Sgp(n, d, graph_desc(w, binding), tau=2) as h:
        h.ring_import(rx, rw)
        for k in range(4, 9):
            h.step(X2, W2, M2, inputs.gradient(w, k, G), Z2, k, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
    for a, b in ((X, X2), (W, W2), (M, M2), (Z, Z2)):
        assert torch.equal(a, b)
    with binding.Sgp(n, d, graph_desc(w, binding), tau=0) as h:
        with pytest.raises(binding.SgpError) as ei:
            h.ring_export(rx, rw)
        assert ei.value.code == binding.SGP_ERR_STATE


@pytest.mark.parametrize("d", [50_004, 50_005])
def test_step_host_matches_device_step(binding, inputs, d):
    """Host-buffer entry point (chunked copy/compute pipeline) == device entry point, bit for bit; d = 50,005 with the
    dense pitch puts the rows off the 16-byte grid, so every chunk runs the peeled kernel from its own first column."""
    import dataclasses
    for tau in (0, 1):
        w = dataclasses.replace(inputs.sweep_workload(16, d), tau=tau, K=4)
        n, d = w.n, w.d
        X = inputs.initial_x(w, device=DEV).contiguous(); W = torch.ones(n, device=DEV)
        M = torch.zeros((n, d), device=DEV); Z = torch.empty((n, d), device=DEV); G = torch.empty((n, d), device=DEV)
        X2, W2, M2 = X.clone(), W.clone(), M.clone()
        dG = torch.empty((n, d), device=DEV); dZ = torch.empty((n, d), device=DEV)
        hG = torch.empty((n, d), pin_memory=True); hZ = torch.empty((n, d), pin_memory=True)
        with binding.Sgp(n, d, graph_desc(w, binding), tau=tau) as h1, binding.Sgp(n, d, graph_desc(w, binding), tau=tau) as h2:
            for k in range(w.K):
                inputs.gradient(w, k, G)
                hG.copy_(G)
                h1.step(X, W, M, G, Z, k, w.lr, w.momentum, 0.0, True)
                torch.cuda.synchronize()
                h2.step_host(X2, W2, M2, hG, hZ, dG, dZ, k, w.lr, w.momentum, 0.0, True, chunk_cols=8192)
                assert torch.equal(hZ, Z.cpu())
        assert torch.equal(X, X2) and torch.equal(W, W2) and torch.equal(M, M2)


def test_step_host_default_chunking_ramps_and_matches_device_step(binding, inputs):
    """With the default chunk width the pipeline starts and ends on narrower chunks (n = 256: 8 K, 16 K, 32 K columns,
    then 64 K): more launches than equal chunks would need, the same bits as the device entry point."""
    import dataclasses
    for tau in (0, 1):
        w = dataclasses.replace(inputs.sweep_workload(256, 300_004), tau=tau, K=2)
        n, d = w.n, w.d
        X = inputs.initial_x(w, device=DEV).contiguous(); W = torch.ones(n, device=DEV)
        M = torch.zeros((n, d), device=DEV); Z = torch.empty((n, d), device=DEV); G = torch.empty((n, d), device=DEV)
        X2, W2, M2 = X.clone(), W.clone(), M.clone()
        dG = torch.empty((n, d), device=DEV); dZ = torch.empty((n, d), device=DEV)
        hG = torch.empty((n, d), pin_memory=True); hZ = torch.empty((n, d), pin_memory=True)
        with binding.Sgp(n, d, graph_desc(w, binding), tau=tau) as h1, binding.Sgp(n, d, graph_desc(w, binding), tau=tau) as h2:
            for k in range(w.K):
                inputs.gradient(w, k, G)
                hG.copy_(G)
                h1.step(X, W, M, G, Z, k, w.lr, w.momentum, 0.0, True)
                torch.cuda.synchronize()
                before = h2.get_option("launches")
                h2.step_host(X2, W2, M2, hG, hZ, dG, dZ, k, w.lr, w.momentum, 0.0, True)
                assert h2.get_option("launches") - before >= 8          # equal 64 K chunks would be 5
                assert torch.equal(hZ, Z.cpu())
            assert h2.device_status() == 0
        assert torch.equal(X, X2) and torch.equal(W, W2) and torch.equal(M, M2)


def test_invalid_step_arguments(binding, inputs):
    n, d = 4, 64
    X = torch.zeros((n, d), device=DEV); W = torch.ones(n, device=DEV); G = torch.zeros((n, d), device=DEV)
    lib = binding.lib()
    with binding.Sgp(n, d, binding.GraphDesc.exp_peers(1)) as h:
        p = lambda t: t.data_ptr()
        assert lib.sgp_step(h._h, p(X), p(W), None, p(G), None, -1, 0.1, 0.0, 0.0, 1, None) == binding.SGP_ERR_ARG
        assert lib.sgp_step(h._h, p(X), p(W), None, p(G), None, 0, 0.1, 0.9, 0.0, 1, None) == binding.SGP_ERR_ARG
        assert lib.sgp_step(h._h, None, p(W), None, p(G), None, 0, 0.1, 0.0, 0.0, 1, None) == binding.SGP_ERR_ARG
        with pytest.raises(binding.SgpError):
            h.set_option("no_such_knob", 1)
        h.set_option("ctas_per_sm", 3)
        assert h.get_option("ctas_per_sm") == 3


# ------------------------------------------------------------------ bulk-copy pipelined kernel (variant 2)
def _tma_cases(inputs):
    import dataclasses
    W = inputs.WORKLOADS
    return [
        W["resnet50"].scaled(8200),
        W["resnet50"].scaled(128 * 700 + 4, K=7),
        W["transformer"].scaled(256 * 9 + 12),
        dataclasses.replace(W["resnet50_osgp1"].scaled(4104, K=20), tau=1),
        dataclasses.replace(W["resnet50_osgp1"].scaled(4104, K=9), tau=3),
        inputs.sweep_workload(4, 10_000), inputs.sweep_workload(16, 10_000),
        inputs.sweep_workload(64, 10_000), inputs.sweep_workload(256, 10_000),
        dataclasses.replace(inputs.sweep_workload(5, 516), nesterov=False),
        inputs.Workload("one", n=1, d=4, K=3, graph="exp", lr=0.1, momentum=0.9),
    ]


@pytest.mark.parametrize("case", range(11))
@pytest.mark.parametrize("opts", [{"variant": 2}, {"variant": 2, "stages": 4, "ctas_per_sm": 1},
                                  {"variant": 2, "stages": 3, "tile_cols": 64}, {"variant": 3},
                                  {"variant": 3, "stages": 3, "tile_cols": 512, "ctas_per_sm": 1}])
def test_bulk_copy_kernel_matches_oracle_and_register_kernel(binding, inputs, case, opts):
    w = _tma_cases(inputs)[case]
    ref = _run_gpu(binding, inputs, w, options={"variant": 1})
    out = _run_gpu(binding, inputs, w, options=opts)
    _compare(w, out)
    for name in ("X", "W", "M", "Z"):
        assert np.array_equal(ref[name], out[name], equal_nan=True), name     # same FMA order: same bits
    if w.tau > 0:
        assert np.array_equal(ref["ring"][0], out["ring"][0]) and np.array_equal(ref["ring"][1], out["ring"][1])


def test_bulk_copy_kernel_with_row_pitch(binding, inputs):
    w = inputs.sweep_workload(16, 2052)
    for variant in (2, 3):
        out = _run_gpu(binding, inputs, w, ld=w.d + 8, offset=4, options={"variant": variant})
        _compare(w, out)


def test_param_deviation_matches_oracle(binding, inputs):
    from oracle import sgp as osgp
    for n, d, pitch in ((32, 10_007, 256), (5, 300, 1), (256, 1029, 1), (16, 65_536, 256)):
        A, ld = binding.empty_matrix(n, d, device=DEV, pitch_multiple=pitch, fill=float("nan"))
        inputs.fill_normal(A, seed=77, stream=1, step=0, std=0.5)
        A += torch.linspace(-1, 1, n, device=DEV)[:, None]            # nodes really differ
        with binding.Sgp(n, d, binding.GraphDesc.exp_peers(1), ld=ld) as h:
            got = h.param_deviation(A)
        want = osgp.param_deviation(A.cpu().numpy())
        assert np.allclose(got, want, rtol=2e-6), (n, d, np.abs(got / want - 1).max())
    A, ld = binding.empty_matrix(8, 1000, device=DEV)
    A[:] = torch.randn(1000, device=DEV)
    with binding.Sgp(8, 1000, binding.GraphDesc.exp_peers(1), ld=ld) as h:
        assert np.all(h.param_deviation(A) <= 1e-5)                   # consensus: zero deviation


@pytest.mark.parametrize("variant,lockstep", [(1, 0), (3, 0), (1, 2), (1, 4)])
def test_steps_can_be_captured_in_a_cuda_graph(binding, inputs, variant, lockstep):
    """One schedule period captured once and replayed: same bits as eager launches (launch-bound small cases); the
    cluster launches of the lockstep mode are captured like any other."""
    w = inputs.sweep_workload(16, 10_000)
    n, d = w.n, w.d
    period = 10
    def fresh():
        return (inputs.initial_x(w, device=DEV).contiguous(), torch.ones(n, device=DEV), torch.zeros((n, d), device=DEV),
                torch.empty((n, d), device=DEV))
    G = [inputs.gradient(w, k, torch.empty((n, d), device=DEV)) for k in range(period)]
    X, W, M, Z = fresh()
    with binding.Sgp(n, d, graph_desc(w, binding)) as h:
        h.set_option("variant", variant)
        for rep in range(2):
            for k in range(period):
                h.step(X, W, M, G[k], Z, rep * period + k, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
    X2, W2, M2, Z2 = fresh()
    with binding.Sgp(n, d, graph_desc(w, binding)) as h:
        h.set_option("variant", variant)
        h.set_option("lockstep", lockstep)
        h.step(X2, W2, M2, G[0], Z2, 0, w.lr, w.momentum, 0.0, True)       # warm-up outside capture (sets attributes)
        torch.cuda.synchronize()
        X2, W2, M2, Z2 = fresh()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for k in range(period):
                    h.step(X2, W2, M2, G[k], Z2, k, w.lr, w.momentum, 0.0, True, stream=side)
        graph.replay()
        graph.replay()
        torch.cuda.synchronize()
        assert h.device_status() == 0
        assert h.get_option("last_lockstep") == lockstep
    for a, b in ((X, X2), (W, W2), (M, M2), (Z, Z2)):
        assert torch.equal(a, b)


@pytest.mark.parametrize("tau", [0, 1])
@pytest.mark.parametrize("variant", [1, 3])
def test_custom_weighted_schedule_on_gpu(binding, inputs, tau, variant):
    """Per-edge, non-uniform mixing weights on an irregular time-varying digraph (three steps)."""
    from test_schedule_compiler import _random_custom_schedule
    from oracle import schedule as osched
    n, steps = 12, 3
    step, send, recv, wt = _random_custom_schedule(n, steps, seed=5)
    g = binding.GraphDesc.custom(steps, step, send, recv, wt)
    mats = [osched.custom_mixing_matrix(n, send[step == k], recv[step == k], wt[step == k].astype(np.float32))
            for k in range(steps)]
    w = inputs.Workload("custom", n=n, d=3000, K=11, graph="custom", lr=0.05, momentum=0.9, tau=tau)
    out = _run_gpu(binding, inputs, w, graph=g, options={"variant": variant})
    _compare(w, out, P_of_k=lambda k: mats[k % steps])
    assert np.ptp(out["W"]) > 1e-2


@pytest.mark.parametrize("first,tau", [("complete", 0), ("two_peer", 0), ("two_peer", 2)])
def test_hybrid_schedules_switch_graph_mid_run(binding, inputs, first, tau):
    """AR/1P-SGP and 2P/1P-SGP (Table 3): dense mixing for the first steps, one-peer graph afterwards."""
    from oracle import schedule as osched
    n, d, K, K1 = 16, 3000, 14, 5
    w = inputs.Workload("hybrid", n=n, d=d, K=K, graph="exp", peers=1, lr=0.1, momentum=0.9, weight_decay=1e-4, tau=tau)
    g_first = binding.GraphDesc.complete() if first == "complete" else binding.GraphDesc.exp_peers(2)
    def P_of_k(k):
        if k < K1:
            return osched.mixing_matrix("complete", n, k) if first == "complete" else osched.mixing_matrix("exp", n, k, peers=2)
        return osched.mixing_matrix("exp", n, k, peers=1)
    X = inputs.initial_x(w, device=DEV).contiguous(); W = torch.ones(n, device=DEV)
    M = torch.zeros((n, d), device=DEV); Z = torch.empty((n, d), device=DEV); G = torch.empty((n, d), device=DEV)
    x0 = X.cpu().numpy().copy(); grads = []
    with binding.Sgp(n, d, g_first, tau=tau) as h:
        for k in range(K):
            if k == K1:
                h.set_graph(binding.GraphDesc.exp_peers(1))
                assert h.schedule.period == 4
            grads.append(inputs.gradient(w, k, G).cpu().numpy().copy())
            h.step(X, W, M, G, Z, k, w.lr, w.momentum, w.weight_decay, True)
        torch.cuda.synchronize()
        with pytest.raises(binding.SgpError):
            h.set_graph(binding.GraphDesc.exp_peers(0))             # rejected: the old schedule stays
        assert h.schedule.period == 4
        out = dict(x0=x0, grads=grads, X=X.cpu().numpy(), W=W.cpu().numpy(), M=M.cpu().numpy(), Z=Z.cpu().numpy(),
                   stats=h.check(X, W), ring=None)
        if tau:
            rx = torch.empty((tau, n, d), device=DEV); rw = torch.empty((tau, n), device=DEV)
            h.ring_export(rx, rw); torch.cuda.synchronize()
            out["ring"] = (rx.cpu().numpy(), rw.cpu().numpy())
    _compare(w, out, P_of_k=P_of_k)


def test_bounded_wait_reports_status_instead_of_hanging(binding, inputs):
    """Failure detection without a fault: one CTA's tile is never requested, its consumers' wait runs out after
    the configured bound, the kernel returns, the status word says so, and the handle keeps working."""
    import time
    w = inputs.WORKLOADS["resnet50"].scaled(256 * 600, K=1)
    n, d = w.n, w.d
    def state():
        X = inputs.initial_x(w, device=DEV).contiguous()
        return X, torch.ones(n, device=DEV), torch.zeros((n, d), device=DEV), torch.empty((n, d), device=DEV)
    G = inputs.gradient(w, 0, torch.empty((n, d), device=DEV))
    with binding.Sgp(n, d, graph_desc(w, binding)) as h:
        h.set_option("variant", 3)
        h.set_option("wait_limit_ms", 200)
        h.set_option("inject_stall", 1)
        X, W, M, Z = state()
        t0 = time.perf_counter()
        h.step(X, W, M, G, Z, 0, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()                                   # returns: no hang, no CUDA error
        assert time.perf_counter() - t0 < 5.0
        assert h.get_option("last_variant") == 3
        status = h.device_status()
        assert status & 1                                          # consumers gave up on the missing tile
        h.reset()
        h.set_option("inject_stall", 0)
        assert h.device_status() == 0
        X, W, M, Z = state()
        h.step(X, W, M, G, Z, 0, w.lr, w.momentum, 0.0, True)     # the context and the handle are still usable
        torch.cuda.synchronize()
        assert h.device_status() == 0
        ref = state()
        h.set_option("variant", 1)
        h.step(ref[0], ref[1], ref[2], G, ref[3], 0, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
        assert torch.equal(X, ref[0]) and torch.equal(Z, ref[3]) and torch.equal(M, ref[2])


@pytest.mark.parametrize("n,tau,nesterov", [(1, 2, True), (2, 1, True), (3, 3, False), (2, 1, False)])
def test_degenerate_node_counts_with_delay(binding, inputs, n, tau, nesterov):
    """n = 1 (no peers: the ring stays empty), n = 2 (one hop, the two nodes swap), heavy-ball with a ring."""
    w = inputs.Workload("degenerate", n=n, d=777, K=9, graph="exp", peers=1, lr=0.1, momentum=0.9, nesterov=nesterov,
                        tau=tau, weight_decay=1e-3)
    out = _run_gpu(binding, inputs, w)
    _compare(w, out)
    if n == 1:
        assert np.array_equal(out["W"], np.ones(1, dtype=np.float32)) and not out["ring"][0].any()


@pytest.mark.parametrize("n,d", [(2, 1000), (7, 3000), (32, 8200), (64, 2052), (256, 1029)])
@pytest.mark.parametrize("variant", [1, 3])
def test_complete_graph_shared_column_sum_path(binding, inputs, n, d, variant):
    """All receivers alike (complete graph): the mix is one column sum shared by every row; momentum and Z on."""
    w = inputs.Workload("complete", n=n, d=d, K=6, graph="complete", lr=0.1, momentum=0.9, weight_decay=1e-4)
    out = _run_gpu(binding, inputs, w, options={"variant": variant})
    _compare(w, out)
    assert np.abs(out["Z"] - out["Z"][0]).max() == 0.0               # every node holds the same vector, bit for bit


# ------------------------------------------------------------------ thread-block-cluster kernel (many nodes)
@pytest.mark.parametrize("n,d,tau,cluster", [(256, 1_029, 0, 4), (256, 4_100, 1, 4), (200, 3_001, 0, 4), (130, 2_052, 2, 4),
                                             (129, 1_500, 0, 2), (64, 9_000, 0, 2), (5, 2_000, 1, 4), (2, 700, 0, 2),
                                             (256, 70_001, 0, 4), (3, 1_000, 0, 4)])
def test_cluster_kernel_matches_oracle_and_register_kernel(binding, inputs, n, d, tau, cluster):
    """A cluster of CTAs holds the tile's rows together and gathers through distributed shared memory: same CSR
    order and FMA chain as the one-CTA kernels, so results are bit-identical to theirs and within tolerance of the
    oracle.  n = 3 with four CTAs leaves one CTA without rows; n = 200 leaves the last CTA a partial slice."""
    w = dataclasses.replace(inputs.sweep_workload(n, d), tau=tau, weight_decay=1e-3, K=5)
    a = _run_gpu(binding, inputs, w, options={"variant": 4, "cluster": cluster})
    _compare(w, a)
    b = _run_gpu(binding, inputs, w, options={"variant": 1})
    for name in ("X", "Z", "M", "W"):
        assert np.array_equal(a[name], b[name]), name


def test_dynamic_shared_memory_just_under_48_kb(binding, inputs):
    """n = 88 with the sweep's tenth graph needs 49,148 bytes of dynamic shared memory: with the kernel's few static
    bytes that is over the 48 KB a launch gets without the opt-in attribute (the launch used to fail with
    cudaErrorInvalidValue on exactly that step)."""
    w = dataclasses.replace(inputs.sweep_workload(88, 3_000), K=12)
    out = _run_gpu(binding, inputs, w, options={"variant": 1})
    _compare(w, out)


@pytest.mark.parametrize("tau,diag", [(0, 0), (1, 0), (0, 1), (2, 1)])
def test_every_node_count_launches(binding, inputs, tau, diag):
    """Every n from 1 to 256 on the sweep's ten random digraphs (table sizes, tile widths and shared-memory sizes all
    differ), with and without a delay ring and the fused diagnostics: no launch fails, no status bit, the weights
    (ring included) still sum to n."""
    d = 1_030
    for n in range(1, 257):
        w = inputs.sweep_workload(n, d)
        X = torch.zeros((n, d), device=DEV); M = torch.zeros((n, d), device=DEV); Z = torch.empty((n, d), device=DEV)
        G = torch.ones((n, d), device=DEV); W = torch.ones(n, device=DEV)
        with binding.Sgp(n, d, graph_desc(w, binding), tau=tau) as h:
            h.set_option("diagnostics", diag)
            for k in range(10):
                h.step(X, W, M, G, Z, k, w.lr, w.momentum, 0.0, True)
            torch.cuda.synchronize()
            assert h.device_status() == 0, n
            stats = h.check(X, W)
            assert stats["code"] == binding.SGP_OK and abs(stats["sum_w"] - n) < 1e-4 * n, (n, stats)
        assert torch.isfinite(X).all() and torch.isfinite(Z).all(), n


# ------------------------------------------------------------------ peeled kernel (rows off the 16-byte grid)
@pytest.mark.parametrize("n,d,pad,offset,tau,momentum", [
    (32, 4_101, 0, 0, 0, 0.9), (32, 4_102, 0, 0, 1, 0.9), (32, 4_103, 0, 0, 0, 0.0), (5, 1_029, 1, 0, 2, 0.9),
    (16, 3_000, 3, 1, 0, 0.9), (16, 3_000, 0, 3, 1, 0.9), (64, 2_049, 0, 2, 0, 0.9), (256, 1_031, 0, 0, 0, 0.9),
    (130, 777, 2, 1, 3, 0.9), (1, 19, 0, 1, 0, 0.9), (3, 16, 1, 0, 1, 0.0), (8, 70_003, 0, 0, 0, 0.9)])
def test_peeled_kernel_matches_oracle_and_scalar_instantiation(binding, inputs, n, d, pad, offset, tau, momentum):
    """Rows that do not start on 16-byte boundaries (ld = d + pad not a multiple of 4 and / or every array offset by the
    same odd number of floats): the automatic choice is the peeled kernel (last_variant 5), whose results are those of
    the scalar instantiation bit for bit and within tolerance of the oracle.  Shapes cover every row phase, one-row
    and many-row tiles, tiles narrower than four columns of slack, the delay ring and plain SGD."""
    w = dataclasses.replace(inputs.sweep_workload(n, d), tau=tau, momentum=momentum, weight_decay=1e-3, K=5)
    a = _run_gpu(binding, inputs, w, ld=d + pad, offset=offset)
    _compare(w, a)
    b = _run_gpu(binding, inputs, w, ld=d + pad, offset=offset, options={"variant": 1})
    for name in ("X", "Z", "W") + (("M",) if momentum else ()):
        assert np.array_equal(a[name], b[name]), name
    if tau:
        assert np.array_equal(a["ring"][0], b["ring"][0]) and np.array_equal(a["ring"][1], b["ring"][1])


@pytest.mark.parametrize("pad,offset,want", [(1, 0, 5), (0, 1, 5), (0, 0, 1), (4, 4, 1)])
def test_peeled_kernel_is_the_automatic_choice_off_the_16_byte_grid(binding, inputs, pad, offset, want):
    w = inputs.sweep_workload(16, 40_000)
    n, d, ld = w.n, w.d, w.d + pad
    def alloc():
        buf = torch.zeros(n * ld + offset + 8, device=DEV)
        return buf[offset:offset + n * ld].view(n, ld)[:, :d]
    X, M, Z, G = alloc(), alloc(), alloc(), alloc()
    W = torch.ones(n, device=DEV)
    with binding.Sgp(n, d, graph_desc(w, binding), ld=ld) as h:
        h.step(X, W, M, G, Z, 0, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
        assert h.get_option("last_variant") == want and h.device_status() == 0
        h.set_option("variant", 5)                      # forced: runs on aligned rows as well
        h.step(X, W, M, G, Z, 1, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
        assert h.get_option("last_variant") == 5 and h.device_status() == 0


def test_peeled_kernel_on_aligned_rows_equals_the_vector_kernel(binding, inputs):
    w = dataclasses.replace(inputs.sweep_workload(32, 9_004), tau=1, K=6, weight_decay=1e-3)
    a = _run_gpu(binding, inputs, w, options={"variant": 5})
    _compare(w, a)
    b = _run_gpu(binding, inputs, w, options={"variant": 1})
    for name in ("X", "Z", "M", "W"):
        assert np.array_equal(a[name], b[name]), name


# ------------------------------------------------------------------ lockstep clusters of the register-staged kernel
@pytest.mark.parametrize("n,d,tau,size,diag", [(32, 1_029, 0, 2, 0), (32, 70_001, 1, 2, 0), (64, 9_003, 0, 4, 0), (5, 2_000, 2, 4, 0),
                                               (130, 2_052, 0, 4, 0), (2, 260, 0, 2, 0), (48, 40_000, 1, 2, 1), (8, 300_001, 0, 4, 1)])
def test_lockstep_clusters_change_no_bit(binding, inputs, n, d, tau, size, diag):
    """CTAs launched as clusters that meet before each tile share no data: the step's results are those of independent
    CTAs bit for bit and within tolerance of the oracle.  The shapes leave the last cluster with fewer tiles than CTAs
    (1,029 columns are 5 tiles of 256), use the delay ring, the scalar tail and the fused diagnostics."""
    w = dataclasses.replace(inputs.sweep_workload(n, d), tau=tau, weight_decay=1e-3, K=5)
    a = _run_gpu(binding, inputs, w, options={"variant": 1, "lockstep": size, "diagnostics": diag})
    _compare(w, a)
    b = _run_gpu(binding, inputs, w, options={"variant": 1, "lockstep": 1, "diagnostics": diag})
    for name in ("X", "Z", "M", "W"):
        assert np.array_equal(a[name], b[name]), name


def test_lockstep_is_automatic_for_rows_off_the_128_byte_grid(binding, inputs):
    """A dense pitch whose rows start on 32-byte boundaries takes the register-staged kernel in lockstep pairs; the same
    step with rows on 1 KB boundaries does not; both give the same bits."""
    w = dataclasses.replace(inputs.sweep_workload(32, 400_008), K=1)
    assert (w.d * 4) % 128 == 32
    results = []
    for ld in (w.d, (w.d + 255) // 256 * 256):
        X = inputs.initial_x(w, device=DEV, ld=ld)
        M = torch.zeros((w.n, ld), device=DEV)[:, :w.d]; Z = torch.empty((w.n, ld), device=DEV)[:, :w.d]
        G = inputs.gradient(w, 0, torch.empty((w.n, ld), device=DEV)[:, :w.d])
        W = torch.ones(w.n, device=DEV)
        with binding.Sgp(w.n, w.d, graph_desc(w, binding), ld=ld) as h:
            h.step(X, W, M, G, Z, 0, w.lr, w.momentum, 0.0, True)
            torch.cuda.synchronize()
            assert h.device_status() == 0
            results.append((h.get_option("last_lockstep"), h.get_option("last_variant"), h.get_option("last_grid"), Z.cpu().numpy().copy()))
    assert results[0][0] == 2 and results[0][1] == 1 and results[0][2] % 2 == 0
    assert results[1][0] == 0
    assert np.array_equal(results[0][3], results[1][3])


def test_cluster_kernel_is_opt_in(binding, inputs):
    w = inputs.sweep_workload(256, 300_000)
    X = inputs.initial_x(w, device=DEV).contiguous()
    W = torch.ones(w.n, device=DEV); M = torch.zeros_like(X); Z = torch.empty_like(X)
    G = inputs.gradient(w, 0, torch.empty_like(X))
    with binding.Sgp(w.n, w.d, graph_desc(w, binding)) as h:
        h.step(X, W, M, G, Z, 0, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
        assert h.get_option("last_variant") == 1
        h.set_option("variant", 4)
        h.set_option("cluster", 4)
        h.step(X, W, M, G, Z, 1, w.lr, w.momentum, 0.0, True)
        torch.cuda.synchronize()
        assert h.get_option("last_variant") == 4 and h.get_option("last_tile_cols") == 256
        assert h.get_option("last_grid") % 4 == 0
        assert h.device_status() == 0
