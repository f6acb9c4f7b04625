"""sgp_step_static: the fused step for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits (the whole device budget belongs to a
framework pool, or an allocation's device-wide synchronisation would break a latency target), so they
cannot create a handle.  This test drives the handle-free entry point through the C ABI and requires
its results to equal the handle-based sgp_step's bit for bit on the same inputs and to match the float64
oracle, for two calls in a row (the two steps use different mixing tables, so the shared static table is
rewritten between them).

Collected last on purpose: a failure here must not hide any other test's result."""
import ctypes as C

import numpy as np
import pytest
import torch

from parity_util import REL_TOL, assert_close, graph_desc, oracle_P_of_k

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


def _state(inputs, w, ld):
    n, d = w.n, w.d

    def matrix():
        return torch.full((n, ld), float("nan"), device=DEV)[:, :d]

    X = matrix()
    X.copy_(inputs.initial_x(w, device=DEV))
    M = matrix()
    M.zero_()
    Z = matrix()
    return X, torch.ones(n, device=DEV), M, Z


@pytest.mark.parametrize("n,d,ld_extra,momentum", [(16, 5003, 0, 0.9), (16, 4104, 8, 0.9), (64, 2052, 0, 0.0),
                                                    (4, 9000, 0, 0.9)])
def test_static_step_matches_handle_step_two_calls_in_a_row(binding, inputs, n, d, ld_extra, momentum):
    import dataclasses
    w = dataclasses.replace(inputs.sweep_workload(n, d), momentum=momentum, weight_decay=1e-3)
    ld = d + ld_extra
    G = [torch.full((n, ld), float("nan"), device=DEV)[:, :d] for _ in range(2)]
    for k in range(2):
        inputs.gradient(w, k, G[k])
    Xa, Wa, Ma, Za = _state(inputs, w, ld)
    Xb, Wb, Mb, Zb = _state(inputs, w, ld)
    x0 = Xa.cpu().numpy().astype(np.float64)
    with binding.Sgp(n, d, graph_desc(w, binding), ld=ld) as h:
        tables = [h.schedule.get(k) for k in range(2)]
        assert not np.array_equal(tables[0][1], tables[1][1])            # the two steps really differ
        for k in range(2):
            h.step(Xa, Wa, Ma if momentum else None, G[k], Za, k, w.lr, momentum, w.weight_decay, True)
        torch.cuda.synchronize()
    for k in range(2):                                                    # two calls in a row, one stream
        rowptr, col, val = tables[k]
        binding.step_static(n, d, ld, rowptr, col, val, Xb, Wb, Mb if momentum else None, G[k], Zb, w.lr, momentum,
                            w.weight_decay, True)
    torch.cuda.synchronize()
    for name, a, b in (("X", Xa, Xb), ("W", Wa, Wb), ("M", Ma, Mb), ("Z", Za, Zb)):
        assert_close(name, b.cpu().numpy(), a.cpu().numpy(), tol=REL_TOL)
        assert torch.equal(a, b), f"{name}: the static path and the handle path run the same kernel arithmetic"
    # ... and against the oracle directly, on the fp32 bits the GPU consumed
    from oracle import sgp as osgp
    st = osgp.sgp_run(x0, 2, oracle_P_of_k(w), lambda k, z: G[k].cpu().numpy().astype(np.float64), w.lr,
                      momentum=momentum, nesterov=True, weight_decay=w.weight_decay)
    assert_close("X vs oracle", Xb.cpu().numpy(), st.x)
    assert_close("Z vs oracle", Zb.cpu().numpy(), st.z)
    assert_close("W vs oracle", Wb.cpu().numpy(), st.w)
    if momentum:
        assert_close("M vs oracle", Mb.cpu().numpy(), st.u)
    assert np.ptp(Wb.cpu().numpy()) > 1e-3                                # irregular graph: the weight path is exercised
    # padding between rows untouched
    if ld_extra:
        full = Xb.as_strided((n, ld), (ld, 1))
        assert torch.isnan(full[:, d:]).all().item()


def test_handle_step_still_launches_after_a_smaller_static_step(binding, inputs):
    """Both paths run the same kernel instantiations and share one record of the shared-memory limit each was
    granted.  A static step that needs less must not shrink what a handle step at a larger shape was given:
    handle step (n = 80, one 80 KB exchange tile), static step (n = 64), then the same handle step again."""
    import dataclasses
    big = dataclasses.replace(inputs.sweep_workload(80, 300_000), weight_decay=0.0)
    small = dataclasses.replace(inputs.sweep_workload(64, 40_000), weight_decay=0.0)
    Xa, Wa, Ma, Za = _state(inputs, big, big.d)
    Ga = inputs.gradient(big, 0, torch.empty_like(Xa))
    Xs, Ws, Ms, Zs = _state(inputs, small, small.d)
    Gs = inputs.gradient(small, 0, torch.empty_like(Xs))
    x0 = Xa.cpu().numpy().astype(np.float64)
    sched = binding.Schedule(small.n, graph_desc(small, binding))
    with binding.Sgp(big.n, big.d, graph_desc(big, binding)) as h:
        h.set_option("variant", 1)
        h.step(Xa, Wa, Ma, Ga, Za, 0, big.lr, big.momentum, 0.0, True)
        torch.cuda.synchronize()
        smem_big = h.get_option("last_smem")
        assert smem_big > 64 * 1024
        binding.step_static(small.n, small.d, small.d, *sched.get(0), Xs, Ws, Ms, Gs, Zs, small.lr, small.momentum, 0.0,
                            True)
        torch.cuda.synchronize()
        h.step(Xa, Wa, Ma, Ga, Za, 1, big.lr, big.momentum, 0.0, True)       # must launch: SGP_OK, no CUDA error
        torch.cuda.synchronize()
        assert h.get_option("last_smem") == smem_big and h.last_cuda_error() == 0 and h.device_status() == 0
    from oracle import sgp as osgp
    g = Ga.cpu().numpy().astype(np.float64)
    st = osgp.sgp_run(x0, 2, oracle_P_of_k(big), lambda k, z: g, big.lr, momentum=big.momentum, nesterov=True)
    assert_close("X", Xa.cpu().numpy(), st.x)
    assert_close("Z", Za.cpu().numpy(), st.z)


def test_static_step_refuses_a_stream_that_is_being_captured(binding, inputs):
    w = inputs.sweep_workload(8, 4_096)
    X, W, M, Z = _state(inputs, w, w.d)
    G = inputs.gradient(w, 0, torch.empty_like(X))
    sched = binding.Schedule(w.n, graph_desc(w, binding))
    binding.step_static(w.n, w.d, w.d, *sched.get(0), X, W, M, G, Z, w.lr, w.momentum, 0.0, True)   # set-up call
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            with pytest.raises(binding.SgpError) as e:
                binding.step_static(w.n, w.d, w.d, *sched.get(1), X, W, M, G, Z, w.lr, w.momentum, 0.0, True,
                                    stream=side)
            X.add_(0.0)                                                    # the capture itself stays valid
    assert e.value.code == binding.SGP_ERR_STATE
    torch.cuda.synchronize()


def test_static_step_rejects_what_does_not_fit(binding):
    lib = binding.lib()
    n, d = 8, 64
    X = torch.zeros((n, d), device=DEV); W = torch.ones(n, device=DEV); G = torch.zeros((n, d), device=DEV)
    sched = binding.Schedule(n, binding.GraphDesc.exp_peers(1))
    rowptr, col, val = sched.get(0)
    p = lambda a: a.ctypes.data
    t = lambda a: a.data_ptr()

    def call(n_, nnz, rp=rowptr, cl=col):
        return lib.sgp_step_static(n_, d, d, p(rp), p(cl), p(val), nnz, t(X), t(W), None, t(G), None, 0.1, 0.0, 0.0, 1,
                                   None)

    assert call(n, len(col)) == binding.SGP_OK
    assert call(binding.SGP_MAX_NODES + 1, len(col)) == binding.SGP_ERR_ARG
    assert call(n, binding.SGP_STATIC_MAX_NNZ + 1) == binding.SGP_ERR_ARG          # table larger than the static array
    assert call(n, len(col) - 1) == binding.SGP_ERR_GRAPH                          # rowptr[n] != nnz
    skew = val.copy(); skew[0] *= 1.5
    assert lib.sgp_step_static(n, d, d, p(rowptr), p(col), p(skew), len(col), t(X), t(W), None, t(G), None, 0.1, 0.0,
                               0.0, 1, None) == binding.SGP_ERR_GRAPH              # a column no longer sums to one
    bad = col.copy(); bad[3] = n
    assert call(n, len(col), cl=bad) == binding.SGP_ERR_GRAPH                      # sender index out of range
    assert lib.sgp_step_static(n, d, d, p(rowptr), p(col), p(val), len(col), t(X), t(W), None, t(G), None, 0.1, 0.9,
                               0.0, 1, None) == binding.SGP_ERR_ARG                # momentum without M
    torch.cuda.synchronize()
    big = binding.Schedule(256, binding.GraphDesc.complete())
    assert big.nnz(0) > binding.SGP_STATIC_MAX_NNZ
