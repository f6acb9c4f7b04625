"""sgp_step_static: the fused step for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits (the whole device budget belongs to a
framework pool, or an allocation's device-wide synchronisation would break a latency target), so they
cannot create a handle.  This test drives the handle-free entry point through the C ABI and requires
its results to agree with the handle-based sgp_step on the same inputs, for two calls in a row (the
two steps use different mixing tables, so the shared static table is rewritten between them).

Collected last on purpose: a failure here must not hide any other test's result."""
import ctypes as C

import numpy as np
import pytest
import torch

from parity_util import REL_TOL, assert_close, graph_desc

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
    assert np.ptp(Wb.cpu().numpy()) > 1e-3                                # irregular graph: the weight path is exercised
    # padding between rows untouched
    if ld_extra:
        full = Xb.as_strided((n, ld), (ld, 1))
        assert torch.isnan(full[:, d:]).all().item()


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
    bad = col.copy(); bad[3] = n
    assert call(n, len(col), cl=bad) == binding.SGP_ERR_GRAPH                      # sender index out of range
    assert lib.sgp_step_static(n, d, d, p(rowptr), p(col), p(val), len(col), t(X), t(W), None, t(G), None, 0.1, 0.9,
                               0.0, 1, None) == binding.SGP_ERR_ARG                # momentum without M
    torch.cuda.synchronize()
    big = binding.Schedule(256, binding.GraphDesc.complete())
    assert big.nnz(0) > binding.SGP_STATIC_MAX_NNZ
