"""GPU parity of the Adam-SGP step (sgp_step_adam) against the float64 oracle."""
import dataclasses

import numpy as np
import pytest
import torch

from parity_util import assert_close, graph_desc, oracle_P_of_k

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
BETAS = (0.9, 0.98)      # the Transformer recipe's Adam decay rates
EPS = 1e-8


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


def _run(binding, inputs, w, options=None, ld=None, offset=0, lr=1e-2, wd=0.0, write_z=True):
    n, d, K = w.n, w.d, w.K
    ld = d if ld is None else ld

    def alloc(fill):
        buf = torch.full((n * ld + offset + 8,), float("nan"), device=DEV)
        view = buf[offset:offset + n * ld].view(n, ld)[:, :d]
        if fill is not None:
            view.fill_(fill)
        return buf, view

    _, X = alloc(None)
    X.copy_(inputs.initial_x(w, device=DEV))
    m1b, M1 = alloc(0.0)
    m2b, M2 = alloc(0.0)
    zb, Z = alloc(None)
    _, G = alloc(0.0)
    W = torch.ones(n, device=DEV)
    x0 = X.cpu().numpy().copy()
    grads = []
    with binding.Sgp(n, d, graph_desc(w, binding), tau=w.tau, ld=ld) as h:
        for key, val in (options or {}).items():
            h.set_option(key, val)
        for k in range(K):
            inputs.gradient(w, k, G)
            grads.append(G.cpu().numpy().copy())
            h.step_adam(X, W, M1, M2, G, Z if write_z else None, k, k + 1, lr, BETAS[0], BETAS[1], EPS, wd)
        torch.cuda.synchronize()
        assert h.device_status() == 0
    for buf in (m1b, m2b):
        full = buf.cpu().numpy()
        mask = np.ones(full.shape, dtype=bool)
        mask[offset:offset + n * ld].reshape(n, ld)[:, :d] = False
        assert np.all(np.isnan(full[mask]))                              # padding untouched
    return dict(x0=x0, grads=grads, X=X.cpu().numpy(), W=W.cpu().numpy(), M1=M1.cpu().numpy(), M2=M2.cpu().numpy(),
                Z=Z.cpu().numpy())


def _compare(w, out, lr=1e-2, wd=0.0, write_z=True):
    from oracle import sgp as osgp
    st = osgp.sgp_run(out["x0"].astype(np.float64), w.K, oracle_P_of_k(w),
                      lambda k, z: out["grads"][k].astype(np.float64), lr, weight_decay=wd, tau=w.tau,
                      adam=(BETAS[0], BETAS[1], EPS))
    assert_close("X", out["X"], st.x)
    assert_close("W", out["W"], st.w)
    assert_close("M1", out["M1"], st.u)
    assert_close("M2", out["M2"], st.v)
    if write_z:
        assert_close("Z", out["Z"], st.z)


def _cases(inputs):
    W = inputs.WORKLOADS
    return [
        W["transformer"].scaled(256 * 9 + 12),                            # the paper's Adam workload shape (n = 16, 2-peer)
        W["resnet50"].scaled(8200, K=12),
        dataclasses.replace(W["resnet50_osgp1"].scaled(4104, K=12), tau=1),
        dataclasses.replace(inputs.sweep_workload(16, 3000), tau=2),
        inputs.sweep_workload(4, 10_000), inputs.sweep_workload(64, 5000), inputs.sweep_workload(256, 1029),
        inputs.Workload("one", n=1, d=5, K=4, graph="exp"),
    ]


@pytest.mark.parametrize("case", range(8))
@pytest.mark.parametrize("variant", [0, 1, 3])
def test_adam_step_matches_oracle(binding, inputs, case, variant):
    w = _cases(inputs)[case]
    out = _run(binding, inputs, w, options={"variant": variant} if variant else None, wd=1e-2)
    _compare(w, out, wd=1e-2)
    if variant:
        ref = _run(binding, inputs, w, options={"variant": 1}, wd=1e-2)
        for name in ("X", "W", "M1", "M2", "Z"):
            assert np.array_equal(ref[name], out[name], equal_nan=True), name


@pytest.mark.parametrize("ld_extra,offset", [(4, 0), (3, 0), (0, 1), (252, 0)])
def test_adam_pitch_and_alignment(binding, inputs, ld_extra, offset):
    w = inputs.sweep_workload(16, 2052)
    out = _run(binding, inputs, w, ld=w.d + ld_extra, offset=offset)
    _compare(w, out)


def test_adam_without_z(binding, inputs):
    w = inputs.sweep_workload(8, 3000)
    out = _run(binding, inputs, w, write_z=False)
    _compare(w, out, write_z=False)
    assert np.all(np.isnan(out["Z"]))


def test_adam_argument_checks(binding):
    n, d = 4, 64
    X = torch.zeros((n, d), device=DEV); W = torch.ones(n, device=DEV); G = torch.zeros((n, d), device=DEV)
    M1 = torch.zeros((n, d), device=DEV); M2 = torch.zeros((n, d), device=DEV)
    lib = binding.lib()
    p = lambda t: t.data_ptr()
    with binding.Sgp(n, d, binding.GraphDesc.exp_peers(1)) as h:
        ok = lambda **kw: lib.sgp_step_adam(h._h, p(X), p(W), kw.get("m1", p(M1)), kw.get("m2", p(M2)), p(G), None,
                                            kw.get("k", 0), kw.get("t", 1), 0.1, kw.get("b1", 0.9), 0.999, 1e-8, 0.0,
                                            None)
        assert ok() == binding.SGP_OK
        assert ok(t=0) == binding.SGP_ERR_ARG
        assert ok(k=-1) == binding.SGP_ERR_ARG
        assert ok(b1=1.0) == binding.SGP_ERR_ARG
        assert ok(m2=None) == binding.SGP_ERR_ARG
        torch.cuda.synchronize()


def test_adam_step_host_matches_device_step(binding, inputs):
    """Host-buffer entry point for Adam-SGP: bit-identical to the device step (columns are independent, chunks too)."""
    import dataclasses
    w = dataclasses.replace(inputs.WORKLOADS["transformer_adam"].scaled(40_003, K=3), tau=1)
    n, d = w.n, w.d
    def state():
        X = inputs.initial_x(w, device=DEV).contiguous()
        return X, torch.ones(n, device=DEV), torch.zeros_like(X), torch.zeros_like(X), torch.empty_like(X)
    Xa, Wa, M1a, M2a, Za = state()
    Xb, Wb, M1b, M2b, Zb = state()
    G = torch.empty((n, d), device=DEV)
    hG = torch.empty((n, d), pin_memory=True)
    hZ = torch.empty((n, d), pin_memory=True)
    dG = torch.empty((n, d), device=DEV)
    with binding.Sgp(n, d, graph_desc(w, binding), tau=1) as h1, binding.Sgp(n, d, graph_desc(w, binding), tau=1) as h2:
        for k in range(3):
            inputs.gradient(w, k, G)
            hG.copy_(G)
            torch.cuda.synchronize()
            h1.step_adam(Xa, Wa, M1a, M2a, G, Za, k, k + 1, w.lr, w.beta1, w.beta2, w.adam_eps, 1e-3)
            h2.step_adam_host(Xb, Wb, M1b, M2b, hG, hZ, dG, Zb, k, k + 1, w.lr, w.beta1, w.beta2, w.adam_eps, 1e-3,
                              chunk_cols=8192)
        torch.cuda.synchronize()
    for a, b in ((Xa, Xb), (Wa, Wb), (M1a, M1b), (M2a, M2b), (Za, Zb)):
        assert torch.equal(a, b)
    assert torch.equal(hZ.to(DEV), Za)
