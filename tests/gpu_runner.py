"""Runner shared by the GPU parity tests: K fused steps through the C ABI on seeded inputs, NaN sentinels in all
padding, then the comparison with the float64 oracle on the very same fp32 input bits."""
import numpy as np
import torch

from parity_util import assert_close, graph_desc, oracle_P_of_k

DEV = "cuda:0"


def run_gpu(binding, inputs, w, K=None, ld=None, write_z=True, options=None, graph=None, x0=None, offset=0, flags=0,
            want_diagnostics=False):
    """Runs K fused steps on the GPU; returns (x0, grads, X, W, M, Z, handle-free ring copies)."""
    K = w.K if K is None else K
    n, d = w.n, w.d
    ld = d if ld is None else ld
    pad = float("nan")
    def alloc():
        buf = torch.full((n * ld + offset + 8,), pad, dtype=torch.float32, device=DEV)
        return buf, buf[offset:offset + n * ld].view(n, ld)[:, :d]
    Xb, X = alloc()
    Mb, M = alloc()
    Gb, G = alloc()
    Zb, Z = alloc()
    X.copy_(inputs.initial_x(w, device=DEV) if x0 is None else torch.as_tensor(x0, dtype=torch.float32, device=DEV))
    M.zero_()
    W = torch.ones(n, dtype=torch.float32, device=DEV)
    x0_bits = X.cpu().numpy().copy()
    grads = []
    ring = None
    diags = []
    with binding.Sgp(n, d, graph_desc(w, binding) if graph is None else graph, tau=w.tau, ld=ld, flags=flags) as h:
        for key, val in (options or {}).items():
            h.set_option(key, val)
        if want_diagnostics:
            h.set_option("diagnostics", 1)
        for k in range(K):
            inputs.gradient(w, k, G)
            grads.append(G.cpu().numpy().copy())
            h.step(X, W, M if w.momentum != 0.0 else None, G, Z if write_z else None, k, w.lr, w.momentum,
                   w.weight_decay, w.nesterov)
            if want_diagnostics:
                diags.append(h.diagnostics())
        torch.cuda.synchronize()
        assert h.device_status() == 0
        stats = h.check(X, W)
        if w.tau > 0:
            rx = torch.empty((w.tau, n, ld), dtype=torch.float32, device=DEV)
            rw = torch.empty((w.tau, n), dtype=torch.float32, device=DEV)
            h.ring_export(rx, rw)
            torch.cuda.synchronize()
            ring = (rx[:, :, :d].cpu().numpy(), rw.cpu().numpy())
    # padding between rows and around the arrays must be untouched (NaN sentinels)
    for name, buf in (("X", Xb), ("M", Mb), ("Z", Zb)):
        full = buf.cpu().numpy()
        mask = np.ones(full.shape, dtype=bool)
        body = mask[offset:offset + n * ld].reshape(n, ld)
        body[:, :d] = False
        assert np.all(np.isnan(full[mask])), f"{name}: padding was overwritten"
    return dict(x0=x0_bits, grads=grads, X=X.cpu().numpy(), W=W.cpu().numpy(), M=M.cpu().numpy(),
                Z=Z.cpu().numpy(), ring=ring, stats=stats, diagnostics=diags)


def compare_with_oracle(w, out, K=None, write_z=True, P_of_k=None, send_period=1, biased=False):
    from oracle import sgp as osgp
    K = w.K if K is None else K
    if P_of_k is None:
        P_of_k = oracle_P_of_k(w)
    st = osgp.sgp_run(out["x0"].astype(np.float64), K, P_of_k, lambda k, z: out["grads"][k].astype(np.float64),
                      w.lr, momentum=w.momentum, nesterov=w.nesterov, weight_decay=w.weight_decay, tau=w.tau,
                      send_period=send_period, biased=biased)
    assert_close("X", out["X"], st.x)
    assert_close("W", out["W"], st.w)
    if w.momentum != 0.0:
        assert_close("M", out["M"], st.u)
    if write_z:
        assert_close("Z", out["Z"], st.z)
    if w.tau > 0:
        # ring slot s holds the message written at the last step k with k mod tau == s
        ring_x, ring_w = out["ring"]
        msgs_x, msgs_w = list(st.transit_x), list(st.transit_w)      # oldest first: sent at K-tau .. K-1
        for age, (mx, mw) in enumerate(zip(msgs_x, msgs_w)):
            k_sent = K - w.tau + age
            assert_close(f"ring_x[{k_sent % w.tau}]", ring_x[k_sent % w.tau], mx)
            assert_close(f"ring_w[{k_sent % w.tau}]", ring_w[k_sent % w.tau], mw)
    # invariants from the GPU's own check kernel
    stats = out["stats"]
    assert stats["code"] == 0 and stats["status"] == 0
    assert abs(stats["sum_w"] - w.n) <= 1e-4 * w.n and stats["min_w"] > 0 and stats["nonfinite"] == 0
    return st
