"""Helpers shared by the parity tests: oracle schedule lookup for a workload, error metrics, runners."""
from __future__ import annotations

import numpy as np

from oracle import schedule as osched
from oracle import sgp as osgp

REL_TOL = 1e-5   # fp32 state vs float64 oracle (max relative error after K steps)


def oracle_P_of_k(w):
    """Dense mixing matrices of a workload, from the oracle's own generator."""
    if w.graph == "exp":
        return lambda k: osched.mixing_matrix("exp", w.n, k, peers=w.peers)
    if w.graph in ("complete", "bipartite"):
        return lambda k: osched.mixing_matrix(w.graph, w.n, k)
    if w.graph == "random":
        return lambda k: osched.mixing_matrix("random", w.n, k, seed=w.seed, max_outdeg=w.max_outdeg,
                                              num_steps=w.num_steps)
    raise ValueError(w.graph)


def graph_desc(w, binding):
    return binding.graph_desc(w)


def assert_close(name, got, want, tol=REL_TOL):
    """Gate: max|got - want| <= tol * max|want| and, element by element,
    |got - want| <= tol * max(|want|, rms(want)) (pure relative error is meaningless next to zero)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (name, got.shape, want.shape)
    assert np.all(np.isfinite(got)), f"{name}: non-finite values"
    diff = np.abs(got - want)
    scale = np.abs(want).max()
    if scale == 0.0:
        assert diff.max() == 0.0, f"{name}: expected exact zeros, max |diff| = {diff.max()}"
        return 0.0
    normwise = diff.max() / scale
    assert normwise <= tol, f"{name}: normwise error {normwise:.3e} > {tol}"
    rms = np.sqrt(np.mean(want * want))
    floor = np.maximum(np.abs(want), rms)
    elem = (diff / floor).max()
    assert elem <= tol, f"{name}: element-wise error {elem:.3e} > {tol}"
    return normwise


def run_oracle(w, x0, grads, K=None, tau=None):
    """Oracle trajectory for pre-generated gradients grads[k] (n x d arrays)."""
    K = w.K if K is None else K
    tau = w.tau if tau is None else tau
    return osgp.sgp_run(np.asarray(x0, dtype=np.float64), K, oracle_P_of_k(w),
                        lambda k, z: np.asarray(grads[k], dtype=np.float64), w.lr, momentum=w.momentum,
                        nesterov=w.nesterov, weight_decay=w.weight_decay, tau=tau)
