"""Seeded random configurations of the fused step against the float64 oracle: node count, parameter count, row pitch
and pointer offset, delay, optimiser flavour, graph kind, kernel family, lockstep clusters and diagnostics are drawn
together, so that combinations no hand-written case lists get exercised (Alg. 1 lines 4-8, Alg. 2, Alg. 3)."""
import os

import numpy as np
import pytest

from gpu_runner import compare_with_oracle, run_gpu
from parity_util import assert_close, oracle_P_of_k


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


def _draw(case: int):
    rng = np.random.RandomState(1811_10792 + case)
    n = int(np.clip(np.round(2.0 ** rng.uniform(0.0, 8.0)), 1, 256))
    graph = rng.choice(["exp", "exp2", "random", "complete", "bipartite"], p=[0.3, 0.15, 0.35, 0.1, 0.1])
    if graph == "bipartite" and n % 2:
        n += 1
    d = int(rng.choice([rng.randint(1, 40), rng.randint(40, 700), rng.randint(700, 6000)]))
    tau = int(rng.choice([0, 0, 1, 2, 3]))
    momentum = float(rng.choice([0.0, 0.9, 0.5]))
    opts = {"variant": int(rng.choice([0, 0, 1, 3])), "lockstep": int(rng.choice([0, 0, 1, 2, 4]))}
    if rng.rand() < 0.25:
        opts["tile_cols"] = int(rng.choice([32, 64, 128, 256, 512]))
    if rng.rand() < 0.2:
        opts["single_buffer"] = int(rng.choice([1, 2]))
    return dict(
        n=n, d=d, tau=tau, momentum=momentum, nesterov=bool(rng.rand() < 0.6),
        weight_decay=float(rng.choice([0.0, 1e-4, 1e-2])), graph=graph, K=int(rng.randint(3, 8)),
        pad=int(rng.choice([0, 0, 1, 3, 4, 8])), offset=int(rng.choice([0, 0, 1, 4])), write_z=bool(rng.rand() < 0.8),
        diag=bool(rng.rand() < 0.25), opts=opts, seed=int(rng.randint(1, 1 << 30)))


# SGP_FUZZ_CASES in the environment widens the three sweeps for a longer run by hand (the draws are seeded by case number)
_EXTRA = max(1, int(os.environ.get("SGP_FUZZ_CASES", "0")) // 256)


@pytest.mark.gpu
@pytest.mark.parametrize("case", range(256 * _EXTRA))
def test_random_configuration_matches_oracle(binding, inputs, case):
    c = _draw(case)
    kind, peers = ("exp", 2) if c["graph"] == "exp2" else (c["graph"], 1)
    w = inputs.Workload(f"fuzz{case}", n=c["n"], d=c["d"], K=c["K"], graph=kind, peers=peers, max_outdeg=4, num_steps=5,
                        lr=0.05, momentum=c["momentum"], nesterov=c["nesterov"], weight_decay=c["weight_decay"],
                        tau=c["tau"], seed=c["seed"])
    out = run_gpu(binding, inputs, w, ld=c["d"] + c["pad"], offset=c["offset"], write_z=c["write_z"], options=c["opts"],
                  want_diagnostics=c["diag"])
    compare_with_oracle(w, out, write_z=c["write_z"])
    if c["diag"]:
        for per_step in out["diagnostics"]:
            dev, cons = np.asarray(per_step[0]), np.asarray(per_step[1])
            assert np.all(np.isfinite(dev)) and np.all(np.isfinite(cons)) and np.all(dev >= 0) and np.all(cons >= 0)


def test_draws_cover_the_space():
    """The generator itself (no GPU work): the draws reach every graph kind, delay, kernel family and both paddings."""
    draws = [_draw(i) for i in range(256)]
    assert {c["graph"] for c in draws} == {"exp", "exp2", "random", "complete", "bipartite"}
    assert {c["tau"] for c in draws} == {0, 1, 2, 3}
    assert {c["opts"]["variant"] for c in draws} == {0, 1, 3}
    assert {c["opts"]["lockstep"] for c in draws} == {0, 1, 2, 4}
    assert any(c["pad"] % 4 for c in draws) and any(c["offset"] % 4 for c in draws)
    assert min(c["n"] for c in draws) <= 2 and max(c["n"] for c in draws) >= 128


def _draw_adam(case: int):
    rng = np.random.RandomState(9_1811 + case)
    n = int(np.clip(np.round(2.0 ** rng.uniform(0.0, 8.0)), 1, 256))
    graph = rng.choice(["exp", "exp2", "random", "complete"], p=[0.35, 0.2, 0.35, 0.1])
    d = int(rng.choice([rng.randint(1, 40), rng.randint(40, 700), rng.randint(700, 5000)]))
    opts = {"variant": int(rng.choice([0, 0, 1, 3])), "lockstep": int(rng.choice([0, 1, 2]))}
    return dict(n=n, d=d, tau=int(rng.choice([0, 0, 1, 2])), graph=graph, K=int(rng.randint(3, 7)),
                pad=int(rng.choice([0, 0, 2, 4])), offset=int(rng.choice([0, 0, 1, 4])), write_z=bool(rng.rand() < 0.8),
                wd=float(rng.choice([0.0, 1e-2])), opts=opts, seed=int(rng.randint(1, 1 << 30)))


@pytest.mark.gpu
@pytest.mark.parametrize("case", range(64 * _EXTRA))
def test_random_adam_configuration_matches_oracle(binding, inputs, case):
    """The same for the Adam-preconditioned step (Sec. 6.2 / App. C.1)."""
    from test_adam_gpu import _run as adam_run
    c = _draw_adam(case)
    kind, peers = ("exp", 2) if c["graph"] == "exp2" else (c["graph"], 1)
    w = inputs.Workload(f"fuzz_adam{case}", n=c["n"], d=c["d"], K=c["K"], graph=kind, peers=peers, max_outdeg=4,
                        num_steps=5, tau=c["tau"], seed=c["seed"], optimizer="adam")
    out = adam_run(binding, inputs, w, options=c["opts"], ld=c["d"] + c["pad"], offset=c["offset"], wd=c["wd"],
                   write_z=c["write_z"])
    _adam_compare_conditioned(w, out, wd=c["wd"], write_z=c["write_z"])


def _adam_compare_conditioned(w, out, wd, write_z, lr=1e-2):
    """The Adam step divides by sqrt(v) + eps: where the effective gradient g + wd x all but cancels, the ratio is close
    to sign(g~) and ANY two precisions disagree there by up to 2 lr (about one element in a million with these inputs).
    Such elements are found from the oracle alone -- the same run with every gradient scaled by 1 + 2^-22, four fp32
    roundings -- and are held to a bound of 4 K lr instead of the relative tolerance; at most one element in a thousand
    may be of that kind.  Everything else meets the usual gate."""
    from oracle import sgp as osgp
    from test_adam_gpu import BETAS, EPS
    from parity_util import REL_TOL

    def run(scale):
        return osgp.sgp_run(out["x0"].astype(np.float64), w.K, oracle_P_of_k(w),
                            lambda k, z: out["grads"][k].astype(np.float64) * scale, lr, weight_decay=wd, tau=w.tau,
                            adam=(BETAS[0], BETAS[1], EPS))
    st, st_eps = run(1.0), run(1.0 + 2.0 ** -22)
    names = [("X", out["X"], st.x, st_eps.x), ("M1", out["M1"], st.u, st_eps.u), ("M2", out["M2"], st.v, st_eps.v)]
    if write_z:
        names.append(("Z", out["Z"], st.z, st_eps.z))
    for name, got, want, want_eps in names:
        got = got.astype(np.float64)
        floor = np.maximum(np.abs(want), np.sqrt(np.mean(want * want)))
        ill = np.abs(want_eps - want) > 0.5 * REL_TOL * floor
        assert ill.mean() <= 1e-3, (name, float(ill.mean()))
        diff = np.abs(got - want)
        assert np.all(diff[ill] <= 4 * w.K * lr * np.maximum(1.0, np.abs(want[ill]))), name
        if (~ill).any():
            assert (diff[~ill] / floor[~ill]).max() <= REL_TOL, (name, float((diff[~ill] / floor[~ill]).max()))
    assert_close("W", out["W"], st.w)


def _draw_rank(case: int):
    rng = np.random.RandomState(7_1811 + case)
    n = int(np.clip(np.round(2.0 ** rng.uniform(0.0, 5.3)), 1, 40))
    graph = rng.choice(["exp", "exp2", "random", "complete", "bipartite"], p=[0.3, 0.2, 0.3, 0.1, 0.1])
    if graph == "bipartite" and n % 2:
        n += 1
    if graph == "complete":
        n = min(n, 32)                       # a mix takes at most 32 sources in this mode
    return dict(n=n, d=int(rng.choice([rng.randint(1, 40), rng.randint(40, 3000)])), tau=int(rng.choice([0, 0, 1, 2, 3])),
                graph=graph, momentum=float(rng.choice([0.0, 0.9])), nesterov=bool(rng.rand() < 0.6),
                offset=int(rng.choice([0, 0, 0, 1, 2])), write_z=bool(rng.rand() < 0.8), K=int(rng.randint(3, 7)),
                seed=int(rng.randint(1, 1 << 30)))


@pytest.mark.gpu
@pytest.mark.parametrize("case", range(64 * _EXTRA))
def test_random_one_node_per_gpu_configuration_equals_stacked_step(binding, inputs, case):
    """The split kernels (update / pull + mix, fused overlap step) in loopback give the stacked step's bits
    (App. C setting, Alg. 1 lines 4-8, Alg. 2), whatever the shape, delay, graph and alignment."""
    import torch
    from test_rowshard_gpu import _run_both
    c = _draw_rank(case)
    kind, peers = ("exp", 2) if c["graph"] == "exp2" else (c["graph"], 1)
    w = inputs.Workload(f"fuzz_rank{case}", n=c["n"], d=c["d"], K=c["K"], graph=kind, peers=peers, max_outdeg=4,
                        num_steps=5, lr=0.05, momentum=c["momentum"], nesterov=c["nesterov"], weight_decay=1e-3,
                        tau=c["tau"], seed=c["seed"])
    _x0, _grads, got, stacked = _run_both(binding, inputs, w, c["K"], offset=c["offset"], write_z=c["write_z"])
    names = ("X", "W") + (("Z",) if c["write_z"] else ()) + (("M",) if c["momentum"] else ())
    # where every row of a step's matrix is the same (complete graph, or n = 3 with two peers) and tau = 0, the stacked
    # step sums interleaved partial sums: equal to rounding, not bit for bit
    P_of_k = oracle_P_of_k(w)
    shortcut = c["tau"] == 0 and any(bool(np.all(P_of_k(k) == P_of_k(k)[0])) for k in range(c["K"])) and c["n"] > 1
    for name in names:
        if shortcut:
            assert_close(name, got[name].cpu().numpy(), stacked[name].cpu().numpy().astype(np.float64))
        else:
            assert torch.equal(got[name], stacked[name]), f"{name}: one-node-per-GPU and stacked results differ"
