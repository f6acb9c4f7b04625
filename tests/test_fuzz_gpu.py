"""Seeded random configurations of the fused step against the float64 oracle: node count, parameter count, row pitch
and pointer offset, delay, optimiser flavour, graph kind, kernel family, lockstep clusters and diagnostics are drawn
together, so that combinations no hand-written case lists get exercised (Alg. 1 lines 4-8, Alg. 2, Alg. 3)."""
import numpy as np
import pytest

from gpu_runner import compare_with_oracle, run_gpu


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


@pytest.mark.gpu
@pytest.mark.parametrize("case", range(256))
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
