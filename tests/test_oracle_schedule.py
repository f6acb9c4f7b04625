"""Pins for the oracle's mixing-matrix generator (CPU only).

Each test ties oracle/schedule.py to something the paper prints or the
mathematics fixes, so that a wrong orientation, hop, cycle length or weight
fails at least one of them.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import schedule as S
from conftest import read_golden


def _frac(tok):
    return float(Fraction(tok))


def test_four_node_worked_matrix_matches_paper():
    # Out-neighbour sets read off the printed matrix's columns: 0->{0,1}, 1->{1,2}, 2->{2,3}, 3->{0,1,3}.
    P = S.uniform_mixing_matrix([[0, 1], [1, 2], [2, 3], [0, 1, 3]])
    want = np.array([[_frac(t) for t in row] for row in read_golden("four_node_mixing_matrix.txt")])
    assert np.array_equal(P, want)
    assert np.allclose(P.sum(axis=0), 1.0, atol=0, rtol=0)            # column stochastic
    assert np.allclose(P.sum(axis=1), [5 / 6, 4 / 3, 1.0, 5 / 6])     # not row stochastic


def test_four_node_update_equations_orientation():
    P = S.uniform_mixing_matrix([[0, 1], [1, 2], [2, 3], [0, 1, 3]])
    rng = np.random.default_rng(0)
    x = rng.standard_normal((4, 3))
    want = np.zeros_like(x)
    for r, s, c in read_golden("four_node_update_equations.txt"):
        want[int(r)] += _frac(c) * x[int(s)]
    assert np.allclose(P @ x, want, rtol=1e-15, atol=1e-15)
    rowptr, col, val = S.csr_in_neighbours(P)
    assert rowptr.tolist() == [0, 2, 5, 7, 9]
    assert col.tolist() == [0, 3, 0, 1, 3, 1, 2, 2, 3]


def test_four_node_pushsum_weight_limit_closed_form():
    # w^(inf) = n * pi with P pi = pi (Sec. 2); for the worked matrix pi = (2,4,4,3)/13.
    P = S.uniform_mixing_matrix([[0, 1], [1, 2], [2, 3], [0, 1, 3]])
    w = np.ones(4)
    for _ in range(400):
        w = P @ w
    assert np.allclose(w, np.array([8, 16, 16, 12]) / 13.0, rtol=1e-13)
    evals, evecs = np.linalg.eig(P)
    pi = np.real(evecs[:, np.argmax(np.real(evals))])
    pi /= pi.sum()
    assert np.allclose(4 * pi, w, rtol=1e-12)


def test_exp_graph_direction_and_hops_n8():
    for step, peer in read_golden("exp_graph_n8_node0_peers.txt"):
        out = S.exp_out_neighbours(8, int(step), 1)
        assert out[0] == sorted({0, int(peer)})
        # period 3: the list repeats
        assert S.exp_out_neighbours(8, int(step) + 3, 1) == out
    # node i sends to (i + h) mod n  =>  P[(i+h) mod n, i] = 1/2 and the diagonal is 1/2
    P = S.mixing_matrix("exp", 8, 1, peers=1)
    for i in range(8):
        assert P[(i + 2) % 8, i] == 0.5 and P[i, i] == 0.5
        assert np.count_nonzero(P[:, i]) == 2


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 7, 8, 9, 16, 31, 32, 33, 64, 256])
def test_cycle_length(n):
    L = S.exp_cycle_length(n)
    if n == 1:
        assert L == 0
    else:
        # hop list 2^0 .. 2^floor(log2(n-1)): the largest hop is < n, the next one is not
        assert (1 << (L - 1)) <= n - 1 < (1 << L)
    if n & (n - 1) == 0 and n > 1:
        assert L == int(np.log2(n))


@pytest.mark.parametrize("n", [2, 4, 8, 16, 32, 64])
def test_one_peer_exact_consensus_after_log2n_steps(n):
    L = S.exp_cycle_length(n)
    rng = np.random.default_rng(n)
    y0 = rng.integers(-1000, 1000, size=(n, 5)).astype(np.float64) * n   # exact dyadic arithmetic
    y = y0.copy()
    for k in range(L):
        if k == L - 1 and n > 2:
            assert np.ptp(y, axis=0).max() > 0                           # not yet averaged
        y = S.mixing_matrix("exp", n, k, peers=1) @ y
    assert np.array_equal(y, np.broadcast_to(y0.mean(axis=0), y.shape))  # bit-exact average
    # and from any phase of the cycle
    y = y0.copy()
    for k in range(3, 3 + L):
        y = S.mixing_matrix("exp", n, k, peers=1) @ y
    assert np.array_equal(y, np.broadcast_to(y0.mean(axis=0), y.shape))


def _sigma2_sq(M):
    s = np.linalg.svd(M, compute_uv=False)
    return float(s[1] ** 2)


def test_averaging_quality_figures_n32():
    gold = {r[0]: (float(r[1]), float(r[2])) for r in read_golden("averaging_quality_n32.txt")}
    n = 32
    # deterministic exponential cycle
    M = np.eye(n)
    for k in range(5):
        M = S.mixing_matrix("exp", n, k, peers=1) @ M
    v, tol = gold["exp_cycle_deterministic"]
    assert abs(_sigma2_sq(M) - v) <= tol
    assert np.allclose(M, 1.0 / n, atol=1e-16)
    # cycling through the edges of the complete graph: hops 1, 2, 3, 4, 5
    M = np.eye(n)
    for hop in range(1, 6):
        M = S.uniform_mixing_matrix([sorted({i, (i + hop) % n}) for i in range(n)]) @ M
    v, tol = gold["complete_graph_cycle"]
    assert abs(_sigma2_sq(M) - v) <= tol
    # random peer among the exponential-graph neighbours / among all other nodes
    rng = np.random.default_rng(1811)
    acc_exp, acc_any, trials = 0.0, 0.0, 200
    for _ in range(trials):
        Me, Ma = np.eye(n), np.eye(n)
        for _k in range(5):
            hops = 1 << rng.integers(0, 5, size=n)
            Me = S.uniform_mixing_matrix([sorted({i, (i + int(hops[i])) % n}) for i in range(n)]) @ Me
            offs = rng.integers(1, n, size=n)
            Ma = S.uniform_mixing_matrix([sorted({i, (i + int(offs[i])) % n}) for i in range(n)]) @ Ma
        acc_exp += _sigma2_sq(Me)
        acc_any += _sigma2_sq(Ma)
    v, tol = gold["random_exp_peer_expected"]
    assert abs(acc_exp / trials - v) <= tol
    v, tol = gold["random_any_peer_expected"]
    assert abs(acc_any / trials - v) <= tol


def test_two_peer_structure():
    n = 16
    for k in range(8):
        P = S.mixing_matrix("exp", n, k, peers=2)
        L = 4
        for i in range(n):
            nz = set(np.nonzero(P[:, i])[0].tolist())
            assert nz == {i, (i + (1 << (k % L))) % n, (i + (1 << ((k + 1) % L))) % n}
            assert np.all(P[list(nz), i] == 1.0 / 3.0)
        assert np.allclose(P.sum(axis=1), 1.0)        # regular graph: also row stochastic
    # two-peer n=16 does not average exactly in 4 steps (unlike one-peer)
    M = np.eye(n)
    for k in range(4):
        M = S.mixing_matrix("exp", n, k, peers=2) @ M
    assert abs(np.sqrt(_sigma2_sq(M)) - 1.0 / 9.0) < 1e-12


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 16, 64, 256])
def test_every_kind_is_column_stochastic(n):
    mats = [S.mixing_matrix("exp", n, k, peers=p) for k in range(4) for p in (1, 2)]
    mats += [S.mixing_matrix("complete", n, 0)]
    mats += [S.mixing_matrix("random", n, k, seed=7, max_outdeg=4, num_steps=10) for k in range(12)]
    for P in mats:
        assert P.shape == (n, n)
        assert np.all(P >= 0)
        assert np.all(np.diag(P) > 0)                 # self-loop convention (Assumption 4)
        assert np.allclose(P.sum(axis=0), 1.0, rtol=0, atol=4e-16)


def test_complete_graph_is_uniform():
    assert np.array_equal(S.mixing_matrix("complete", 5, 3), np.full((5, 5), 0.2))


@pytest.mark.parametrize("n", [2, 4, 16, 64, 256])
def test_random_digraph_spec(n):
    seen_degrees = set()
    for k in range(10):
        out = S.random_out_neighbours(n, k, seed=42, max_outdeg=4)
        assert out == S.random_out_neighbours(n, k, seed=42, max_outdeg=4)   # pure function
        for i, targets in enumerate(out):
            assert i in targets and targets == sorted(set(targets))
            deg = len(targets) - 1
            assert 1 <= deg <= min(4, n - 1)
            assert all(0 <= t < n for t in targets)
            seen_degrees.add(deg)
    assert seen_degrees == set(range(1, min(4, n - 1) + 1))
    # different seeds / steps give different graphs, period wraps
    assert S.random_out_neighbours(n, 0, 42, 4) != S.random_out_neighbours(n, 0, 43, 4) or n == 2
    P10 = S.mixing_matrix("random", n, 13, seed=42, max_outdeg=4, num_steps=10)
    P3 = S.mixing_matrix("random", n, 3, seed=42, max_outdeg=4, num_steps=10)
    assert np.array_equal(P10, P3)


def test_mix64_known_vector():
    # splitmix64 generator seeded with 0: first output = finaliser applied to the golden-ratio increment.
    assert S.mix64(0x9E3779B97F4A7C15) == 0xE220A8397B1DCDAF


def test_fp32_weight_rounding_is_single_rounding_safe():
    # the compiled schedule stores float32(1/len); rounding the float64 quotient gives the same bits
    # as a float32 division for every out-degree that can occur (n <= 256 and beyond)
    for length in range(1, 1025):
        assert np.float32(1.0 / length) == np.float32(1.0) / np.float32(length)


# ---------------------------------------------------------------- App. A, undirected bipartite exponential graph
def test_bipartite_hop_list_matches_formula_in_paper():
    for row in read_golden("bipartite_exp_hops.txt"):
        n, hops = int(row[0]), [int(t) for t in row[1:]]
        assert S.bipartite_exp_hops(n) == hops
        assert S.schedule_period("bipartite", n) == len(hops)
    assert S.bipartite_exp_hops(2) == [1]
    with pytest.raises(ValueError):
        S.bipartite_exp_hops(7)


@pytest.mark.parametrize("n", [2, 4, 8, 16, 32, 6, 10, 12])
def test_bipartite_steps_are_perfect_odd_even_matchings(n):
    for k in range(2 * S.schedule_period("bipartite", n)):
        out = S.bipartite_exp_out_neighbours(n, k)
        P = S.mixing_matrix("bipartite", n, k)
        assert np.array_equal(P, P.T)                                    # undirected: message and reply
        assert np.allclose(P.sum(axis=0), 1.0, atol=0) and np.allclose(P.sum(axis=1), 1.0, atol=0)
        assert set(np.unique(P)) <= {0.0, 0.5}                           # self 1/2, partner 1/2 (App. C weights)
        hop = S.bipartite_exp_hops(n)[k % S.schedule_period("bipartite", n)]
        for i in range(n):
            assert len(out[i]) == 2 and i in out[i]                      # exactly one partner each: regular graph
            partner = [j for j in out[i] if j != i][0]
            assert partner % 2 != i % 2                                  # bipartite: odd talks to even
            if i % 2 == 1:
                assert partner == (i + hop) % n                          # odd nodes initiate, hop taken forwards


def test_bipartite_node1_partners_n8():
    # hops 1 and 3: node 1 pairs with node 2, then node 4; node 0 is reached by node 7 (hop 1) and node 5 (hop 3)
    assert S.bipartite_exp_out_neighbours(8, 0)[1] == [1, 2]
    assert S.bipartite_exp_out_neighbours(8, 1)[1] == [1, 4]
    assert S.bipartite_exp_out_neighbours(8, 0)[0] == [0, 7]
    assert S.bipartite_exp_out_neighbours(8, 1)[0] == [0, 5]


@pytest.mark.parametrize("n", [4, 8, 16, 32])
def test_bipartite_cycle_contracts_towards_the_average(n):
    # symmetric doubly stochastic steps keep the average and, over a few cycles, shrink every deviation from it
    L = S.schedule_period("bipartite", n)
    M = np.eye(n)
    for k in range(8 * L):
        M = S.mixing_matrix("bipartite", n, k) @ M
    assert np.allclose(M.sum(axis=0), 1.0) and np.allclose(M.sum(axis=1), 1.0)
    if n > 4:                                   # n = 4 has the single hop 1: two disjoint pairs never mix
        assert _sigma2_sq(M) < 1e-2
    else:
        assert abs(_sigma2_sq(M) - 1.0) < 1e-12
