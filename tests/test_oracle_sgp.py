"""Pins for the oracle's SGP recursion (CPU only).

The recursion is tied to: invariants of column-stochastic mixing, exact
rational brute force on tiny problems, the AllReduce and D-PSGD special cases
the paper names, a library optimiser for the n = 1 momentum update, the
augmented (virtual-node) matrix of the delay model, and hand-derived numbers.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import schedule as S
from oracle import sgp as O


def _rand_grads(n, d, K, seed):
    rng = np.random.default_rng(seed)
    G = rng.standard_normal((K, n, d))
    return G, (lambda k, z: G[k])


# ---------------------------------------------------------------- invariants
@pytest.mark.parametrize("tau", [0, 1, 2, 3])
@pytest.mark.parametrize("kind", ["exp1", "exp2", "random"])
def test_mass_conservation_every_step(kind, tau):
    n, d, K = 8, 6, 25
    rng = np.random.default_rng(3)
    x0 = rng.standard_normal((n, d))
    G, _ = _rand_grads(n, d, K, 4)

    def P_of_k(k):
        if kind == "exp1":
            return S.mixing_matrix("exp", n, k, peers=1)
        if kind == "exp2":
            return S.mixing_matrix("exp", n, k, peers=2)
        return S.mixing_matrix("random", n, k, seed=5, max_outdeg=4, num_steps=10)

    st = O.init_state(x0, tau)
    lr = 0.05
    for k in range(K):
        sx_before, sw_before = O.total_mass(st)
        O.sgp_step(st, G[k], P_of_k(k), lr)            # plain SGD: sum_i h_i = sum_i x_i - lr sum_i g_i
        sx_after, sw_after = O.total_mass(st)
        assert abs(sw_after - n) < 1e-12               # sum of push-sum weights (incl. in transit) = n
        assert np.allclose(sx_after, sx_before - lr * G[k].sum(axis=0), rtol=1e-12, atol=1e-12)
        assert np.allclose(st.z, st.x / st.w[:, None])
    if kind != "random" and tau == 0:
        assert np.array_equal(st.w, np.ones(n))        # regular graphs keep w = 1 (Sec. 5 remark on D-PSGD)
    if kind == "random":
        assert np.ptp(st.w) > 1e-3                     # irregular graph: weights really move


def test_brute_force_rational_products_tiny_n():
    # zero gradients: x^(K) = P^(K-1) ... P^(0) x^(0), w^(K) = P^(K-1) ... P^(0) 1, exactly, in rationals
    n, K = 5, 7
    x0_int = [[3, -1], [4, 1], [-5, 9], [2, -6], [5, 3]]
    mats = [S.mixing_matrix("random", n, k, seed=11, max_outdeg=3, num_steps=4) for k in range(K)]
    X = [[Fraction(v) for v in row] for row in x0_int]
    W = [Fraction(1)] * n
    for P in mats:
        PF = [[Fraction(P[i, j]).limit_denominator(64) for j in range(n)] for i in range(n)]
        X = [[sum(PF[i][j] * X[j][c] for j in range(n)) for c in range(2)] for i in range(n)]
        W = [sum(PF[i][j] * W[j] for j in range(n)) for i in range(n)]
    st = O.sgp_run(np.array(x0_int, dtype=float), K, lambda k: mats[k], lambda k, z: np.zeros((n, 2)), lr=0.1)
    assert np.allclose(st.x, [[float(v) for v in row] for row in X], rtol=1e-14, atol=1e-14)
    assert np.allclose(st.w, [float(v) for v in W], rtol=1e-14)
    assert np.allclose(st.z, [[float(X[i][c] / W[i]) for c in range(2)] for i in range(n)], rtol=1e-13)
    assert sum(W) == n


def test_debiased_ratio_recovers_average_on_asymmetric_graph():
    # PushSum (Sec. 2): y_i / w_i -> average although y_i alone -> pi_i * sum
    P = S.uniform_mixing_matrix([[0, 1], [1, 2], [2, 3], [0, 1, 3]])
    rng = np.random.default_rng(8)
    x0 = rng.standard_normal((4, 3))
    st = O.sgp_run(x0, 300, lambda k: P, lambda k, z: np.zeros_like(z), lr=1.0)
    assert np.allclose(st.z, np.broadcast_to(x0.mean(axis=0), (4, 3)), rtol=1e-12, atol=1e-12)
    pi = np.array([2, 4, 4, 3]) / 13.0
    assert np.allclose(st.x, pi[:, None] * x0.sum(axis=0)[None, :], rtol=1e-12, atol=1e-12)


def test_one_peer_consensus_through_the_full_recursion():
    n, d = 16, 4
    rng = np.random.default_rng(2)
    x0 = rng.integers(-50, 50, size=(n, d)).astype(float) * n
    st = O.sgp_run(x0, 4, lambda k: S.mixing_matrix("exp", n, k, peers=1), lambda k, z: np.zeros_like(z),
                   lr=0.1, momentum=0.9)
    assert np.array_equal(st.z, np.broadcast_to(x0.mean(axis=0), (n, d)))


# ---------------------------------------------------------------- special cases the paper names
def test_complete_graph_identical_init_is_parallel_sgd():
    # Sec. 3: every entry of P equal to 1/n and identical initial values == AllReduce parallel SGD
    n, d, K, lr = 6, 5, 12, 0.07
    rng = np.random.default_rng(1)
    x_row = rng.standard_normal(d)
    G, gfun = _rand_grads(n, d, K, 9)
    st = O.sgp_run(np.tile(x_row, (n, 1)), K, lambda k: S.mixing_matrix("complete", n, k), gfun, lr)
    want = x_row.copy()
    for k in range(K):
        want = want - lr * G[k].mean(axis=0)
    assert np.allclose(st.z, np.broadcast_to(want, (n, d)), rtol=1e-13, atol=1e-13)
    assert np.allclose(st.w, 1.0, rtol=1e-15)


def test_symmetric_doubly_stochastic_keeps_unit_weights():
    # Sec. 5: symmetric mixing weights => w = 1 always => D-PSGD:  x' = P (x - lr g)
    n, d, K, lr = 6, 3, 9, 0.1
    ring = np.zeros((n, n))
    for i in range(n):
        ring[i, i] = ring[i, (i + 1) % n] = ring[i, (i - 1) % n] = 1.0 / 3.0
    rng = np.random.default_rng(6)
    x0 = rng.standard_normal((n, d))
    G, gfun = _rand_grads(n, d, K, 10)
    st = O.sgp_run(x0, K, lambda k: ring, gfun, lr)
    x = x0.copy()
    for k in range(K):
        x = ring @ (x - lr * G[k])
    assert np.allclose(st.w, 1.0, rtol=0, atol=1e-15)
    assert np.allclose(st.z, x, rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("nesterov", [True, False])
@pytest.mark.parametrize("wd", [0.0, 1e-4, 0.3])
def test_single_node_matches_torch_sgd(nesterov, wd):
    # n = 1, P = [1]: Alg. 3 must be the library's momentum SGD (u0 = 0, weight decay on the stepped tensor)
    d, K, lr, m = 7, 15, 0.1, 0.9
    rng = np.random.default_rng(12)
    x0 = rng.standard_normal((1, d))
    G, gfun = _rand_grads(1, d, K, 13)
    st = O.sgp_run(x0, K, lambda k: np.ones((1, 1)), gfun, lr, momentum=m, nesterov=nesterov, weight_decay=wd)
    p = torch.tensor(x0[0].copy(), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=lr, momentum=m, nesterov=nesterov, weight_decay=wd)
    for k in range(K):
        p.grad = torch.tensor(G[k, 0].copy(), dtype=torch.float64)
        opt.step()
    assert np.allclose(st.x[0], p.detach().numpy(), rtol=1e-12, atol=1e-13)
    assert np.allclose(st.u[0], opt.state[p]["momentum_buffer"].numpy(), rtol=1e-12, atol=1e-13)


def test_plain_sgd_matches_torch_sgd():
    d, K, lr = 5, 10, 1e-3
    rng = np.random.default_rng(14)
    x0 = rng.standard_normal((1, d))
    G, gfun = _rand_grads(1, d, K, 15)
    st = O.sgp_run(x0, K, lambda k: np.ones((1, 1)), gfun, lr)
    p = torch.tensor(x0[0].copy(), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=lr)
    for k in range(K):
        p.grad = torch.tensor(G[k, 0].copy(), dtype=torch.float64)
        opt.step()
    assert np.allclose(st.x[0], p.detach().numpy(), rtol=1e-14, atol=1e-15)
    assert np.array_equal(st.u, np.zeros((1, d)))


def test_nesterov_two_steps_by_hand():
    # x0 = 1, g = 1, m = 0.9, lr = 0.1 (Alg. 3 lines 4-5):
    # u1 = 1,   x1 = 1 - 0.1 (0.9*1 + 1)     = 0.81
    # u2 = 1.9, x2 = 0.81 - 0.1 (0.9*1.9 + 1) = 0.539
    st = O.sgp_run(np.ones((1, 1)), 2, lambda k: np.ones((1, 1)), lambda k, z: np.ones((1, 1)), 0.1,
                   momentum=0.9, nesterov=True)
    assert abs(st.x[0, 0] - 0.539) < 1e-15 and abs(st.u[0, 0] - 1.9) < 1e-15


def test_gradients_are_evaluated_at_z_not_x():
    # quadratic f_i = 0.5 ||x - c_i||^2 on an irregular graph: the fixed point of the de-biased
    # iterates must be near mean(c); feeding x instead of z would drag it away because w != 1.
    n, d = 4, 3
    P = S.uniform_mixing_matrix([[0, 1], [1, 2], [2, 3], [0, 1, 3]])
    rng = np.random.default_rng(20)
    c = rng.standard_normal((n, d))
    seen = []

    def grad(k, z):
        seen.append(z.copy())
        return z - c

    hist = []
    st = O.sgp_run(np.zeros((n, d)), 4000, lambda k: P, grad, lr=0.002, history=hist)
    assert np.array_equal(seen[1], hist[0][3])                 # the z handed to step 1 is step 0's z
    assert not np.allclose(hist[0][3], hist[0][0])             # and it differs from x there
    assert np.allclose(st.z.mean(axis=0), c.mean(axis=0), atol=2e-2)
    assert np.abs(st.z - st.z.mean(axis=0)).max() < 2e-2       # near-consensus neighbourhood ~ lr


# ---------------------------------------------------------------- delay model
def _augmented_matrix(P, tau):
    """Block matrix of the delay model with every off-diagonal message delayed by exactly tau."""
    n = P.shape[0]
    A = np.zeros((n * (tau + 1), n * (tau + 1)))
    A[0:n, 0:n] = np.diag(np.diag(P))                                   # P~_0
    A[tau * n:(tau + 1) * n, 0:n] += P - np.diag(np.diag(P))            # P~_tau
    for r in range(tau):                                                # identity super-diagonal blocks
        A[r * n:(r + 1) * n, (r + 1) * n:(r + 2) * n] = np.eye(n)
    return A


@pytest.mark.parametrize("tau", [1, 2, 3])
@pytest.mark.parametrize("kind", ["exp", "random"])
def test_delayed_mix_equals_augmented_matrix_recursion(kind, tau):
    n, d, K, lr = 8, 4, 17, 0.05
    rng = np.random.default_rng(30 + tau)
    x0 = rng.standard_normal((n, d))
    G, gfun = _rand_grads(n, d, K, 31)

    def P_of_k(k):
        if kind == "exp":
            return S.mixing_matrix("exp", n, k, peers=1)
        return S.mixing_matrix("random", n, k, seed=77, max_outdeg=4, num_steps=6)

    hist = []
    O.sgp_run(x0, K, P_of_k, gfun, lr, tau=tau, history=hist)
    # Eq. 4 on the augmented state; virtual nodes start at 0 and take no gradient
    Xa = np.vstack([x0] + [np.zeros((n, d))] * tau)
    Wa = np.concatenate([np.ones(n)] + [np.zeros(n)] * tau)
    for k in range(K):
        A = _augmented_matrix(P_of_k(k), tau)
        assert np.allclose(A.sum(axis=0), 1.0)                          # still column stochastic
        Ga = np.vstack([G[k]] + [np.zeros((n, d))] * tau)
        Xa = A @ (Xa - lr * Ga)
        Wa = A @ Wa
        assert np.allclose(hist[k][0], Xa[:n], rtol=1e-13, atol=1e-13)
        assert np.allclose(hist[k][1], Wa[:n], rtol=1e-13, atol=1e-13)
        assert np.allclose(hist[k][3], Xa[:n] / Wa[:n, None], rtol=1e-12, atol=1e-12)


def test_one_osgp_weight_sequence_by_hand():
    # 1-peer graph, tau = 1 (Alg. 2): w1 = 1/2, w2 = 1/2*1/2 + 1/2*1 = 3/4, w3 = 1/2*3/4 + 1/2*1/2 = 5/8,
    # w_{k+1} = (w_k + w_{k-1}) / 2 -> 2/3: a third of the mass is always in transit.
    n = 8
    hist = []
    O.sgp_run(np.ones((n, 1)), 60, lambda k: S.mixing_matrix("exp", n, k, peers=1),
              lambda k, z: np.zeros_like(z), lr=0.1, tau=1, history=hist)
    for k, want in enumerate([0.5, 0.75, 0.625, 0.6875]):
        assert np.array_equal(hist[k][1], np.full(n, want))
    assert np.allclose(hist[-1][1], 2.0 / 3.0, rtol=1e-12)
    assert np.allclose(hist[-1][3], 1.0, rtol=1e-12)                    # z stays the true average


def test_tau_zero_equals_no_transit():
    n, d, K = 8, 3, 6
    rng = np.random.default_rng(40)
    x0 = rng.standard_normal((n, d))
    G, gfun = _rand_grads(n, d, K, 41)
    Pk = lambda k: S.mixing_matrix("exp", n, k, peers=2)
    a = O.sgp_run(x0, K, Pk, gfun, 0.1, momentum=0.9)
    x, u = x0.copy(), np.zeros_like(x0)
    for k in range(K):
        u = 0.9 * u + G[k]
        x = Pk(k) @ (x - 0.1 * (0.9 * u + G[k]))
    assert np.allclose(a.x, x, rtol=1e-14, atol=1e-14)
    assert np.allclose(a.u, u, rtol=1e-14, atol=1e-14)                  # momentum is local, never mixed


def test_debias_helper():
    x = np.arange(6, dtype=float).reshape(2, 3)
    assert np.array_equal(O.debias(x, [2.0, 0.5]), [[0, 0.5, 1.0], [6, 8, 10]])


# ---------------------------------------------------------------- Adam-SGP
@pytest.mark.parametrize("wd", [0.0, 1e-2])
def test_single_node_adam_matches_torch_adam(wd):
    # n = 1, P = [1]: the Adam half step must be the library's Adam (bias correction, eps outside the sqrt)
    d, K, lr, b1, b2, eps = 9, 25, 1e-2, 0.9, 0.98, 1e-8
    rng = np.random.default_rng(50)
    x0 = rng.standard_normal((1, d))
    G, gfun = _rand_grads(1, d, K, 51)
    st = O.sgp_run(x0, K, lambda k: np.ones((1, 1)), gfun, lr, weight_decay=wd, adam=(b1, b2, eps))
    p = torch.tensor(x0[0].copy(), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    for k in range(K):
        p.grad = torch.tensor(G[k, 0].copy(), dtype=torch.float64)
        opt.step()
    assert np.allclose(st.x[0], p.detach().numpy(), rtol=1e-11, atol=1e-13)
    assert np.allclose(st.u[0], opt.state[p]["exp_avg"].numpy(), rtol=1e-12, atol=1e-14)
    assert np.allclose(st.v[0], opt.state[p]["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-16)


def test_adam_first_step_by_hand():
    # t = 1: m_hat = g, v_hat = g^2  =>  h = x - lr * g / (|g| + eps) = x - lr * sign(g) (up to eps)
    x0 = np.array([[1.0, -2.0, 0.5]])
    g = np.array([[0.3, -4.0, 1e-3]])
    st = O.sgp_run(x0, 1, lambda k: np.ones((1, 1)), lambda k, z: g, 0.1, adam=(0.9, 0.999, 1e-12))
    assert np.allclose(st.x, x0 - 0.1 * np.sign(g), rtol=0, atol=1e-9)
    assert np.allclose(st.u, 0.1 * g) and np.allclose(st.v, 1e-3 * g * g)


def test_adam_sgp_moments_stay_local_and_mass_is_mixed():
    n, d, K = 8, 5, 6
    rng = np.random.default_rng(52)
    x0 = rng.standard_normal((n, d))
    G, gfun = _rand_grads(n, d, K, 53)
    Pk = lambda k: S.mixing_matrix("random", n, k, seed=9, max_outdeg=3, num_steps=5)
    st = O.sgp_run(x0, K, Pk, gfun, 1e-2, adam=(0.9, 0.99, 1e-8), tau=1)
    m = np.zeros((n, d)); v = np.zeros((n, d))
    for k in range(K):
        m = 0.9 * m + 0.1 * G[k]
        v = 0.99 * v + 0.01 * G[k] ** 2
    assert np.allclose(st.u, m, rtol=1e-13) and np.allclose(st.v, v, rtol=1e-13)     # independent of the graph
    _, sw = O.total_mass(st)
    assert abs(sw - n) < 1e-12


# ---------------------------------------------------------------- parameter deviation (Fig. 2 metric)
def test_param_deviation_closed_forms():
    a = np.array([3.0, -4.0, 12.0])
    # two nodes at +a and -a: the average is 0, each is ||a|| = 13 away
    assert np.allclose(O.param_deviation(np.stack([a, -a])), [13.0, 13.0])
    # a common shift changes nothing; consensus gives zero
    rng = np.random.default_rng(60)
    x = rng.standard_normal((6, 50))
    assert np.allclose(O.param_deviation(x + 7.5), O.param_deviation(x), rtol=1e-12)
    assert np.all(O.param_deviation(np.tile(x[0], (6, 1))) < 1e-14)
    # one node displaced by e from n-1 identical ones: it is (n-1)/n*||e|| away, the others ||e||/n
    e = rng.standard_normal(50)
    y = np.tile(x[0], (6, 1)); y[2] += e
    want = np.full(6, np.linalg.norm(e) / 6); want[2] *= 5
    assert np.allclose(O.param_deviation(y), want, rtol=1e-12)


# ---------------------------------------------------------------- Alg. 2 line 5 taken literally: send every s steps
@pytest.mark.parametrize("tau", [0, 1, 2, 3])
def test_send_period_one_is_the_fixed_delay_reading(tau):
    n, d, K = 8, 4, 9
    rng = np.random.default_rng(70 + tau)
    x0 = rng.standard_normal((n, d))
    _, gfun = _rand_grads(n, d, K, 71)
    Pk = lambda k: S.mixing_matrix("exp", n, k, peers=1)
    a = O.sgp_run(x0, K, Pk, gfun, 0.05, momentum=0.9, tau=tau)
    b = O.sgp_run(x0, K, Pk, gfun, 0.05, momentum=0.9, tau=tau, send_period=1)
    for f in ("x", "w", "u", "z"):
        assert np.array_equal(getattr(a, f), getattr(b, f))


def test_send_period_weight_sequence_by_hand():
    # n = 2, one-peer graph, tau = 2, transmissions on even steps only (Alg. 2 with send period tau).
    # w after steps 0..5: 1/2 (kept half, nothing arrives), 1/2 (no send, nothing arrives), 1/4 + 1/2 = 3/4
    # (the step-0 message lands), 3/4, 3/8 + 1/4 = 5/8 (the step-2 message was half of 1/2), 5/8: the 1-OSGP
    # sequence 1/2, 3/4, 5/8, ... with every entry held for two steps.
    hist = []
    O.sgp_run(np.ones((2, 1)), 8, lambda k: S.mixing_matrix("exp", 2, k, peers=1), lambda k, z: np.zeros_like(z),
              lr=0.1, tau=2, send_period=2, history=hist)
    got = [h[1][0] for h in hist]
    assert got == [0.5, 0.5, 0.75, 0.75, 0.625, 0.625, 0.6875, 0.6875]
    assert all(np.allclose(h[3], 1.0, rtol=1e-15) for h in hist)       # z keeps the average throughout


@pytest.mark.parametrize("tau,s", [(0, 2), (0, 3), (2, 2), (3, 3), (1, 2), (3, 2)])
def test_send_period_conserves_mass_and_idles_between_transmissions(tau, s):
    n, d, K = 8, 3, 13
    rng = np.random.default_rng(80)
    x0 = rng.standard_normal((n, d))
    G, gfun = _rand_grads(n, d, K, 81)
    lr = 0.1
    used = []

    def Pk(c):
        used.append(c)
        return S.mixing_matrix("exp", n, c, peers=1)

    st = O.init_state(x0, tau)
    for k in range(K):
        x_before, transit_arriving = st.x.copy(), (st.transit_x[0].copy() if tau else 0.0)
        mass_before, w_before = O.total_mass(st)
        P = Pk(k // s) if k % s == 0 else np.eye(n)
        O.sgp_step(st, G[k], P, lr)
        mass_after, w_after = O.total_mass(st)
        assert np.allclose(mass_after, mass_before - lr * G[k].sum(axis=0), rtol=0, atol=1e-13)
        assert abs(w_after - n) < 1e-13
        if k % s != 0:      # a node that does not transmit keeps its whole half step (Alg. 2 lines 10-11)
            assert np.array_equal(st.x, (x_before - lr * G[k]) + transit_arriving)
    # sgp_run hands the c-th transmission the c-th matrix of the schedule
    calls = []
    O.sgp_run(x0, K, lambda c: (calls.append(c), S.mixing_matrix("exp", n, c, peers=1))[1], gfun, lr, tau=tau,
              send_period=s)
    assert calls == list(range((K + s - 1) // s))


# ---------------------------------------------------------------- Table 4: biased 1-OSGP (push-sum weight not used)
def test_biased_osgp_closed_form():
    # identical constant rows c, zero gradients, one-peer graph, tau = 1: the numerators shrink with the weights,
    # x_i^(k) = c * w^(k) with w = 1/2, 3/4, 5/8, ... -> 2/3.  The de-biased z stays c; the biased one is x.
    n, c = 8, np.array([3.0, -1.5, 0.25])
    x0 = np.tile(c, (n, 1))
    hist_b, hist_u = [], []
    kw = dict(lr=0.1, tau=1)
    O.sgp_run(x0, 40, lambda k: S.mixing_matrix("exp", n, k, peers=1), lambda k, z: np.zeros_like(z), biased=True,
              history=hist_b, **kw)
    O.sgp_run(x0, 40, lambda k: S.mixing_matrix("exp", n, k, peers=1), lambda k, z: np.zeros_like(z),
              history=hist_u, **kw)
    for k, wk in enumerate([0.5, 0.75, 0.625]):
        assert np.allclose(hist_b[k][3], wk * x0, rtol=1e-15)
        assert np.array_equal(hist_b[k][3], hist_b[k][0])               # z is the numerator itself
        assert np.allclose(hist_u[k][3], x0, rtol=1e-15)
        assert np.array_equal(hist_b[k][1], hist_u[k][1])               # the weights themselves are mixed as usual
    assert np.allclose(hist_b[-1][3], (2.0 / 3.0) * x0, rtol=1e-9)


def test_biased_flag_is_invisible_without_delay_on_regular_graphs():
    n, d, K = 8, 3, 6
    rng = np.random.default_rng(90)
    x0 = rng.standard_normal((n, d))
    _, gfun = _rand_grads(n, d, K, 91)
    Pk = lambda k: S.mixing_matrix("exp", n, k, peers=2)
    a = O.sgp_run(x0, K, Pk, gfun, 0.1, momentum=0.9)
    b = O.sgp_run(x0, K, Pk, gfun, 0.1, momentum=0.9, biased=True)
    assert np.allclose(a.z, b.z, rtol=1e-14, atol=1e-14)                 # w == 1: nothing to ignore


# ---------------------------------------------------------------- half step accessor and consensus distance
def test_half_step_accessor_closed_form():
    # plain SGD: the half step is x - lr g whatever the graph; the mix is applied to exactly that
    n, d = 4, 5
    rng = np.random.default_rng(100)
    x0 = rng.standard_normal((n, d))
    G, gfun = _rand_grads(n, d, 3, 101)
    halves, hist = [], []
    P = lambda k: S.mixing_matrix("exp", n, k, peers=1)
    O.sgp_run(x0, 3, P, gfun, 0.25, half_steps=halves, history=hist)
    assert np.array_equal(halves[0], x0 - 0.25 * G[0])
    for k in range(3):
        assert np.allclose(hist[k][0], P(k) @ halves[k], rtol=1e-15, atol=1e-15)
    # two nodes at a and b after the gradient step: each is ||a - b|| / 2 from their mean (Fig. 2 metric)
    a, b = np.array([1.0, 2.0, 2.0]), np.array([-2.0, -2.0, 2.0])
    halves = []
    O.sgp_run(np.stack([a, b]), 1, lambda k: S.mixing_matrix("complete", 2, k), lambda k, z: np.zeros_like(z), 0.1,
              half_steps=halves)
    assert np.allclose(O.param_deviation(halves[0]), [2.5, 2.5])


def test_consensus_distance_counts_mass_in_transit():
    # n = 2, one-peer graph, tau = 1, zero gradients, rows a and b.  After one step x = (a/2, b/2), the messages
    # (b/2, a/2) are in transit, w = 1/2 so z = (a, b).  xbar counts the transit: (a + b)/2, so both nodes are
    # |a - b|/2 away; leaving the transit out would give xbar = (a + b)/4 instead.
    a, b = np.array([4.0, 0.0]), np.array([0.0, 3.0])
    st = O.sgp_run(np.stack([a, b]), 1, lambda k: S.mixing_matrix("exp", 2, k, peers=1),
                   lambda k, z: np.zeros_like(z), 0.1, tau=1)
    assert np.allclose(st.z, np.stack([a, b]))
    assert np.allclose(O.consensus_distance(st), [2.5, 2.5])
    # complete graph, no delay: every z is the average, distance 0
    st = O.sgp_run(np.stack([a, b]), 1, lambda k: S.mixing_matrix("complete", 2, k), lambda k, z: np.zeros_like(z), 0.1)
    assert np.all(O.consensus_distance(st) < 1e-15)
    # asymmetric 4-node graph: distances shrink geometrically towards zero (consensus lemma)
    P = np.array([[1/2, 0, 0, 1/3], [1/2, 1/2, 0, 1/3], [0, 1/2, 1/2, 0], [0, 0, 1/2, 1/3]])
    x0 = np.random.default_rng(110).standard_normal((4, 6))
    d10 = O.consensus_distance(O.sgp_run(x0, 10, lambda k: P, lambda k, z: np.zeros_like(z), 0.1))
    d40 = O.consensus_distance(O.sgp_run(x0, 40, lambda k: P, lambda k, z: np.zeros_like(z), 0.1))
    assert d40.max() < 1e-3 * d10.max()


def test_bipartite_graph_keeps_unit_weights_d_psgd_case():
    # symmetric doubly stochastic mixing (the D-PSGD topology of App. A): w == 1 at every step, z == x
    n, d, K = 8, 4, 7
    rng = np.random.default_rng(120)
    x0 = rng.standard_normal((n, d))
    _, gfun = _rand_grads(n, d, K, 121)
    hist = []
    O.sgp_run(x0, K, lambda k: S.mixing_matrix("bipartite", n, k), gfun, 0.1, momentum=0.9, history=hist)
    for x, w, u, z in hist:
        assert np.array_equal(w, np.ones(n)) and np.array_equal(z, x)
