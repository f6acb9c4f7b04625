"""Float64 oracle of the SGP / momentum-SGP / overlap-SGP recursion (test infrastructure).

Written from Alg. 1 (SGP), Alg. 3 (SGP with Nesterov momentum) and Alg. 2
(Overlap SGP) read through the supplementary delay model (virtual nodes, block
mixing matrix, Eq. 4).  State is stacked by node: ``x`` is ``n x d`` (push-sum
numerators), ``w`` is ``n`` (push-sum weights), ``u`` is ``n x d`` (momentum,
never gossiped), ``z = x / w`` (de-biased parameters).

Everything is float64 numpy, one statement per line of the algorithms, dense
``P @ h`` for the mix.  No blocking, no fusion, nothing shared with the CUDA
path.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
import this module.

Readings fixed here where the paper leaves a choice:
  * K steps means k = 0 .. K-1; u^(0) = 0; w^(0) = 1; z^(0) = x^(0).
  * Weight decay adds lambda * x (the biased numerator the optimiser steps on,
    App. C description of the compute thread) to the gradient.
  * Adam: Sec. 6.2 / App. C.1 run Adam-preconditioned SGP on the Transformer without a listing.  Reading: the bias-corrected Adam step of Kingma & Ba replaces
    Alg. 3 lines 4-5 (gradient taken at z, step applied to the numerator x, both moment vectors local
    to a node and never gossiped); weight decay is added to the gradient as for SGD.
  * Delay tau: the self term p_ii h_i is never delayed; every other message
    (p_ij h_j, p_ij w_j) sent at step k is added at step k + tau, i.e. it lands
    in x^(k+tau+1); messages are sent every step; both parts accumulate;
    virtual nodes start at zero.  For tau = 1 this is Alg. 2 (Table 4 caption:
    fixed 1-step delay).
  * send_period s (Alg. 2 line 5 taken literally with s = tau; Sec. 3: nodes send every tau
    iterations): a node sends only on steps with k mod s = 0; on every other step it keeps its
    whole half step (Alg. 2 lines 10-11: the step's mixing matrix is the identity), while messages
    sent earlier still arrive tau steps after they were sent.  The c-th transmission uses the
    c-th matrix of the schedule, P^(k/s) (App. A describes the peer cycle per transmission).
    s = 1 is the reading above.
  * biased (Sec. 6.1 / Table 4, "biased 1-OSGP": the push-sum weight is not used): z = x; the
    weights are still mixed so that they can be inspected, they just do not enter z.

Pins: tests/test_oracle_sgp.py.
"""
from __future__ import annotations

from collections import deque
from dataclasses import dataclass, field

import numpy as np


@dataclass
class SGPState:
    x: np.ndarray                      # n x d numerators
    w: np.ndarray                      # n push-sum weights
    u: np.ndarray                      # n x d momentum buffers
    z: np.ndarray                      # n x d de-biased parameters
    v: np.ndarray = None               # n x d Adam second moments (u holds the first moments)
    h: np.ndarray = None               # n x d half step x^(k+1/2) of the latest iteration (before the mix)
    transit_x: deque = field(default_factory=deque)   # tau in-flight (n x d) messages, oldest first
    transit_w: deque = field(default_factory=deque)   # tau in-flight (n) weight messages


def init_state(x0, tau: int = 0) -> SGPState:
    """Alg. 1 'Require' line: w = 1, z = x; Alg. 3: u = 0; virtual nodes hold 0."""
    x = np.array(x0, dtype=np.float64)
    n, d = x.shape
    st = SGPState(x=x, w=np.ones(n), u=np.zeros((n, d)), z=x.copy(), v=np.zeros((n, d)))
    for _ in range(tau):
        st.transit_x.append(np.zeros((n, d)))
        st.transit_w.append(np.zeros(n))
    return st


def local_update(x, u, g, lr, momentum=0.0, nesterov=True, weight_decay=0.0):
    """Half step x^(k+1/2) on the numerators (Alg. 1 line 4 / Alg. 3 lines 4-5).

    Returns (h, u_next) with h = x^(k+1/2).
    """
    g = np.asarray(g, dtype=np.float64)
    if weight_decay != 0.0:
        g = g + weight_decay * x
    if momentum != 0.0:
        u_next = momentum * u + g                      # Alg. 3 line 4
        if nesterov:
            s = momentum * u_next + g                  # Alg. 3 line 5
        else:
            s = u_next                                 # classical (heavy-ball) momentum
    else:
        u_next = u
        s = g                                          # Alg. 1 line 4
    h = x - lr * s
    return h, u_next


def local_update_adam(x, m, v, g, t, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0):
    """Half step with the Adam preconditioner; t = 1, 2, ... counts the steps taken including this one.

    Returns (h, m_next, v_next).
    """
    g = np.asarray(g, dtype=np.float64)
    if weight_decay != 0.0:
        g = g + weight_decay * x
    m_next = beta1 * m + (1.0 - beta1) * g
    v_next = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m_next / (1.0 - beta1 ** t)
    v_hat = v_next / (1.0 - beta2 ** t)
    h = x - lr * m_hat / (np.sqrt(v_hat) + eps)
    return h, m_next, v_next


def mix(P, h, w):
    """One PushSum iteration, no delay (Alg. 1 lines 6-7): x' = P h, w' = P w."""
    return P @ h, P @ w


def mix_delayed(P, h, w, transit_x, transit_w):
    """One PushSum iteration where every off-diagonal message is tau steps late.

    Block form of the augmented matrix: P~_0 = diag(P) acts now, P~_tau =
    P - diag(P) enters the far end of the delay chain, virtual nodes forward.
    ``transit_*`` hold exactly tau messages, oldest first.
    """
    diag = np.diag(P)
    off = P - np.diag(diag)
    arriving_x = transit_x.popleft()
    arriving_w = transit_w.popleft()
    x_next = diag[:, None] * h + arriving_x            # Alg. 2 lines 7, 21
    w_next = diag * w + arriving_w                     # Alg. 2 lines 8, 22 (accumulating)
    transit_x.append(off @ h)                          # Alg. 2 line 6 (non-blocking send)
    transit_w.append(off @ w)
    return x_next, w_next


def sgp_step(st: SGPState, g, P, lr, momentum=0.0, nesterov=True, weight_decay=0.0, adam=None,
             biased=False) -> SGPState:
    """One full SGP iteration in place on ``st`` (gradient g was taken at st.z).

    ``adam`` = (t, beta1, beta2, eps) switches the local update to Adam.  ``biased`` leaves the
    push-sum weight out of z (Table 4, biased 1-OSGP).  The half step is kept in ``st.h``.
    """
    if adam is None:
        h, st.u = local_update(st.x, st.u, g, lr, momentum, nesterov, weight_decay)
    else:
        t, beta1, beta2, eps = adam
        h, st.u, st.v = local_update_adam(st.x, st.u, st.v, g, t, lr, beta1, beta2, eps, weight_decay)
    st.h = h
    if len(st.transit_x) == 0:
        st.x, st.w = mix(P, h, st.w)
    else:
        st.x, st.w = mix_delayed(P, h, st.w, st.transit_x, st.transit_w)
    if biased:
        st.z = st.x.copy()                             # Table 4, biased 1-OSGP: w ignored
    else:
        st.z = st.x / st.w[:, None]                    # Alg. 1 line 8
    return st


def sgp_run(x0, K, P_of_k, grad_of_k, lr, momentum=0.0, nesterov=True, weight_decay=0.0,
            tau=0, history=None, adam=None, send_period=1, biased=False, half_steps=None) -> SGPState:
    """K iterations k = 0 .. K-1.

    ``P_of_k(k)`` returns the dense mixing matrix of step k; ``grad_of_k(k, z)``
    returns the n x d stochastic gradients evaluated at the de-biased ``z``.
    If ``history`` is a list, a snapshot (x, w, u, z) is appended after every step.
    ``adam`` = (beta1, beta2, eps) runs Adam-SGP (step count t = k + 1).
    ``send_period`` = s: nodes transmit on steps k = 0, s, 2s, ... with the matrix P_of_k(k // s) and keep
    everything (identity matrix) on the other steps (Alg. 2 lines 5-12).  If ``half_steps`` is a list the
    half step x^(k+1/2) of every iteration is appended to it.
    """
    st = init_state(x0, tau)
    n = st.x.shape[0]
    for k in range(K):
        g = grad_of_k(k, st.z)
        P = P_of_k(k // send_period) if k % send_period == 0 else np.eye(n)
        sgp_step(st, g, P, lr, momentum, nesterov, weight_decay,
                 adam=None if adam is None else (k + 1, *adam), biased=biased)
        if history is not None:
            history.append((st.x.copy(), st.w.copy(), st.u.copy(), st.z.copy()))
        if half_steps is not None:
            half_steps.append(st.h.copy())
    return st


def debias(x, w):
    """z_i = x_i / w_i (Alg. 1 line 8)."""
    return np.asarray(x, dtype=np.float64) / np.asarray(w, dtype=np.float64)[:, None]


def total_mass(st: SGPState):
    """(sum of x over real and in-transit nodes, same for w): conserved by the mix."""
    sx = st.x.sum(axis=0)
    sw = st.w.sum()
    for mx, mw in zip(st.transit_x, st.transit_w):
        sx = sx + mx.sum(axis=0)
        sw = sw + mw.sum()
    return sx, sw


def consensus_distance(st: SGPState):
    """|| xbar - z_i ||_2 for every node, xbar = (1/n) * (sum of x over real AND virtual nodes).

    The quantity bounded by the consensus lemma of the supplementary material; the node-wise average
    counts the parameters that are in transit (definition of xbar after Eq. 4).
    """
    sx, _ = total_mass(st)
    xbar = sx / st.x.shape[0]
    return np.linalg.norm(st.z - xbar[None, :], axis=1)


def param_deviation(a):
    """Sec. 6.1 "Parameter deviations": distance of every node's row from the node-wise average row."""
    a = np.asarray(a, dtype=np.float64)
    return np.linalg.norm(a - a.mean(axis=0, keepdims=True), axis=1)
