"""Oracle generator of the time-varying mixing matrices P^(k) (test infrastructure).

Conventions (Sec. 2 "Approximate distributed averaging"; supplementary
"Modeling message delays", worked 4-node example): nodes are 0-indexed,
``P[i, j] = p_ij`` is the weight receiver ``i`` applies to sender ``j`` (rows =
receivers, columns = senders), every node is an out-neighbour of itself, and
each column of P sums to one.

All matrices are dense float64 ``n x n`` arrays: this module exists to be
checked by eye against the paper, not to be fast.  It shares no code with the
CUDA library's schedule compiler.

Pins (tests/test_oracle_schedule.py): the worked 4-node matrix and its update
equations, exact consensus after log2(n) one-peer steps, the averaging-quality
figures quoted in App. A for n = 32, column-stochasticity of every kind, the bipartite graph's perfect
odd-even matching and symmetry.
"""
from __future__ import annotations

import numpy as np

_MASK64 = (1 << 64) - 1


# --------------------------------------------------------------------------
# App. A, "Directed exponential graph"
# --------------------------------------------------------------------------
def exp_cycle_length(n: int) -> int:
    """Number of distinct hop distances 2^0 .. 2^floor(log2(n-1)) (App. A).

    App. A lists the peers as 2^0, ..., 2^floor(log2(n-1)) hops away, i.e.
    floor(log2(n-1)) + 1 of them, and states that n = 32 reaches the exact
    average after 5 steps; the cycle therefore has floor(log2(n-1)) + 1
    entries (log2 n for powers of two).  n = 1 has no peers.
    """
    if n < 1:
        raise ValueError("n must be >= 1")
    if n == 1:
        return 0
    return (n - 1).bit_length()  # floor(log2(n-1)) + 1, integer-exact


def exp_out_neighbours(n: int, k: int, peers: int) -> list[list[int]]:
    """Out-neighbour sets (self included) of the c-peer exponential schedule.

    At step k every node i sends to (i + 2^((k + t) mod L)) mod n for
    t = 0 .. peers-1 (App. A: one-peer cycles through the hop list, two-peer
    uses two consecutive entries of it).  Targets form a set: coinciding
    targets (tiny n) are sent to once, and a target equal to the sender itself
    is just the self-loop.
    """
    L = exp_cycle_length(n)
    out = []
    for i in range(n):
        s = {i}
        for t in range(peers if L > 0 else 0):
            hop = 1 << ((k + t) % L)
            s.add((i + hop) % n)
        out.append(sorted(s))
    return out


def bipartite_exp_hops(n: int) -> list[int]:
    """Hop distances of the undirected bipartite exponential graph (App. A, "Undirected exponential graph").

    Odd-numbered nodes pair with the even-numbered nodes 2^1 - 1, 2^2 - 1, ..., 2^floor(log2(n-1)) - 1 hops
    away.  Reading for n = 2, where that list is empty: the single hop 1 (the only even node there is).
    """
    if n < 2 or n % 2 != 0:
        raise ValueError("the bipartite exponential graph needs an even number of nodes")
    top = (n - 1).bit_length() - 1               # floor(log2(n-1))
    return [(1 << j) - 1 for j in range(1, top + 1)] or [1]


def bipartite_exp_out_neighbours(n: int, k: int) -> list[list[int]]:
    """Out-neighbour sets (self included) of step k of the undirected bipartite exponential graph.

    Odd node i sends to the even node (i + hop_k) mod n and that node sends back to i (App. A: the odd
    node waits for the message in return), the hop cycling through `bipartite_exp_hops` one entry per
    step like the one-peer directed schedule.  Every node therefore has exactly one partner per step
    and the edge set is symmetric.
    """
    hops = bipartite_exp_hops(n)
    hop = hops[k % len(hops)]
    partner = [None] * n
    for i in range(1, n, 2):                     # odd nodes initiate
        j = (i + hop) % n
        partner[i] = j
        partner[j] = i
    return [sorted({i, partner[i]}) for i in range(n)]


def complete_out_neighbours(n: int) -> list[list[int]]:
    """Every node sends to every node: P = (1/n) 1 1^T (Sec. 3, AllReduce case)."""
    return [list(range(n)) for _ in range(n)]


# --------------------------------------------------------------------------
# Random time-varying digraph (not from the paper: the scaling-sweep workload).
# An integer-only keyed hash so that two independent implementations can agree
# bit for bit.  mix64 is the published splitmix64 finaliser.
# --------------------------------------------------------------------------
def mix64(x: int) -> int:
    x &= _MASK64
    x ^= x >> 30
    x = (x * 0xBF58476D1CE4E5B9) & _MASK64
    x ^= x >> 27
    x = (x * 0x94D049BB133111EB) & _MASK64
    x ^= x >> 31
    return x


def graph_hash(seed: int, k: int, i: int, t: int) -> int:
    """64-bit draw number t of node i at step k."""
    a = mix64((seed + 0x9E3779B97F4A7C15) & _MASK64)
    b = mix64(a ^ (k & _MASK64))
    return mix64(b ^ (((i & 0xFFFFFFFF) << 32) | (t & 0xFFFFFFFF)))


def random_out_neighbours(n: int, k: int, seed: int, max_outdeg: int) -> list[list[int]]:
    """Out-degree ~ U{1..min(max_outdeg, n-1)}, distinct targets != self, plus self.

    Draw 0 fixes the out-degree, draws 1, 2, ... propose targets ``h mod n``;
    a proposal equal to the sender or to an earlier target is skipped.
    """
    out = []
    cap = min(max_outdeg, n - 1)
    for i in range(n):
        chosen = {i}
        if cap >= 1:
            deg = 1 + graph_hash(seed, k, i, 0) % cap
            t = 1
            while len(chosen) < deg + 1:
                c = graph_hash(seed, k, i, t) % n
                t += 1
                if c not in chosen:
                    chosen.add(c)
        out.append(sorted(chosen))
    return out


# --------------------------------------------------------------------------
# App. C: uniform mixing weights p_ji = 1 / |N_out_i| (self included)
# --------------------------------------------------------------------------
def uniform_mixing_matrix(out_sets: list[list[int]]) -> np.ndarray:
    n = len(out_sets)
    P = np.zeros((n, n), dtype=np.float64)
    for j, targets in enumerate(out_sets):       # j = sender = column
        for i in targets:                        # i = receiver = row
            P[i, j] = 1.0 / len(targets)
    return P


def custom_mixing_matrix(n: int, senders, receivers, weights) -> np.ndarray:
    """Dense P from an explicit edge list (sender j -> receiver i with weight p_ij)."""
    P = np.zeros((n, n), dtype=np.float64)
    for j, i, p in zip(senders, receivers, weights):
        P[int(i), int(j)] = float(p)
    return P


def mixing_matrix(kind: str, n: int, k: int, *, peers: int = 1, seed: int = 0,
                  max_outdeg: int = 4, num_steps: int = 0) -> np.ndarray:
    """P^(k) for the named schedule.

    ``exp``: c-peer directed exponential graph; ``complete``: all-to-all;
    ``bipartite``: undirected bipartite exponential graph (symmetric pairs);
    ``random``: the hashed random digraph, repeating with period ``num_steps``.
    """
    if kind == "exp":
        return uniform_mixing_matrix(exp_out_neighbours(n, k, peers))
    if kind == "complete":
        return uniform_mixing_matrix(complete_out_neighbours(n))
    if kind == "bipartite":
        return uniform_mixing_matrix(bipartite_exp_out_neighbours(n, k))
    if kind == "random":
        kk = k % num_steps if num_steps > 0 else k
        return uniform_mixing_matrix(random_out_neighbours(n, kk, seed, max_outdeg))
    raise ValueError(f"unknown schedule kind {kind!r}")


def schedule_period(kind: str, n: int, *, peers: int = 1, num_steps: int = 0) -> int:
    if kind == "exp":
        return max(1, exp_cycle_length(n))
    if kind == "complete":
        return 1
    if kind == "bipartite":
        return len(bipartite_exp_hops(n))
    if kind == "random":
        return num_steps
    raise ValueError(kind)


def csr_in_neighbours(P: np.ndarray):
    """Receiver-major lists of P: (rowptr, col, val) with senders ascending.

    ``val`` stays float64; the compiled schedule's fp32 weight must equal
    ``np.float32(val)`` bit for bit.
    """
    n = P.shape[0]
    rowptr = [0]
    col, val = [], []
    for i in range(n):
        for j in range(n):
            if P[i, j] != 0.0:
                col.append(j)
                val.append(P[i, j])
        rowptr.append(len(col))
    return (np.asarray(rowptr, dtype=np.int32), np.asarray(col, dtype=np.int32),
            np.asarray(val, dtype=np.float64))
