"""Graph-schedule compiler (C++ host code behind the C ABI) against the oracle's generator: bit-exact
in-neighbour lists and fp32 weights; validation of custom graphs; ABI surface.  CPU only."""
import ctypes as C
import os
import re

from fractions import Fraction

import numpy as np
import pytest

from oracle import schedule as S
from conftest import ROOT, read_golden


@pytest.fixture(scope="module")
def binding():
    from paper_1811_10792_b200 import build
    build.build()
    from paper_1811_10792_b200 import binding as b
    return b


def _assert_slot_equal(sched, k, P):
    rowptr, col, val = sched.get(k)
    o_rowptr, o_col, o_val = S.csr_in_neighbours(P)
    assert np.array_equal(rowptr, o_rowptr)
    assert np.array_equal(col, o_col)
    want = o_val.astype(np.float32)
    assert np.array_equal(val.view(np.int32), want.view(np.int32))      # bit-exact weights


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 8, 13, 16, 32, 64, 100, 256])
@pytest.mark.parametrize("peers", [1, 2, 3])
def test_exp_peers_bit_exact(binding, n, peers):
    sched = binding.Schedule(n, binding.GraphDesc.exp_peers(peers))
    assert sched.period == S.schedule_period("exp", n)
    for k in range(2 * sched.period + 1):
        _assert_slot_equal(sched, k, S.mixing_matrix("exp", n, k, peers=peers))


@pytest.mark.parametrize("n", [1, 2, 7, 32, 256])
def test_complete_bit_exact(binding, n):
    sched = binding.Schedule(n, binding.GraphDesc.complete())
    assert sched.period == 1
    _assert_slot_equal(sched, 5, S.mixing_matrix("complete", n, 5))
    assert sched.nnz(0) == n * n


@pytest.mark.parametrize("n", [1, 2, 4, 16, 64, 256])
@pytest.mark.parametrize("seed,max_outdeg,steps", [(181110797, 4, 10), (3, 1, 3), (2**63 + 5, 7, 4)])
def test_random_outdeg_bit_exact(binding, n, seed, max_outdeg, steps):
    sched = binding.Schedule(n, binding.GraphDesc.random_outdeg(seed, steps, max_outdeg))
    assert sched.period == steps
    for k in range(steps + 2):
        _assert_slot_equal(sched, k, S.mixing_matrix("random", n, k, seed=seed, max_outdeg=max_outdeg,
                                                     num_steps=steps))


@pytest.mark.parametrize("n", [2, 4, 6, 8, 10, 16, 32, 64, 100, 256])
def test_bipartite_exp_bit_exact(binding, n):
    sched = binding.Schedule(n, binding.GraphDesc.bipartite_exp())
    assert sched.period == S.schedule_period("bipartite", n)
    for k in range(2 * sched.period + 1):
        _assert_slot_equal(sched, k, S.mixing_matrix("bipartite", n, k))


@pytest.mark.parametrize("n", [1, 3, 7, 255])
def test_bipartite_exp_needs_an_even_node_count(binding, n):
    with pytest.raises(binding.SgpError) as e:
        binding.Schedule(n, binding.GraphDesc.bipartite_exp())
    assert e.value.code == binding.SGP_ERR_ARG


def _four_node_edges():
    rows = read_golden("four_node_update_equations.txt")
    recv = [int(r[0]) for r in rows]
    send = [int(r[1]) for r in rows]
    wt = [float(Fraction(r[2])) for r in rows]     # "1/2", "1/3"
    return send, recv, wt


def test_custom_graph_four_node_example(binding):
    send, recv, wt = _four_node_edges()
    g = binding.GraphDesc.custom(1, [0] * len(send), send, recv, wt)
    sched = binding.Schedule(4, g)
    P = S.custom_mixing_matrix(4, send, recv, np.asarray(wt, dtype=np.float32))
    _assert_slot_equal(sched, 0, P)
    rowptr, col, val = sched.get(0)
    assert rowptr.tolist() == [0, 2, 5, 7, 9]
    assert col.tolist() == [0, 3, 0, 1, 3, 1, 2, 2, 3]


def test_custom_graph_two_steps_any_edge_order(binding):
    # step 0: ring 0->1->2->0 with self-loops (1/2 each); step 1: node 0 broadcasts, others keep
    step = [1, 0, 0, 0, 1, 0, 0, 1, 1, 0, 1]
    send = [0, 2, 0, 1, 0, 0, 2, 2, 1, 1, 0]
    recv = [2, 0, 1, 1, 1, 0, 2, 2, 1, 2, 0]
    wt = [1 / 3, .5, .5, .5, 1 / 3, .5, .5, 1.0, 1.0, .5, 1 / 3]
    sched = binding.Schedule(3, binding.GraphDesc.custom(2, step, send, recv, wt))
    assert sched.period == 2
    for k in (0, 1):
        sel = [e for e in range(len(step)) if step[e] == k]
        P = S.custom_mixing_matrix(3, [send[e] for e in sel], [recv[e] for e in sel],
                                   np.asarray([wt[e] for e in sel], dtype=np.float32))
        _assert_slot_equal(sched, k, P)
        assert np.allclose(P.sum(axis=0), 1.0, atol=1e-7)


@pytest.mark.parametrize("mutate", ["colsum", "no_self", "dup", "range", "neg", "nan", "step_range"])
def test_custom_graph_rejected(binding, mutate):
    send, recv, wt = _four_node_edges()
    step = [0] * len(send)
    if mutate == "colsum":
        wt[0] = 0.6
    elif mutate == "no_self":
        # drop node 2's self-loop and give its whole mass to node 3
        idx = [e for e in range(len(send)) if send[e] == 2 and recv[e] == 2][0]
        del send[idx], recv[idx], wt[idx], step[idx]
        wt[[e for e in range(len(send)) if send[e] == 2][0]] = 1.0
    elif mutate == "dup":
        send.append(send[0]); recv.append(recv[0]); wt.append(wt[0]); step.append(0)
    elif mutate == "range":
        recv[1] = 4
    elif mutate == "neg":
        wt[2] = -0.5
    elif mutate == "nan":
        wt[2] = float("nan")
    elif mutate == "step_range":
        step[3] = 1
    with pytest.raises(binding.SgpError) as ei:
        binding.Schedule(4, binding.GraphDesc.custom(1, step, send, recv, wt))
    assert ei.value.code == binding.SGP_ERR_GRAPH


def test_bad_arguments(binding):
    for n in (0, -1, binding.SGP_MAX_NODES + 1):
        with pytest.raises(binding.SgpError) as ei:
            binding.Schedule(n, binding.GraphDesc.exp_peers(1))
        assert ei.value.code == binding.SGP_ERR_ARG
    for g in (binding.GraphDesc.exp_peers(0), binding.GraphDesc.random_outdeg(1, 0, 4),
              binding.GraphDesc.random_outdeg(1, 5, 0), binding.GraphDesc(kind=17)):
        with pytest.raises(binding.SgpError) as ei:
            binding.Schedule(4, g)
        assert ei.value.code == binding.SGP_ERR_ARG
    sched = binding.Schedule(4, binding.GraphDesc.exp_peers(1))
    lib = binding.lib()
    nnz = C.c_int64()
    small = np.zeros(2, dtype=np.int32)
    rowptr = np.zeros(5, dtype=np.int32)
    assert lib.sgp_schedule_get(sched._ptr, 0, rowptr.ctypes.data, small.ctypes.data, small.ctypes.data, 2,
                                C.byref(nnz)) == binding.SGP_ERR_ARG
    assert nnz.value == 8
    assert lib.sgp_schedule_get(sched._ptr, -1, rowptr.ctypes.data, small.ctypes.data, small.ctypes.data, 2,
                                C.byref(nnz)) == binding.SGP_ERR_ARG
    assert lib.sgp_schedule_period(None, C.byref(nnz)) == binding.SGP_ERR_ARG
    assert binding.strerror(binding.SGP_ERR_GRAPH).startswith("schedule")


def test_library_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "sgp.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(sgp_[a-z_0-9]+)\s*\(", header))
    assert declared == set(binding.EXPORTS), declared ^ set(binding.EXPORTS)
    lib = binding.lib()
    for name in declared:
        assert hasattr(lib, name), name
    assert binding.version() >= 100


def test_handle_calls_reject_null_without_a_gpu(binding):
    lib = binding.lib()
    assert lib.sgp_step(None, None, None, None, None, None, 0, 0.1, 0.0, 0.0, 1, None) == binding.SGP_ERR_ARG
    assert lib.sgp_debias(None, None, None, None, None) == binding.SGP_ERR_ARG
    assert lib.sgp_destroy(None) == binding.SGP_OK
    out = C.c_void_p()
    g = binding.GraphDesc.exp_peers(1)
    assert lib.sgp_create(C.byref(out), 0, 10, 10, C.byref(g.c), 0, 0) == binding.SGP_ERR_ARG
    assert lib.sgp_create(C.byref(out), 4, 10, 8, C.byref(g.c), 0, 0) == binding.SGP_ERR_ARG      # ld < d
    assert lib.sgp_create(C.byref(out), 4, 10, 10, C.byref(g.c), -1, 0) == binding.SGP_ERR_ARG    # tau < 0
    assert out.value is None


def test_new_entry_points_reject_null_without_a_gpu(binding):
    lib = binding.lib()
    stats = (C.c_double * 8)()
    assert lib.sgp_check(None, None, None, None, stats, None) == binding.SGP_ERR_ARG
    assert lib.sgp_colsum(None, None, 0, None, None) == binding.SGP_ERR_ARG
    assert lib.sgp_get_diagnostics(None, None, None, None, None) == binding.SGP_ERR_ARG
    assert lib.sgp_step_adam_host(None, None, None, None, None, None, None, None, None, 0, 1, 0.1, 0.9, 0.99, 1e-8, 0.0, 0,
                                  None) == binding.SGP_ERR_ARG
    assert lib.sgp_rank_update(None, None, None, None, None, 0, 0.1, 0.0, 0.0, 1, None) == binding.SGP_ERR_ARG
    assert lib.sgp_rank_mix(None, None, None, None, 0, None) == binding.SGP_ERR_ARG
    assert lib.sgp_rank_step_overlap(None, None, None, None, None, None, 0, 0.1, 0.0, 0.0, 1, None) == binding.SGP_ERR_ARG
    assert lib.sgp_rank_destroy(None) == binding.SGP_OK
    assert lib.sgp_ipc_export(None, None) == binding.SGP_ERR_ARG and lib.sgp_ipc_close(None) == binding.SGP_OK
    out = C.c_void_p()
    g = binding.GraphDesc.exp_peers(1)
    assert lib.sgp_rank_create(C.byref(out), 4, 4, 100, C.byref(g.c), 0, 0) == binding.SGP_ERR_ARG       # rank == world
    assert lib.sgp_rank_create(C.byref(out), 0, 4, 100, C.byref(g.c), 0, 8) == binding.SGP_ERR_ARG       # unknown flag
    assert out.value is None
    for code, word in ((binding.SGP_ERR_ZERO_WEIGHT, "weight"), (binding.SGP_ERR_INVARIANT, "invariant"),
                       (binding.SGP_ERR_DEVICE, "wait")):
        assert word in binding.strerror(code)


def test_rank_plan_host_only(binding):
    """sgp_rank_plan needs no GPU: slots, self weight and the in-neighbour list in the order of the sum."""
    sched = binding.Schedule(8, binding.GraphDesc.exp_peers(2))
    for k in range(7):
        P = S.mixing_matrix("exp", 8, k, peers=2)
        for r in range(8):
            plan = binding.rank_plan(sched, r, k, 0)
            want = [j for j in range(8) if P[r, j] != 0.0]
            assert plan["senders"] == want and plan["self_pos"] == want.index(r)
            assert plan["write_slot"] == plan["read_slot"] == k % 2
            assert np.array_equal(plan["weights"], np.array([P[r, j] for j in want], dtype=np.float32))
            late = binding.rank_plan(sched, r, k, 3)
            Pd = S.mixing_matrix("exp", 8, k - 3, peers=2) if k >= 3 else np.zeros((8, 8))
            assert late["senders"] == [j for j in range(8) if Pd[r, j] != 0.0 and j != r]
            assert late["write_slot"] == k % 5 and late["read_slot"] == (k - 3) % 5 and late["self_pos"] == -1
            assert late["self_weight"] == np.float32(P[r, r])
    for bad in ((8, 0, 0), (-1, 0, 0), (0, -1, 0), (0, 0, -1), (0, 0, 65)):
        with pytest.raises(binding.SgpError) as e:
            binding.rank_plan(sched, *bad)
        assert e.value.code == binding.SGP_ERR_ARG


@pytest.mark.parametrize("n,kind,tau,period", [(8, "exp1", 0, 2), (8, "exp1", 1, 2), (8, "exp2", 2, 2), (6, "random", 1, 3),
                                               (6, "random", 0, 3), (16, "exp1", 3, 4), (5, "random", 2, 1)])
def test_rank_plans_with_a_send_period_reproduce_the_oracle_recursion(binding, n, kind, tau, period):
    """sgp_rank_plan_period (host only): all ranks emulated in one process -- each publishes its half step into slot
    write_slot, then mixes what its plan says -- end on the oracle's state for the same send period (Alg. 2 line 5:
    transmissions only on steps k with k mod s = 0; identity mixing in between; messages arrive tau steps later)."""
    from oracle import schedule as osched
    from oracle import sgp as osgp
    graph = {"exp1": binding.GraphDesc.exp_peers(1), "exp2": binding.GraphDesc.exp_peers(2),
             "random": binding.GraphDesc.random_outdeg(11, 4, 3)}[kind]
    okind = dict(exp1=("exp", dict(peers=1)), exp2=("exp", dict(peers=2)),
                 random=("random", dict(seed=11, max_outdeg=3, num_steps=4)))[kind]
    P_of_k = lambda k: osched.mixing_matrix(okind[0], n, k, **okind[1])
    K, d, lr = 11, 5, 0.1
    rng = np.random.default_rng(5)
    x = rng.standard_normal((n, d))
    grads = rng.standard_normal((K, n, d))
    w = np.ones(n)
    slots = tau + 2
    slot_x = np.zeros((n, slots, d))
    slot_w = np.zeros((n, slots))
    sched = binding.Schedule(n, graph)
    for k in range(K):
        plans = [binding.rank_plan(sched, r, k, tau, send_period=period) for r in range(n)]
        h = x - lr * grads[k]
        for r in range(n):                                   # every rank publishes (the barrier comes after this loop)
            slot_x[r, plans[r]["write_slot"]] = h[r]
            slot_w[r, plans[r]["write_slot"]] = w[r]
        new_x, new_w = np.zeros_like(x), np.zeros_like(w)
        for r, plan in enumerate(plans):
            if tau > 0:
                new_x[r] = float(plan["self_weight"]) * h[r]
                new_w[r] = float(plan["self_weight"]) * w[r]
                assert plan["self_pos"] == -1
                if k % period:
                    assert plan["self_weight"] == np.float32(1.0)
            for e, j in enumerate(plan["senders"]):
                new_x[r] += float(plan["weights"][e]) * slot_x[j, plan["read_slot"]]
                new_w[r] += float(plan["weights"][e]) * slot_w[j, plan["read_slot"]]
            if tau == 0 and k % period:
                assert plan["senders"] == [r] and plan["self_pos"] == 0 and plan["weights"][0] == np.float32(1.0)
            if tau > 0 and (k < tau or (k - tau) % period):
                assert plan["senders"] == []                 # nothing was sent tau steps ago
        x, w = new_x, new_w
    rng = np.random.default_rng(5)
    x0 = rng.standard_normal((n, d))
    st = osgp.sgp_run(x0, K, P_of_k, lambda k, z: grads[k], lr, tau=tau, send_period=period)
    assert np.allclose(x, st.x, rtol=1e-6, atol=1e-7) and np.allclose(w, st.w, rtol=1e-6, atol=1e-7)   # fp32 plan weights


def _random_custom_schedule(n, steps, seed):
    """Random column-stochastic schedule with NON-uniform fp32 weights (every column sums to 1 in fp32 exactly
    enough for the compiler's check): per sender a random out-set incl. self and Dirichlet-like weights."""
    rng = np.random.default_rng(seed)
    step, send, recv, wt = [], [], [], []
    for k in range(steps):
        for j in range(n):
            deg = int(rng.integers(0, min(5, n)))
            targets = [j] + [int(t) for t in rng.choice([t for t in range(n) if t != j], size=deg, replace=False)]
            raw = rng.random(len(targets)) + 0.1
            w = (raw / raw.sum()).astype(np.float32)
            w[0] = np.float32(1.0 - float(w[1:].astype(np.float64).sum()))        # make the fp32 column sum ~1
            for t, p in zip(targets, w):
                step.append(k); send.append(j); recv.append(t); wt.append(float(p))
    perm = rng.permutation(len(step))                                             # any edge order is accepted
    return [np.asarray(a)[perm] for a in (step, send, recv, wt)]


@pytest.mark.parametrize("n,steps,seed", [(2, 1, 0), (7, 3, 1), (33, 4, 2), (256, 2, 3)])
def test_custom_random_weighted_schedules_bit_exact(binding, n, steps, seed):
    step, send, recv, wt = _random_custom_schedule(n, steps, seed)
    sched = binding.Schedule(n, binding.GraphDesc.custom(steps, step, send, recv, wt))
    assert sched.period == steps
    for k in range(steps):
        sel = step == k
        P = S.custom_mixing_matrix(n, send[sel], recv[sel], wt[sel].astype(np.float32))
        assert np.allclose(P.sum(axis=0), 1.0, atol=1e-6)
        _assert_slot_equal(sched, k, P)


def test_header_is_valid_c_and_library_links_from_c(binding, tmp_path):
    """A C99 program built with gcc against include/sgp.h and libsgp.so reproduces the oracle's schedule."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("gcc not available")
    exe = tmp_path / "c_abi_smoke"
    lib_dir = os.path.dirname(binding.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                    os.path.join(ROOT, "tests", "c_abi_smoke.c"), "-o", str(exe), "-L", lib_dir, "-l:libsgp.so",
                    f"-Wl,-rpath,{lib_dir}"], check=True, capture_output=True, text=True)
    n = 8
    out = subprocess.run([str(exe), str(n)], check=True, capture_output=True, text=True).stdout.splitlines()
    assert out[0].split() == ["version", str(binding.version()), "n", str(n), "period", "3"]
    got = {}
    for line in out[1:]:
        k, i, j, p = line.split()
        got[(int(k), int(i), int(j))] = float(p)
    want = {}
    for k in range(3):
        P = S.mixing_matrix("exp", n, k, peers=1)
        for i in range(n):
            for j in range(n):
                if P[i, j] != 0.0:
                    want[(k, i, j)] = P[i, j]
    assert got == want
