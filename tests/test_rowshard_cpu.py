"""One node per GPU, host side, on CPU with gloo ranks (world size 2 and 4): who publishes into which slot, who pulls
from whom with which weight at step k, and that the step protocol's barrier placement never lets a slot be
rewritten before its readers are done.  The plan comes from the library (sgp_rank_plan, host only); the expected
values come from the oracle's dense mixing matrices.  The rows themselves travel over gloo send/recv here and are
mixed with numpy by the TEST, so that the pull pattern is validated end to end against the oracle recursion."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from conftest import ROOT


def _worker(rank, world, port, kind, tau, K, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from oracle import schedule as osched
    from paper_1811_10792_b200 import binding, rowshard
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        graph = {"exp1": binding.GraphDesc.exp_peers(1), "exp2": binding.GraphDesc.exp_peers(2),
                 "bipartite": binding.GraphDesc.bipartite_exp(),
                 "random": binding.GraphDesc.random_outdeg(7, 5, 3)}[kind]
        okind = dict(exp1=("exp", dict(peers=1)), exp2=("exp", dict(peers=2)), bipartite=("bipartite", {}),
                     random=("random", dict(seed=7, max_outdeg=3, num_steps=5)))[kind]
        P_of_k = lambda k: osched.mixing_matrix(okind[0], world, k, **okind[1])
        sched = binding.Schedule(world, graph)
        slots = tau + 2
        d = 6
        rng = np.random.default_rng(100 + rank)
        h_row = rng.standard_normal(d)                       # this rank's row; zero gradients: h = x
        w_val = 1.0
        slot_x = [np.zeros(d) for _ in range(slots)]
        slot_w = [0.0] * slots
        slot_tag = [-1] * slots                              # which step's message a slot holds
        # handles travel exactly as DistributedRank sends them (fake 64-byte handles: no GPU here)
        handles = rowshard.exchange_handles(rank, world, bytes([rank]) * binding.SGP_IPC_HANDLE_BYTES)
        assert [hd[0] for hd in handles] == list(range(world))
        ok = True
        for k in range(K):
            plan = binding.rank_plan(sched, rank, k, tau)
            # ---- the plan against the oracle's matrices, bit for bit
            if tau == 0:
                row = P_of_k(k)[rank]
                want_s = [j for j in range(world) if row[j] != 0.0]
                want_w = np.array([row[j] for j in want_s], dtype=np.float32)
                ok &= plan["senders"] == want_s and plan["self_pos"] == want_s.index(rank)
                ok &= plan["read_slot"] == plan["write_slot"] == k % slots
            else:
                row = P_of_k(k - tau)[rank] if k >= tau else np.zeros(world)
                want_s = [j for j in range(world) if row[j] != 0.0 and j != rank]
                want_w = np.array([row[j] for j in want_s], dtype=np.float32)
                ok &= plan["senders"] == want_s and plan["self_pos"] == -1
                ok &= plan["write_slot"] == k % slots and plan["read_slot"] == (k - tau) % slots
            ok &= np.array_equal(plan["weights"].view(np.int32), want_w.view(np.int32))
            ok &= plan["self_weight"] == np.float32(P_of_k(k)[rank, rank])
            # ---- who pulls from me is what the others' plans say (the union of the pulls is P's off-diagonal)
            all_plans = [None] * world
            dist.all_gather_object(all_plans, (rank, plan["senders"], plan["read_slot"]))
            readers = [r for r, senders, _ in all_plans if rank in senders and r != rank]
            Pk = P_of_k(k if tau == 0 else k - tau) if (tau == 0 or k >= tau) else np.zeros((world, world))
            ok &= sorted(readers) == [i for i in range(world) if i != rank and Pk[i, rank] != 0.0]
            # ---- the step protocol: publish, barrier, pull
            for call in rowshard.step_protocol(tau):
                if call in ("update", "step_overlap"):
                    ok &= slot_tag[plan["write_slot"]] in (-1, k - slots)    # rewritten only tau + 2 steps later
                    slot_x[plan["write_slot"]] = h_row.copy()
                    slot_w[plan["write_slot"]] = w_val
                    slot_tag[plan["write_slot"]] = k
                if call == "barrier":
                    dist.barrier()
                if call in ("mix", "step_overlap"):
                    # serve my slot `read_slot` to my readers, fetch my in-neighbours' (a pull, done with send/recv)
                    reqs = []
                    for r in readers:
                        payload = torch.tensor(np.concatenate([slot_x[plan["read_slot"]], [slot_w[plan["read_slot"]],
                                                                                         float(slot_tag[plan["read_slot"]])]]))
                        reqs.append(dist.isend(payload, dst=r))
                    acc_x = np.zeros(d)
                    acc_w = 0.0
                    for e, j in enumerate(plan["senders"]):
                        if j == rank:
                            got = np.concatenate([slot_x[plan["read_slot"]], [slot_w[plan["read_slot"]],
                                                                              float(slot_tag[plan["read_slot"]])]])
                        else:
                            buf = torch.zeros(d + 2, dtype=torch.float64)
                            dist.recv(buf, src=j)
                            got = buf.numpy()
                        ok &= int(got[-1]) == (k if tau == 0 else k - tau)     # the slot holds the message of the right step
                        acc_x = acc_x + float(plan["weights"][e]) * got[:d]
                        acc_w = acc_w + float(plan["weights"][e]) * got[d]
                    for q in reqs:
                        q.wait()
                    if tau > 0:
                        acc_x = float(plan["self_weight"]) * h_row + acc_x
                        acc_w = float(plan["self_weight"]) * w_val + acc_w
                    h_row, w_val = acc_x, acc_w
        gathered = [None] * world
        dist.all_gather_object(gathered, (rank, h_row, w_val))
        out[rank] = (bool(ok), {r: (x, w) for r, x, w in gathered})
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,kind,tau", [(2, "exp1", 0), (2, "exp1", 1), (4, "exp1", 0), (4, "exp2", 0), (4, "exp1", 1),
                                            (4, "random", 0), (4, "random", 2), (4, "bipartite", 0)])
def test_exchange_schedule_over_gloo(world, kind, tau):
    from oracle import schedule as osched
    from oracle import sgp as osgp
    K = 7
    port = 29800 + world * 10 + tau + {"exp1": 0, "exp2": 3, "random": 5, "bipartite": 8}[kind] * 20
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, kind, tau, K, out), nprocs=world, join=True)
        res = dict(out)
    assert all(res[r][0] for r in range(world)), "a plan, a reader set or a slot tag was wrong"
    # the rows every rank ended with equal the oracle's recursion on the stacked state
    x0 = np.stack([np.random.default_rng(100 + r).standard_normal(6) for r in range(world)])
    okind = dict(exp1=("exp", dict(peers=1)), exp2=("exp", dict(peers=2)), bipartite=("bipartite", {}),
                 random=("random", dict(seed=7, max_outdeg=3, num_steps=5)))[kind]
    st = osgp.sgp_run(x0, K, lambda k: osched.mixing_matrix(okind[0], world, k, **okind[1]),
                      lambda k, z: np.zeros_like(z), 0.1, tau=tau)
    final = res[0][1]
    for r in range(world):
        assert np.allclose(final[r][0], st.x[r], rtol=1e-6, atol=1e-7)       # plan weights are fp32-rounded
        assert abs(final[r][1] - st.w[r]) <= 1e-6


def test_step_protocol_shape():
    sys.path.insert(0, ROOT)
    from paper_1811_10792_b200 import rowshard
    assert rowshard.step_protocol(0) == ("update", "barrier", "mix")
    assert rowshard.step_protocol(1) == ("step_overlap", "barrier")
    assert rowshard.step_protocol(3) == ("step_overlap", "barrier")
