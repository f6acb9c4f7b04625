"""One node per GPU: orchestration of the split SGP step (plumbing only -- every arithmetic step is a kernel of
libsgp.so, reached through binding.SgpRank).

Two ways to run it:

* ``LoopbackGroup``: all ``world`` ranks live in ONE process on ONE device, each with its own message slots
  (separate allocations) and its own rows; "peer pointers" are then just the other ranks' local addresses and
  stream order stands in for the barrier.  This is how the kernels and the pointer tables are tested on a
  single GPU, and how the split step is timed without NVLink.
* ``DistributedRank``: one process per GPU under ``torch.distributed``.  Every rank exports its message slots as a
  CUDA IPC handle, the handles travel through ``all_gather_object``, each rank maps its peers' slots, and the
  mix kernel reads them with plain loads over NVLink.  The per-step barrier is a one-element all-reduce on the
  step's stream (NCCL), or a host barrier for process groups without device collectives (gloo).

Step protocol (Alg. 1 lines 4-8; Alg. 2 for tau >= 1):
    tau == 0 :  update  ->  BARRIER  ->  mix
    tau >= 1 :  step_overlap  ->  BARRIER        (one kernel; the barrier is off the kernel's critical path:
                                                  what step k reads was published at step k - tau)
"""
from __future__ import annotations

from . import binding


def step_protocol(tau: int):
    """The calls of one step, in order; 'barrier' marks where every rank must have finished the call before."""
    return ("update", "barrier", "mix") if tau == 0 else ("step_overlap", "barrier")


class LoopbackGroup:
    """``world`` virtual ranks on the current device of this process."""

    def __init__(self, world: int, d: int, graph: binding.GraphDesc, tau: int = 0, flags: int = 0, send_period: int = 1):
        self.world, self.d, self.tau = world, d, tau
        self.ranks = [binding.SgpRank(r, world, d, graph, tau=tau, flags=flags) for r in range(world)]
        if send_period != 1:
            for rk in self.ranks:
                rk.set_send_period(send_period)
        blocks = [rk.message_block()[0] for rk in self.ranks]
        for rk in self.ranks:
            rk.set_peers(blocks)

    def close(self):
        for rk in self.ranks:
            rk.close()
        self.ranks = []

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def step(self, xs, ws, ms, gs, zs, k: int, lr: float, momentum: float = 0.0, weight_decay: float = 0.0,
             nesterov: bool = True, stream=None) -> None:
        """xs[r], ms[r], gs[r], zs[r]: rank r's rows; ws[r]: its one-element weight tensor.  All launches go to one
        stream, so every update of step k completes before the first mix of step k starts."""
        m_of = (lambda r: ms[r]) if momentum != 0.0 else (lambda r: None)
        z_of = (lambda r: zs[r]) if zs is not None else (lambda r: None)
        if self.tau == 0:
            for r, rk in enumerate(self.ranks):
                rk.update(xs[r], ws[r], m_of(r), gs[r], k, lr, momentum, weight_decay, nesterov, stream=stream)
            for r, rk in enumerate(self.ranks):
                rk.mix(xs[r], ws[r], z_of(r), k, stream=stream)
        else:
            for r, rk in enumerate(self.ranks):
                rk.step_overlap(xs[r], ws[r], m_of(r), gs[r], z_of(r), k, lr, momentum, weight_decay, nesterov,
                                stream=stream)

    def step_adam(self, xs, ws, m1s, m2s, gs, zs, k: int, t: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
                  eps: float = 1e-8, weight_decay: float = 0.0, stream=None) -> None:
        """The same protocol with the Adam preconditioner (m1s[r], m2s[r]: rank r's moment rows)."""
        z_of = (lambda r: zs[r]) if zs is not None else (lambda r: None)
        if self.tau == 0:
            for r, rk in enumerate(self.ranks):
                rk.update_adam(xs[r], ws[r], m1s[r], m2s[r], gs[r], k, t, lr, beta1, beta2, eps, weight_decay, stream=stream)
            for r, rk in enumerate(self.ranks):
                rk.mix(xs[r], ws[r], z_of(r), k, stream=stream)
        else:
            for r, rk in enumerate(self.ranks):
                rk.step_overlap_adam(xs[r], ws[r], m1s[r], m2s[r], gs[r], z_of(r), k, t, lr, beta1, beta2, eps,
                                     weight_decay, stream=stream)

    def device_status(self) -> int:
        status = 0
        for rk in self.ranks:
            status |= rk.device_status()
        return status


def exchange_handles(rank: int, world: int, my_handle: bytes, group=None):
    """Every rank's IPC handle, by rank (all_gather_object over the process group)."""
    import torch.distributed as dist
    gathered = [None] * world
    dist.all_gather_object(gathered, (rank, bytes(my_handle)), group=group)
    by_rank = dict(gathered)
    assert sorted(by_rank) == list(range(world)), "every rank must contribute exactly one handle"
    return [by_rank[r] for r in range(world)]


class DistributedRank:
    """This process's node under torch.distributed (one process per GPU, all GPUs in one NVLink domain)."""

    def __init__(self, d: int, graph: binding.GraphDesc, tau: int = 0, flags: int = 0, group=None, device=None,
                 send_period: int = 1):
        import torch
        import torch.distributed as dist
        self.group = group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.tau = tau
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
        self.node = binding.SgpRank(self.rank, self.world, d, graph, tau=tau, flags=flags)
        if send_period != 1:
            self.node.set_send_period(send_period)
        ptr, _ = self.node.message_block()
        handles = exchange_handles(self.rank, self.world, binding.ipc_export(ptr), group=group)
        self._mapped = []
        peers = [None] * self.world
        for r, handle in enumerate(handles):
            if r != self.rank:
                peers[r] = binding.ipc_open(handle)
                self._mapped.append(peers[r])
        self.node.set_peers(peers)
        self._device_collectives = dist.get_backend(group) == "nccl"
        self._token = torch.zeros(1, device=self.device)

    def close(self):
        for p in self._mapped:
            binding.ipc_close(p)
        self._mapped = []
        self.node.close()

    def barrier(self) -> None:
        """Every rank's work enqueued so far is complete before any rank's work enqueued afterwards starts."""
        import torch
        import torch.distributed as dist
        if self._device_collectives:
            dist.all_reduce(self._token, group=self.group)      # on the current stream: a device-side rendezvous
        else:
            torch.cuda.current_stream().synchronize()
            dist.barrier(group=self.group)

    def step(self, x, w, m, g, z, k: int, lr: float, momentum: float = 0.0, weight_decay: float = 0.0,
             nesterov: bool = True) -> None:
        for call in step_protocol(self.tau):
            if call == "update":
                self.node.update(x, w, m if momentum != 0.0 else None, g, k, lr, momentum, weight_decay, nesterov)
            elif call == "mix":
                self.node.mix(x, w, z, k)
            elif call == "step_overlap":
                self.node.step_overlap(x, w, m if momentum != 0.0 else None, g, z, k, lr, momentum, weight_decay, nesterov)
            else:
                self.barrier()

    def step_adam(self, x, w, m1, m2, g, z, k: int, t: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
                  eps: float = 1e-8, weight_decay: float = 0.0) -> None:
        for call in step_protocol(self.tau):
            if call == "update":
                self.node.update_adam(x, w, m1, m2, g, k, t, lr, beta1, beta2, eps, weight_decay)
            elif call == "mix":
                self.node.mix(x, w, z, k)
            elif call == "step_overlap":
                self.node.step_overlap_adam(x, w, m1, m2, g, z, k, t, lr, beta1, beta2, eps, weight_decay)
            else:
                self.barrier()
