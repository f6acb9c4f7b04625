"""Seeded synthetic inputs and workload definitions (no arithmetic of the SGP method in here).

A counter-based generator addressed by (seed, stream, step, node, column): any column range of any
step can be regenerated independently, on the CPU or on the GPU, with torch integer ops.  The
hash is the splitmix64 finaliser; normals come from one Box-Muller transform per element.  The
oracle never regenerates values: tests hand it the very fp32 bits the GPU path consumed.

`WORKLOADS` describes the synthetic stand-ins for the paper's workloads (ResNet-50-sized and
Transformer-sized parameter vectors across n nodes; the datasets themselves are not needed for
the per-step arithmetic).  N(0, v) is read as variance v.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

_M64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Python int (mod 2^64) -> the same bits as a signed 64-bit value."""
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)
_GOLD = 0x9E3779B97F4A7C15


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64_t(x: torch.Tensor) -> torch.Tensor:
    x = x ^ _lsr(x, 30)
    x = x * _C1
    x = x ^ _lsr(x, 27)
    x = x * _C2
    x = x ^ _lsr(x, 31)
    return x


def _mix64_i(x: int) -> int:
    x &= _M64
    x ^= x >> 30
    x = (x * 0xBF58476D1CE4E5B9) & _M64
    x ^= x >> 27
    x = (x * 0x94D049BB133111EB) & _M64
    x ^= x >> 31
    return x


STREAM_X0, STREAM_GRAD, STREAM_TARGET, STREAM_NOISE = 1, 2, 3, 4
_CHUNK = 1 << 24


def fill_normal(out: torch.Tensor, *, seed: int, stream: int, step: int, std: float, col_offset: int = 0,
                row_offset: int = 0) -> torch.Tensor:
    """out[i, c] = std * N(0,1) keyed by (seed, stream, step, row_offset + i, col_offset + c).  fp32, in place."""
    assert out.dtype == torch.float32 and out.dim() == 2
    n, d = out.shape
    key = _mix64_i(_mix64_i((seed + _GOLD) & _M64) ^ ((stream & 0xFFFF) << 48 | (step & 0xFFFFFFFFFFFF)))
    dev = out.device
    two_pi = 2.0 * math.pi
    for i in range(n):
        row_key = _s64(_mix64_i(key ^ ((row_offset + i) * _GOLD & _M64)))
        for c0 in range(0, d, _CHUNK):
            c1 = min(d, c0 + _CHUNK)
            ctr = torch.arange(col_offset + c0, col_offset + c1, dtype=torch.int64, device=dev)
            h = _mix64_t(ctr + row_key)
            u1 = (_lsr(h, 40).to(torch.float32) + 0.5) * (1.0 / (1 << 24))
            u2 = ((h >> 8) & 0xFFFFFF).to(torch.float32) * (1.0 / (1 << 24))
            r = torch.sqrt(-2.0 * torch.log(u1))
            out[i, c0:c1] = (std * r) * torch.cos(two_pi * u2)
    return out


def normal(n: int, d: int, *, seed: int, stream: int, step: int, std: float, device="cpu", ld: int | None = None,
           col_offset: int = 0) -> torch.Tensor:
    """New n x d fp32 tensor (row pitch ld >= d) of seeded normals."""
    ld = d if ld is None else ld
    buf = torch.empty((n, ld), dtype=torch.float32, device=device)
    view = buf[:, :d]
    fill_normal(view, seed=seed, stream=stream, step=step, std=std, col_offset=col_offset)
    return view


@dataclass(frozen=True)
class Workload:
    name: str
    n: int
    d: int
    K: int
    graph: str            # "exp" | "complete" | "random"
    peers: int = 1
    max_outdeg: int = 4
    num_steps: int = 0    # random graph: distinct steps
    lr: float = 0.1
    momentum: float = 0.0
    nesterov: bool = True
    weight_decay: float = 0.0
    tau: int = 0
    x0_std: float = 0.1
    x0_shared: bool = False   # identical initial row on every node
    grad_std: float = 0.1
    seed: int = 181110792
    optimizer: str = "sgd"          # "sgd" (plain / momentum / Nesterov by `momentum`, `nesterov`) or "adam"
    beta1: float = 0.9
    beta2: float = 0.98
    adam_eps: float = 1e-8

    def scaled(self, d: int, K: int | None = None) -> "Workload":
        """Same recipe on a shorter parameter vector (parity tests, CPU baseline samples)."""
        return Workload(**{**self.__dict__, "d": d, "K": self.K if K is None else K,
                           "name": f"{self.name}[d={d}]"})


WORKLOADS = {
    # n=8 toy run; its closed-loop quadratic gradients are produced by the harness, not here
    "tiny": Workload("tiny", n=8, d=4096, K=100, graph="exp", peers=1, lr=0.1, momentum=0.9, x0_std=0.0,
                     grad_std=0.1, seed=181110793),
    # ResNet-50-sized parameter vector on 32 nodes (the paper's ImageNet runs: Nesterov 0.9, wd 1e-4)
    "resnet50": Workload("resnet50", n=32, d=25_557_032, K=20, graph="exp", peers=1, lr=0.1, momentum=0.9,
                         weight_decay=1e-4, x0_std=0.1, x0_shared=True, grad_std=0.1, seed=181110794),
    # Transformer-sized parameter vector on 16 nodes, two-peer graph, plain SGD
    "transformer": Workload("transformer", n=16, d=61_000_000, K=20, graph="exp", peers=2, lr=1e-3,
                            momentum=0.0, x0_std=math.sqrt(0.02), grad_std=math.sqrt(1e-3), seed=181110795),
    # 1-overlap SGP on the ResNet-50-sized vector
    "resnet50_osgp1": Workload("resnet50_osgp1", n=32, d=25_557_032, K=20, graph="exp", peers=1, lr=0.1,
                               momentum=0.9, tau=1, x0_std=0.1, x0_shared=True, grad_std=0.1, seed=181110796),
}

# Adam-SGP on the Transformer-sized vector (the paper's translation runs combine SGP with Adam)
WORKLOADS["transformer_adam"] = Workload("transformer_adam", n=16, d=61_000_000, K=20, graph="exp", peers=2, lr=1e-3,
                                         x0_std=math.sqrt(0.02), grad_std=math.sqrt(1e-3), seed=181110798,
                                         optimizer="adam")

SWEEP_N = (4, 16, 64, 256)
SWEEP_D = (10_000, 1_000_000, 10_000_000, 100_000_000)


def sweep_workload(n: int, d: int) -> Workload:
    """Scaling-sweep point: random digraphs, out-degree U{1..min(4, n-1)} plus self-loop, 10 distinct steps."""
    return Workload(f"sweep_n{n}_d{d}", n=n, d=d, K=10, graph="random", max_outdeg=4, num_steps=10, lr=0.1,
                    momentum=0.9, x0_std=0.1, grad_std=0.1, seed=181110797)


def initial_x(w: Workload, device="cpu", ld: int | None = None, col_offset: int = 0, d: int | None = None):
    d = w.d if d is None else d
    if w.x0_std == 0.0:
        ldv = d if ld is None else ld
        return torch.zeros((w.n, ldv), dtype=torch.float32, device=device)[:, :d]
    if w.x0_shared:
        row = normal(1, d, seed=w.seed, stream=STREAM_X0, step=0, std=w.x0_std, device=device, col_offset=col_offset)
        ldv = d if ld is None else ld
        buf = torch.empty((w.n, ldv), dtype=torch.float32, device=device)
        buf[:, :d] = row
        return buf[:, :d]
    return normal(w.n, d, seed=w.seed, stream=STREAM_X0, step=0, std=w.x0_std, device=device, ld=ld,
                  col_offset=col_offset)


def gradient(w: Workload, k: int, out: torch.Tensor, col_offset: int = 0) -> torch.Tensor:
    """Fills out (n x d' view) with the step-k gradients of columns [col_offset, col_offset + d')."""
    return fill_normal(out, seed=w.seed, stream=STREAM_GRAD, step=k, std=w.grad_std, col_offset=col_offset)
