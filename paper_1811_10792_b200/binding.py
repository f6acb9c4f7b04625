"""ctypes binding of libsgp.so: argument marshalling only, same names as include/sgp.h.

Every step of the SGP iteration runs inside the CUDA library; nothing here computes.  The library
is loaded from this package's directory and the import fails loudly if it is missing: there is no
CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
# SGP_CHECKED=1 in the environment selects the bounds-checked build of the same library (build.build_checked()).
LIB_PATH = os.path.join(_PKG_DIR, "libsgp_checked.so" if os.environ.get("SGP_CHECKED", "0") not in ("", "0") else "libsgp.so")
LIB_PATH = os.environ.get("SGP_LIBRARY", LIB_PATH)          # an explicit path wins (another build of the same sources)

SGP_OK, SGP_ERR_ARG, SGP_ERR_GRAPH, SGP_ERR_CUDA, SGP_ERR_ALLOC, SGP_ERR_STATE, SGP_ERR_DEVICE = 0, -1, -2, -3, -4, -5, -6
SGP_ERR_ZERO_WEIGHT, SGP_ERR_INVARIANT = -7, -8
SGP_STATUS_WAIT_TILE, SGP_STATUS_WAIT_STAGE, SGP_STATUS_WAIT_DRAIN, SGP_STATUS_ZERO_WEIGHT = 1, 2, 4, 8
SGP_STATUS_NONFINITE, SGP_STATUS_WEIGHT_SUM, SGP_STATUS_COLUMN_SUM, SGP_STATUS_BOUNDS = 16, 32, 64, 128
SGP_FLAG_NONE, SGP_FLAG_BIASED = 0, 1
SGP_MAX_NODES = 256
SGP_STATIC_MAX_NNZ = 4096
SGP_GRAPH_EXP_PEERS, SGP_GRAPH_COMPLETE, SGP_GRAPH_RANDOM_OUTDEG, SGP_GRAPH_CUSTOM, SGP_GRAPH_BIPARTITE_EXP = 0, 1, 2, 3, 4

# every symbol include/sgp.h declares
EXPORTS = [
    "sgp_schedule_compile", "sgp_schedule_destroy", "sgp_schedule_period", "sgp_schedule_nnz", "sgp_schedule_get",
    "sgp_create", "sgp_destroy", "sgp_get_schedule", "sgp_step", "sgp_debias", "sgp_step_host", "sgp_reset",
    "sgp_ring_export", "sgp_ring_import", "sgp_check", "sgp_set_option", "sgp_get_option", "sgp_device_status",
    "sgp_last_cuda_error", "sgp_strerror", "sgp_version", "sgp_step_static",
    "sgp_step_adam", "sgp_param_deviation", "sgp_set_graph", "sgp_colsum", "sgp_get_diagnostics",
    "sgp_rank_plan", "sgp_rank_create", "sgp_rank_destroy", "sgp_rank_get_schedule", "sgp_rank_message_block",
    "sgp_rank_set_peers", "sgp_rank_update", "sgp_rank_mix", "sgp_rank_step_overlap", "sgp_rank_device_status",
    "sgp_ipc_export", "sgp_ipc_open", "sgp_ipc_close", "sgp_step_adam_host", "sgp_rank_update_adam",
    "sgp_rank_step_overlap_adam", "sgp_rank_plan_period", "sgp_rank_set_send_period",
]
SGP_RANK_MAX_SOURCES = 32
SGP_IPC_HANDLE_BYTES = 64


class SgpError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


class sgp_graph_desc(C.Structure):
    _fields_ = [
        ("kind", C.c_int32), ("peers", C.c_int32), ("max_outdeg", C.c_int32), ("reserved", C.c_int32),
        ("seed", C.c_uint64), ("num_steps", C.c_int64),
        ("edge_step", C.POINTER(C.c_int32)), ("edge_sender", C.POINTER(C.c_int32)),
        ("edge_receiver", C.POINTER(C.c_int32)), ("edge_weight", C.POINTER(C.c_float)),
        ("num_edges", C.c_int64),
    ]


class sgp_rank_plan_t(C.Structure):
    _fields_ = [("write_slot", C.c_int32), ("read_slot", C.c_int32), ("self_weight", C.c_float),
                ("self_pos", C.c_int32), ("count", C.c_int32), ("sender", C.c_int32 * 32), ("weight", C.c_float * 32)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_1811_10792_b200.build` "
            "(there is no fallback implementation)")
    lib = C.CDLL(LIB_PATH)
    vp, i64, f32, i32 = C.c_void_p, C.c_int64, C.c_float, C.c_int
    sig = {
        "sgp_schedule_compile": [C.POINTER(vp), i32, C.POINTER(sgp_graph_desc)],
        "sgp_schedule_destroy": [vp],
        "sgp_schedule_period": [vp, C.POINTER(i64)],
        "sgp_schedule_nnz": [vp, i64, C.POINTER(i64)],
        "sgp_schedule_get": [vp, i64, vp, vp, vp, i64, C.POINTER(i64)],
        "sgp_create": [C.POINTER(vp), i32, i64, i64, C.POINTER(sgp_graph_desc), i32, C.c_uint],
        "sgp_destroy": [vp],
        "sgp_get_schedule": [vp, C.POINTER(vp)],
        "sgp_set_graph": [vp, C.POINTER(sgp_graph_desc)],
        "sgp_step": [vp, vp, vp, vp, vp, vp, i64, f32, f32, f32, i32, vp],
        "sgp_debias": [vp, vp, vp, vp, vp],
        "sgp_step_adam": [vp, vp, vp, vp, vp, vp, vp, i64, i64, f32, f32, f32, f32, f32, vp],
        "sgp_step_host": [vp, vp, vp, vp, vp, vp, vp, vp, i64, f32, f32, f32, i32, i64, vp],
        "sgp_step_adam_host": [vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, f32, f32, f32, f32, f32, i64, vp],
        "sgp_reset": [vp, vp],
        "sgp_ring_export": [vp, vp, vp, vp],
        "sgp_ring_import": [vp, vp, vp, vp],
        "sgp_check": [vp, vp, vp, vp, C.POINTER(C.c_double), vp],
        "sgp_colsum": [vp, vp, i32, vp, vp],
        "sgp_get_diagnostics": [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double), vp],
        "sgp_param_deviation": [vp, vp, C.POINTER(C.c_double), vp],
        "sgp_set_option": [vp, C.c_char_p, i64],
        "sgp_get_option": [vp, C.c_char_p, C.POINTER(i64)],
        "sgp_device_status": [vp, C.POINTER(C.c_uint)],
        "sgp_last_cuda_error": [vp],
        "sgp_version": [],
        "sgp_rank_plan": [vp, i32, i64, i32, C.POINTER(sgp_rank_plan_t)],
        "sgp_rank_plan_period": [vp, i32, i64, i32, i64, C.POINTER(sgp_rank_plan_t)],
        "sgp_rank_set_send_period": [vp, i64],
        "sgp_rank_create": [C.POINTER(vp), i32, i32, i64, C.POINTER(sgp_graph_desc), i32, C.c_uint],
        "sgp_rank_destroy": [vp],
        "sgp_rank_get_schedule": [vp, C.POINTER(vp)],
        "sgp_rank_message_block": [vp, C.POINTER(vp), C.POINTER(C.c_size_t)],
        "sgp_rank_set_peers": [vp, C.POINTER(vp)],
        "sgp_rank_update": [vp, vp, vp, vp, vp, i64, f32, f32, f32, i32, vp],
        "sgp_rank_mix": [vp, vp, vp, vp, i64, vp],
        "sgp_rank_step_overlap": [vp, vp, vp, vp, vp, vp, i64, f32, f32, f32, i32, vp],
        "sgp_rank_update_adam": [vp, vp, vp, vp, vp, vp, i64, i64, f32, f32, f32, f32, f32, vp],
        "sgp_rank_step_overlap_adam": [vp, vp, vp, vp, vp, vp, vp, i64, i64, f32, f32, f32, f32, f32, vp],
        "sgp_rank_device_status": [vp, C.POINTER(C.c_uint)],
        "sgp_ipc_export": [vp, C.c_char_p],
        "sgp_ipc_open": [C.c_char_p, C.POINTER(vp)],
        "sgp_ipc_close": [vp],
        "sgp_step_static": [i32, i64, i64, vp, vp, vp, i64, vp, vp, vp, vp, vp, f32, f32, f32, i32, vp],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.sgp_strerror.argtypes = [C.c_int]
    lib.sgp_strerror.restype = C.c_char_p
    return lib


_lib = _load()


def lib() -> C.CDLL:
    return _lib


def strerror(code: int) -> str:
    return _lib.sgp_strerror(code).decode()


def _check(code: int, what: str) -> None:
    if code != SGP_OK:
        raise SgpError(code, what)


class GraphDesc:
    """Owns the host arrays behind a sgp_graph_desc."""

    def __init__(self, kind: int, peers: int = 1, max_outdeg: int = 4, seed: int = 0, num_steps: int = 0,
                 edges=None):
        self.c = sgp_graph_desc()
        self.c.kind, self.c.peers, self.c.max_outdeg = kind, peers, max_outdeg
        self.c.reserved, self.c.seed, self.c.num_steps = 0, seed, num_steps
        self._keep = []
        if edges is not None:
            step, sender, receiver, weight = edges
            arrs = [np.ascontiguousarray(step, dtype=np.int32), np.ascontiguousarray(sender, dtype=np.int32),
                    np.ascontiguousarray(receiver, dtype=np.int32), np.ascontiguousarray(weight, dtype=np.float32)]
            self._keep = arrs
            self.c.edge_step = arrs[0].ctypes.data_as(C.POINTER(C.c_int32))
            self.c.edge_sender = arrs[1].ctypes.data_as(C.POINTER(C.c_int32))
            self.c.edge_receiver = arrs[2].ctypes.data_as(C.POINTER(C.c_int32))
            self.c.edge_weight = arrs[3].ctypes.data_as(C.POINTER(C.c_float))
            self.c.num_edges = len(arrs[0])

    @staticmethod
    def exp_peers(peers: int = 1) -> "GraphDesc":
        return GraphDesc(SGP_GRAPH_EXP_PEERS, peers=peers)

    @staticmethod
    def complete() -> "GraphDesc":
        return GraphDesc(SGP_GRAPH_COMPLETE)

    @staticmethod
    def bipartite_exp() -> "GraphDesc":
        return GraphDesc(SGP_GRAPH_BIPARTITE_EXP)

    @staticmethod
    def random_outdeg(seed: int, num_steps: int, max_outdeg: int = 4) -> "GraphDesc":
        return GraphDesc(SGP_GRAPH_RANDOM_OUTDEG, max_outdeg=max_outdeg, seed=seed, num_steps=num_steps)

    @staticmethod
    def custom(num_steps: int, step, sender, receiver, weight) -> "GraphDesc":
        return GraphDesc(SGP_GRAPH_CUSTOM, num_steps=num_steps, edges=(step, sender, receiver, weight))


class _ScheduleView:
    """Read access to a compiled schedule (host arrays)."""

    def __init__(self, ptr, n):
        self._ptr, self.n = ptr, n

    @property
    def period(self) -> int:
        v = C.c_int64()
        _check(_lib.sgp_schedule_period(self._ptr, C.byref(v)), "sgp_schedule_period")
        return v.value

    def nnz(self, k: int) -> int:
        v = C.c_int64()
        _check(_lib.sgp_schedule_nnz(self._ptr, k, C.byref(v)), "sgp_schedule_nnz")
        return v.value

    def get(self, k: int):
        """(rowptr int32[n+1], col int32[nnz], val float32[nnz]) of step k."""
        nnz = self.nnz(k)
        rowptr = np.empty(self.n + 1, dtype=np.int32)
        col = np.empty(max(nnz, 1), dtype=np.int32)
        val = np.empty(max(nnz, 1), dtype=np.float32)
        out = C.c_int64()
        _check(_lib.sgp_schedule_get(self._ptr, k, rowptr.ctypes.data, col.ctypes.data, val.ctypes.data, nnz,
                                     C.byref(out)), "sgp_schedule_get")
        return rowptr, col[:nnz], val[:nnz]


def rank_plan(schedule: "_ScheduleView", rank: int, k: int, tau: int, send_period: int = 1) -> dict:
    """sgp_rank_plan / sgp_rank_plan_period (host only): what `rank` publishes and pulls at step k in the
    one-node-per-GPU mode."""
    out = sgp_rank_plan_t()
    if send_period == 1:
        _check(_lib.sgp_rank_plan(schedule._ptr, rank, k, tau, C.byref(out)), "sgp_rank_plan")
    else:
        _check(_lib.sgp_rank_plan_period(schedule._ptr, rank, k, tau, send_period, C.byref(out)), "sgp_rank_plan_period")
    return dict(write_slot=out.write_slot, read_slot=out.read_slot, self_weight=np.float32(out.self_weight),
                self_pos=out.self_pos, senders=[out.sender[e] for e in range(out.count)],
                weights=np.array([out.weight[e] for e in range(out.count)], dtype=np.float32))


class Schedule(_ScheduleView):
    """sgp_schedule_compile: host-only graph-schedule compiler (needs no GPU)."""

    def __init__(self, n: int, graph: GraphDesc):
        ptr = C.c_void_p()
        _check(_lib.sgp_schedule_compile(C.byref(ptr), n, C.byref(graph.c)), "sgp_schedule_compile")
        super().__init__(ptr, n)

    def close(self):
        if getattr(self, "_ptr", None) and _lib is not None:
            _lib.sgp_schedule_destroy(self._ptr)
            self._ptr = None

    def __del__(self):
        self.close()


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


_torch = None


def _get_torch():
    global _torch
    if _torch is None:
        import torch
        _torch = torch
    return _torch


def _stream_ptr(stream):
    if stream is not None:
        return C.c_void_p(stream.cuda_stream)
    torch = _get_torch()
    raw = getattr(torch._C, "_cuda_getCurrentRawStream", None)      # the current stream's handle without a Stream object
    if raw is not None:
        return C.c_void_p(raw(torch.cuda.current_device()))
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Sgp:
    """sgp_create / sgp_step / sgp_debias ... on torch CUDA tensors (fp32, row pitch ld)."""

    def __init__(self, n: int, d: int, graph: GraphDesc, tau: int = 0, ld: int | None = None, flags: int = 0):
        self.n, self.d, self.ld, self.tau = n, d, (d if ld is None else ld), tau
        self._h = C.c_void_p()
        _check(_lib.sgp_create(C.byref(self._h), n, d, self.ld, C.byref(graph.c), tau, flags), "sgp_create")

    def close(self):
        if getattr(self, "_h", None) and _lib is not None:      # _lib is None during interpreter shutdown
            _lib.sgp_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def set_graph(self, graph: GraphDesc) -> None:
        """Switches the mixing schedule (hybrid schemes: dense mixing early, sparse later)."""
        _check(_lib.sgp_set_graph(self._h, C.byref(graph.c)), "sgp_set_graph")

    @property
    def schedule(self) -> _ScheduleView:
        p = C.c_void_p()
        _check(_lib.sgp_get_schedule(self._h, C.byref(p)), "sgp_get_schedule")
        return _ScheduleView(p, self.n)

    def _check_mat(self, t, name, allow_none=False):
        if t is None:
            if allow_none:
                return
            raise ValueError(f"{name} is required")
        if t.dtype != _get_torch().float32 or not t.is_cuda:
            raise ValueError(f"{name} must be a float32 CUDA tensor")
        shape, stride = t.shape, t.stride()
        if len(shape) != 2 or shape[0] != self.n or shape[1] != self.d or stride[1] != 1 or \
                (self.n > 1 and stride[0] != self.ld):
            raise ValueError(f"{name} must be n x d with row pitch ld={self.ld}")

    def step(self, X, W, M, G, Z, k: int, lr: float, momentum: float = 0.0, weight_decay: float = 0.0,
             nesterov: bool = True, stream=None) -> None:
        self._check_mat(X, "X")
        self._check_mat(G, "G")
        self._check_mat(M, "M", allow_none=(momentum == 0.0))
        self._check_mat(Z, "Z", allow_none=True)
        _check(_lib.sgp_step(self._h, _ptr(X), _ptr(W), _ptr(M), _ptr(G), _ptr(Z), k, lr, momentum, weight_decay,
                             int(bool(nesterov)), _stream_ptr(stream)), "sgp_step")

    def step_adam(self, X, W, M1, M2, G, Z, k: int, t: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
                  eps: float = 1e-8, weight_decay: float = 0.0, stream=None) -> None:
        for name, m in (("X", X), ("M1", M1), ("M2", M2), ("G", G)):
            self._check_mat(m, name)
        self._check_mat(Z, "Z", allow_none=True)
        _check(_lib.sgp_step_adam(self._h, _ptr(X), _ptr(W), _ptr(M1), _ptr(M2), _ptr(G), _ptr(Z), k, t, lr, beta1,
                                  beta2, eps, weight_decay, _stream_ptr(stream)), "sgp_step_adam")

    def debias(self, X, W, Z, stream=None) -> None:
        self._check_mat(X, "X")
        self._check_mat(Z, "Z")
        _check(_lib.sgp_debias(self._h, _ptr(X), _ptr(W), _ptr(Z), _stream_ptr(stream)), "sgp_debias")

    def step_host(self, X, W, M, h_G, h_Z, d_G, d_Z, k: int, lr: float, momentum: float = 0.0,
                  weight_decay: float = 0.0, nesterov: bool = True, chunk_cols: int = 0, stream=None) -> None:
        """h_G / h_Z are host (ideally pinned) tensors; everything else lives on the device."""
        _check(_lib.sgp_step_host(self._h, _ptr(X), _ptr(W), _ptr(M), _ptr(h_G), _ptr(h_Z), _ptr(d_G), _ptr(d_Z),
                                  k, lr, momentum, weight_decay, int(bool(nesterov)), chunk_cols,
                                  _stream_ptr(stream)), "sgp_step_host")

    def step_adam_host(self, X, W, M1, M2, h_G, h_Z, d_G, d_Z, k: int, t: int, lr: float, beta1: float = 0.9,
                       beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.0, chunk_cols: int = 0,
                       stream=None) -> None:
        _check(_lib.sgp_step_adam_host(self._h, _ptr(X), _ptr(W), _ptr(M1), _ptr(M2), _ptr(h_G), _ptr(h_Z), _ptr(d_G),
                                       _ptr(d_Z), k, t, lr, beta1, beta2, eps, weight_decay, chunk_cols,
                                       _stream_ptr(stream)), "sgp_step_adam_host")

    def reset(self, stream=None) -> None:
        _check(_lib.sgp_reset(self._h, _stream_ptr(stream)), "sgp_reset")

    def ring_export(self, ring_x, ring_w, stream=None) -> None:
        _check(_lib.sgp_ring_export(self._h, _ptr(ring_x), _ptr(ring_w), _stream_ptr(stream)), "sgp_ring_export")

    def ring_import(self, ring_x, ring_w, stream=None) -> None:
        _check(_lib.sgp_ring_import(self._h, _ptr(ring_x), _ptr(ring_w), _stream_ptr(stream)), "sgp_ring_import")

    STAT_NAMES = ("sum_w", "min_w", "nonfinite", "total", "max_colsum_drift", "max_colsum_rel_drift", "sum_w_drift",
                  "status")

    def check(self, X, W, colsum_ref=None, stream=None, raise_on_error: bool = True):
        """sgp_check: dict of the eight statistics plus "code" (the call's return code).

        colsum_ref: float64 CUDA tensor of d expected column sums of X plus ring, or None."""
        import torch
        if colsum_ref is not None and (colsum_ref.dtype != torch.float64 or not colsum_ref.is_cuda or
                                       colsum_ref.numel() != self.d or not colsum_ref.is_contiguous()):
            raise ValueError("colsum_ref must be a contiguous float64 CUDA tensor of d entries")
        out = (C.c_double * 8)()
        code = _lib.sgp_check(self._h, _ptr(X), _ptr(W), _ptr(colsum_ref), out, _stream_ptr(stream))
        if raise_on_error:
            _check(code, "sgp_check")
        res = dict(zip(self.STAT_NAMES, out))
        res["code"] = code
        return res

    def colsum(self, A, include_ring: bool = False, out=None, stream=None):
        """sgp_colsum: float64 CUDA tensor of the d column sums of A (plus the ring's when include_ring)."""
        import torch
        self._check_mat(A, "A")
        if out is None:
            out = torch.empty(self.d, dtype=torch.float64, device=A.device)
        _check(_lib.sgp_colsum(self._h, _ptr(A), int(bool(include_ring)), _ptr(out), _stream_ptr(stream)), "sgp_colsum")
        return out

    def diagnostics(self, stream=None):
        """sgp_get_diagnostics: (param_dev float64[n], consensus float64[n], summary dict of mean/min/max each)."""
        a = (C.c_double * self.n)()
        b = (C.c_double * self.n)()
        s = (C.c_double * 6)()
        _check(_lib.sgp_get_diagnostics(self._h, a, b, s, _stream_ptr(stream)), "sgp_get_diagnostics")
        names = ("param_dev_mean", "param_dev_min", "param_dev_max", "consensus_mean", "consensus_min", "consensus_max")
        return np.array(a[:], dtype=np.float64), np.array(b[:], dtype=np.float64), dict(zip(names, s))

    def param_deviation(self, A, stream=None):
        """Per-node distance from the node-wise average row, ||A_i - mean_j A_j||_2 (numpy float64[n])."""
        self._check_mat(A, "A")
        out = (C.c_double * self.n)()
        _check(_lib.sgp_param_deviation(self._h, _ptr(A), out, _stream_ptr(stream)), "sgp_param_deviation")
        return np.array(out[:], dtype=np.float64)

    def set_option(self, key: str, value: int) -> None:
        _check(_lib.sgp_set_option(self._h, key.encode(), value), "sgp_set_option")

    def get_option(self, key: str) -> int:
        v = C.c_int64()
        _check(_lib.sgp_get_option(self._h, key.encode(), C.byref(v)), "sgp_get_option")
        return v.value

    def device_status(self) -> int:
        v = C.c_uint()
        _check(_lib.sgp_device_status(self._h, C.byref(v)), "sgp_device_status")
        return v.value

    def last_cuda_error(self) -> int:
        return _lib.sgp_last_cuda_error(self._h)


class SgpRank:
    """sgp_rank_*: one node of the one-node-per-GPU mode.  x, m, g, z are 1-D float32 CUDA tensors of d entries,
    w is a float32 CUDA tensor of one entry.  Marshalling only; see rowshard.py for the orchestration."""

    def __init__(self, rank: int, world: int, d: int, graph: GraphDesc, tau: int = 0, flags: int = 0):
        self.rank, self.world, self.d, self.tau = rank, world, d, tau
        self._h = C.c_void_p()
        _check(_lib.sgp_rank_create(C.byref(self._h), rank, world, d, C.byref(graph.c), tau, flags), "sgp_rank_create")

    def close(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.sgp_rank_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    @property
    def schedule(self) -> _ScheduleView:
        p = C.c_void_p()
        _check(_lib.sgp_rank_get_schedule(self._h, C.byref(p)), "sgp_rank_get_schedule")
        return _ScheduleView(p, self.world)

    def message_block(self):
        """(device pointer, bytes) of this rank's message slots."""
        ptr, size = C.c_void_p(), C.c_size_t()
        _check(_lib.sgp_rank_message_block(self._h, C.byref(ptr), C.byref(size)), "sgp_rank_message_block")
        return ptr.value, size.value

    def set_send_period(self, send_period: int) -> None:
        """Nodes transmit only on steps k with k mod send_period == 0 (Alg. 2 line 5); every rank must set the same."""
        _check(_lib.sgp_rank_set_send_period(self._h, send_period), "sgp_rank_set_send_period")

    def set_peers(self, pointers) -> None:
        """pointers[j]: device address (int or None) of rank j's message block in this process."""
        arr = (C.c_void_p * self.world)(*[C.c_void_p(p) if p else None for p in pointers])
        _check(_lib.sgp_rank_set_peers(self._h, arr), "sgp_rank_set_peers")

    def update(self, x, w, m, g, k: int, lr: float, momentum: float = 0.0, weight_decay: float = 0.0,
               nesterov: bool = True, stream=None) -> None:
        _check(_lib.sgp_rank_update(self._h, _ptr(x), _ptr(w), _ptr(m), _ptr(g), k, lr, momentum, weight_decay,
                                    int(bool(nesterov)), _stream_ptr(stream)), "sgp_rank_update")

    def mix(self, x, w, z, k: int, stream=None) -> None:
        _check(_lib.sgp_rank_mix(self._h, _ptr(x), _ptr(w), _ptr(z), k, _stream_ptr(stream)), "sgp_rank_mix")

    def step_overlap(self, x, w, m, g, z, k: int, lr: float, momentum: float = 0.0, weight_decay: float = 0.0,
                     nesterov: bool = True, stream=None) -> None:
        _check(_lib.sgp_rank_step_overlap(self._h, _ptr(x), _ptr(w), _ptr(m), _ptr(g), _ptr(z), k, lr, momentum,
                                          weight_decay, int(bool(nesterov)), _stream_ptr(stream)),
               "sgp_rank_step_overlap")

    def update_adam(self, x, w, m1, m2, g, k: int, t: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
                    eps: float = 1e-8, weight_decay: float = 0.0, stream=None) -> None:
        _check(_lib.sgp_rank_update_adam(self._h, _ptr(x), _ptr(w), _ptr(m1), _ptr(m2), _ptr(g), k, t, lr, beta1, beta2,
                                         eps, weight_decay, _stream_ptr(stream)), "sgp_rank_update_adam")

    def step_overlap_adam(self, x, w, m1, m2, g, z, k: int, t: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
                          eps: float = 1e-8, weight_decay: float = 0.0, stream=None) -> None:
        _check(_lib.sgp_rank_step_overlap_adam(self._h, _ptr(x), _ptr(w), _ptr(m1), _ptr(m2), _ptr(g), _ptr(z), k, t, lr,
                                               beta1, beta2, eps, weight_decay, _stream_ptr(stream)),
               "sgp_rank_step_overlap_adam")

    def device_status(self) -> int:
        v = C.c_uint()
        _check(_lib.sgp_rank_device_status(self._h, C.byref(v)), "sgp_rank_device_status")
        return v.value


def ipc_export(device_ptr: int) -> bytes:
    buf = C.create_string_buffer(SGP_IPC_HANDLE_BYTES)
    _check(_lib.sgp_ipc_export(C.c_void_p(device_ptr), buf), "sgp_ipc_export")
    return buf.raw


def ipc_open(handle: bytes) -> int:
    ptr = C.c_void_p()
    _check(_lib.sgp_ipc_open(handle, C.byref(ptr)), "sgp_ipc_open")
    return ptr.value


def ipc_close(device_ptr: int) -> None:
    _check(_lib.sgp_ipc_close(C.c_void_p(device_ptr)), "sgp_ipc_close")


def step_static(n: int, d: int, ld: int, rowptr, col, val, X, W, M, G, Z, lr: float, momentum: float = 0.0,
                weight_decay: float = 0.0, nesterov: bool = True, stream=None) -> None:
    """sgp_step_static: the tau = 0 fused step without a handle and without any device allocation.

    For callers that cannot call cudaMalloc (all device memory owned by a pool, latency-critical loops).
    rowptr / col / val are HOST numpy arrays in the form Schedule.get(k) returns (at most
    SGP_STATIC_MAX_NNZ entries).  Calls must be ordered on one stream: they share one static device table.
    """
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    col = np.ascontiguousarray(col, dtype=np.int32)
    val = np.ascontiguousarray(val, dtype=np.float32)
    _check(_lib.sgp_step_static(n, d, ld, rowptr.ctypes.data, col.ctypes.data, val.ctypes.data, len(col), _ptr(X),
                                _ptr(W), _ptr(M), _ptr(G), _ptr(Z), lr, momentum, weight_decay, int(bool(nesterov)),
                                _stream_ptr(stream)), "sgp_step_static")


def graph_desc(w) -> GraphDesc:
    """Schedule descriptor of a workload from `inputs` (marshalling of its graph fields, nothing else)."""
    if w.graph == "exp":
        return GraphDesc.exp_peers(w.peers)
    if w.graph == "complete":
        return GraphDesc.complete()
    if w.graph == "bipartite":
        return GraphDesc.bipartite_exp()
    if w.graph == "random":
        return GraphDesc.random_outdeg(w.seed, w.num_steps, w.max_outdeg)
    raise ValueError(w.graph)


def empty_matrix(n: int, d: int, device="cuda", pitch_multiple: int = 256, fill=None):
    """n x d float32 view whose rows start `ld` floats apart, ld = d rounded up to `pitch_multiple`.

    Rows on 1 KB boundaries (pitch_multiple = 256) let the step kernels reach ~0.98 of the copy bandwidth
    instead of ~0.91 with a dense pitch whose rows start off the 128-byte grid.  Returns (view, ld); pass ld to Sgp(...).
    """
    import torch
    ld = (d + pitch_multiple - 1) // pitch_multiple * pitch_multiple
    buf = torch.empty((n, ld), dtype=torch.float32, device=device) if fill is None else \
        torch.full((n, ld), float(fill), dtype=torch.float32, device=device)
    return buf[:, :d], ld


def version() -> int:
    return _lib.sgp_version()
