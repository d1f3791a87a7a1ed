"""ctypes binding of libhfx.so (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libhfx.so")
_lib = None

COMMIT = 1
QUEUED, RUNNING, DONE, REJECTED = 0, 1, 2, 3
COLOCATED, PREFILL, DECODE = 0, 1, 2
BUDGET_SAFE, BUDGET_CAP_ONLY = 0, 1
ST_BAD_REPLICA, ST_BAD_CLASS, ST_BAD_LEN, ST_TIMEOUT = 1, 2, 4, 8
E_ARG, E_ALIGN, E_CAPACITY, E_CUDA, E_TIMEOUT, E_NOMEM = -1, -2, -3, -4, -5, -6

EXPORTED_SYMBOLS = ["hfx_sched_create", "hfx_sched_step", "hfx_sim_run", "hfx_sched_status",
                    "hfx_sched_launch_count", "hfx_sched_destroy", "hfx_strerror", "hfx_sched_set_profiling",
                    "hfx_sched_get_profile", "hfx_sched_set_fused_front", "hfx_kernel_name", "hfx_count_rows_noalloc", "hfx_scale_tick", "hfx_dispatch_step", "hfx_slo_map", "hfx_pd_migrate", "hfx_attainment",
                    "hfx_sched_set_horizon", "hfx_scale_apply", "hfx_dispatch_bind", "hfx_scale_decide"]
NOALLOC_MAX_REPLICAS = 4096
N_KERNELS = 14


class HfxError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {load_library().hfx_strerror(code).decode()} ({code})")


class _Model(C.Structure):
    _fields_ = [(k, C.c_int64) for k in ("c0", "c1", "c2", "d0", "d1", "d2")]


class _SloClass(C.Structure):
    _fields_ = [("ttft_slo_ns", C.c_int64), ("tpot_slo_ns", C.c_int64), ("prio", C.c_int32), ("reserved", C.c_int32)]


class _ReplicaCfg(C.Structure):
    _fields_ = [("mode", C.c_int32), ("token_cap", C.c_int32), ("batch_cap", C.c_int32)]


class _Options(C.Structure):
    _fields_ = [("budget_mode", C.c_int32), ("weight_max", C.c_int32), ("flags", C.c_uint32), ("reserved", C.c_uint32)]


TABLE_COLUMNS = ["replica_id", "class_id", "state", "prompt_len", "output_len", "gen", "arrival_ns",
                 "first_token_ns", "last_token_ns", "finish_ns", "req_id", "weight"]
TABLE_DTYPES = {"replica_id": torch.int32, "class_id": torch.uint8, "state": torch.uint8, "prompt_len": torch.int32,
                "output_len": torch.int32, "gen": torch.int32, "arrival_ns": torch.int64,
                "first_token_ns": torch.int64, "last_token_ns": torch.int64, "finish_ns": torch.int64,
                "req_id": torch.int32, "weight": torch.int32}


class _Table(C.Structure):
    _fields_ = [("n_rows", C.c_int64)] + [(k, C.c_void_p) for k in TABLE_COLUMNS]


class _ReplicaState(C.Structure):
    _fields_ = [("now_ns", C.c_void_p), ("maturity_ns", C.c_void_p)]


STEP_OUT_FIELDS = [("slack_ns", torch.int64, "n"), ("pred_ttft_ns", torch.int64, "n"), ("pred_tpot_ns", torch.int64, "n"),
                   ("key", torch.int64, "n"), ("order", torch.int32, "n"), ("seg_off", torch.int32, "R1"),
                   ("admit", torch.uint8, "n"), ("admitted_rows", torch.int32, "n"), ("budget", torch.int64, "R"),
                   ("e_d_ns", torch.int64, "R"), ("n_run", torch.int32, "R"), ("sum_kv", torch.int64, "R"),
                   ("adm_cost", torch.int64, "R"), ("adm_count", torch.int32, "R"), ("maturity_next", torch.int64, "R")]
STEP_OUT_OPTIONAL = {"pred_ttft_ns", "pred_tpot_ns", "key", "admitted_rows", "e_d_ns", "n_run", "sum_kv"}


class _StepOut(C.Structure):
    _fields_ = [(k, C.c_void_p) for k, _, _ in STEP_OUT_FIELDS]


SIM_OUT_FIELDS = [("iters_executed", torch.int32), ("finished", torch.int32), ("rejected", torch.int32),
                  ("attained", torch.int32), ("ttft_p50_ns", torch.int64), ("ttft_p99_ns", torch.int64),
                  ("tpot_p50_ns", torch.int64), ("tpot_p99_ns", torch.int64), ("now_ns", torch.int64)]


class _Profile(C.Structure):
    _fields_ = [("ms", C.c_double * 14), ("launches", C.c_int64 * 14)]


class _ScaleParams(C.Structure):
    _fields_ = [("window_ns", C.c_int64), ("block_tokens", C.c_int32), ("min_samples", C.c_int32),
                ("eps_out_num", C.c_int32), ("eps_out_den", C.c_int32), ("eps_in_num", C.c_int32),
                ("eps_in_den", C.c_int32), ("eps_wait_num", C.c_int32), ("eps_wait_den", C.c_int32)]


class _ScaleOut(C.Structure):
    _fields_ = [("counts", C.c_void_p), ("used_blocks", C.c_void_p), ("decision", C.c_void_p)]


class _SimOut(C.Structure):
    _fields_ = [(k, C.c_void_p) for k, _ in SIM_OUT_FIELDS]


DISPATCH_OUT_FIELDS = [("assign", torch.int32, "n"), ("queue_order", torch.int32, "n"), ("n_queue", torch.int32, "2"),
                       ("inst_order", torch.int32, "R"), ("n_mature", torch.int32, "2"), ("slack_ns", torch.int64, "n"),
                       ("budget", torch.int64, "R"), ("e_d_ns", torch.int64, "R"), ("n_run", torch.int32, "R"),
                       ("sum_kv", torch.int64, "R"), ("adm_cost", torch.int64, "R"), ("adm_count", torch.int32, "R"),
                       ("maturity_next", torch.int64, "R")]


SLO_BOUND_FIELDS = ("ttft_min_ns", "ttft_max_ns", "ttft_min_relaxed_ns", "tpot_min_ns", "tpot_max_ns", "tpot_min_relaxed_ns")


class _SloWindow(C.Structure):
    _fields_ = [("prio", C.c_void_p), ("ttft_ns", C.c_void_p), ("tpot_ns", C.c_void_p), ("queue_ns", C.c_void_p),
                ("w", C.c_int32), ("reserved", C.c_int32)]


class _SloBounds(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in SLO_BOUND_FIELDS]


class _DispatchOut(C.Structure):
    _fields_ = [(k, C.c_void_p) for k, _, _ in DISPATCH_OUT_FIELDS]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libhfx.so.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2508_15919_b200.build` "
                          "(nvcc, sm_100a); there is no CPU fallback")
    L = C.CDLL(_LIB_PATH)
    L.hfx_sched_create.restype = C.c_int
    L.hfx_sched_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(_Model), C.POINTER(_SloClass), C.c_int,
                                   C.POINTER(_ReplicaCfg), C.c_int, C.c_int64, C.POINTER(_Options), C.c_void_p]
    L.hfx_sched_step.restype = C.c_int
    L.hfx_sched_step.argtypes = [C.c_void_p, C.POINTER(_Table), C.POINTER(_ReplicaState), C.POINTER(_StepOut), C.c_uint32]
    L.hfx_dispatch_step.restype = C.c_int
    L.hfx_dispatch_step.argtypes = [C.c_void_p, C.POINTER(_Table), C.c_int64, C.c_void_p, C.POINTER(_DispatchOut)]
    L.hfx_pd_migrate.restype = C.c_int
    L.hfx_pd_migrate.argtypes = [C.c_void_p, C.POINTER(_Table), C.c_void_p, C.POINTER(_ReplicaState), C.c_void_p, C.c_int64,
                                 C.c_int64, C.c_void_p]
    L.hfx_attainment.restype = C.c_int
    L.hfx_attainment.argtypes = [C.c_void_p, C.POINTER(_Table), C.c_void_p]
    L.hfx_slo_map.restype = C.c_int
    L.hfx_slo_map.argtypes = [C.c_void_p, C.c_int32, C.POINTER(_SloWindow), C.POINTER(_SloBounds), C.c_void_p, C.c_void_p,
                              C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
    L.hfx_sim_run.restype = C.c_int
    L.hfx_sim_run.argtypes = [C.c_void_p, C.POINTER(_Table), C.c_void_p, C.c_int32, C.c_int32, C.POINTER(_SimOut)]
    L.hfx_sched_status.restype = C.c_int
    L.hfx_sched_status.argtypes = [C.c_void_p, C.POINTER(C.c_uint32)]
    L.hfx_sched_launch_count.restype = C.c_int64
    L.hfx_sched_launch_count.argtypes = [C.c_void_p]
    L.hfx_sched_destroy.restype = None
    L.hfx_sched_destroy.argtypes = [C.c_void_p]
    L.hfx_sched_set_profiling.restype = C.c_int
    L.hfx_sched_set_profiling.argtypes = [C.c_void_p, C.c_int]
    L.hfx_sched_set_horizon.restype = C.c_int
    L.hfx_sched_set_horizon.argtypes = [C.c_void_p, C.c_int64]
    L.hfx_scale_decide.restype = C.c_int
    L.hfx_scale_decide.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(_ScaleParams), C.POINTER(_ScaleOut)]
    L.hfx_scale_apply.restype = C.c_int
    L.hfx_scale_apply.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.POINTER(C.c_int64), C.POINTER(_Fleet),
                                  C.POINTER(_ReplicaState), C.c_void_p]
    L.hfx_dispatch_bind.restype = C.c_int
    L.hfx_dispatch_bind.argtypes = [C.c_void_p, C.POINTER(_Table), C.c_void_p, C.c_int64, C.POINTER(_DispatchOut), C.c_void_p]
    L.hfx_sched_set_fused_front.restype = C.c_int
    L.hfx_sched_set_fused_front.argtypes = [C.c_void_p, C.c_int]
    L.hfx_sched_get_profile.restype = C.c_int
    L.hfx_sched_get_profile.argtypes = [C.c_void_p, C.POINTER(_Profile)]
    L.hfx_kernel_name.restype = C.c_char_p
    L.hfx_kernel_name.argtypes = [C.c_int]
    L.hfx_count_rows_noalloc.restype = C.c_int
    L.hfx_count_rows_noalloc.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    L.hfx_scale_tick.restype = C.c_int
    L.hfx_scale_tick.argtypes = [C.c_void_p, C.POINTER(_Table), C.c_int64, C.c_void_p, C.POINTER(_ScaleParams),
                                 C.POINTER(_ScaleOut)]
    L.hfx_strerror.restype = C.c_char_p
    L.hfx_strerror.argtypes = [C.c_int]
    _lib = L
    return L


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def count_rows_noalloc(replica_id: torch.Tensor, n_replicas: int, seg_off: torch.Tensor,
                       n_bad: Optional[torch.Tensor] = None) -> None:
    """hfx_count_rows_noalloc on the current stream: fills seg_off (int32, n_replicas + 1) with the
    start of every replica in a replica-major order, using no device allocation of its own (the
    caller passes every buffer; the counters are a fixed array inside the library).  For callers
    that may not allocate; at most NOALLOC_MAX_REPLICAS replicas."""
    L = load_library()
    assert replica_id.dtype == torch.int32 and seg_off.dtype == torch.int32 and seg_off.numel() >= n_replicas + 1
    rc = L.hfx_count_rows_noalloc(_ptr(replica_id) if replica_id.numel() else None, int(replica_id.numel()),
                                  int(n_replicas), _ptr(seg_off), _ptr(n_bad),
                                  C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if rc != 0:
        raise HfxError(rc, "hfx_count_rows_noalloc")


class DeviceTable:
    """The request table as torch tensors on the GPU (structure of arrays)."""

    def __init__(self, cols: Dict[str, torch.Tensor]):
        self.cols = cols
        self.n_rows = int(cols["class_id"].shape[0])
        for k, t in cols.items():
            if t is not None:
                assert t.is_cuda and t.is_contiguous() and t.dtype == TABLE_DTYPES[k], k

    @staticmethod
    def from_numpy(cols: Dict[str, np.ndarray], device="cuda") -> "DeviceTable":
        out = {}
        for k in TABLE_COLUMNS:
            a = cols.get(k)
            out[k] = None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(device)
        return DeviceTable(out)

    def to_numpy(self) -> Dict[str, np.ndarray]:
        return {k: v.cpu().numpy() for k, v in self.cols.items() if v is not None}

    def c_struct(self) -> _Table:
        s = _Table()
        s.n_rows = self.n_rows
        for k in TABLE_COLUMNS:
            setattr(s, k, _ptr(self.cols.get(k)))
        return s


class StepOut:
    """Output buffers of one step (allocated once, reused)."""

    def __init__(self, n_rows: int, n_replicas: int, device="cuda", optional: bool = True):
        self.t: Dict[str, Optional[torch.Tensor]] = {}
        for k, dt, dim in STEP_OUT_FIELDS:
            size = {"n": max(n_rows, 1), "R": n_replicas, "R1": n_replicas + 1}[dim]
            self.t[k] = None if (k in STEP_OUT_OPTIONAL and not optional) else torch.zeros(size, dtype=dt, device=device)
        self.n_rows = n_rows

    def c_struct(self) -> _StepOut:
        s = _StepOut()
        for k, _, _ in STEP_OUT_FIELDS:
            setattr(s, k, _ptr(self.t[k]))
        return s

    def to_numpy(self) -> Dict[str, np.ndarray]:
        out = {}
        for k, v in self.t.items():
            if v is None:
                continue
            a = v.cpu().numpy()
            if k == "key":
                a = a.view(np.uint64)
            if k in ("slack_ns", "pred_ttft_ns", "pred_tpot_ns", "key", "order", "admit", "admitted_rows"):
                a = a[:self.n_rows]
            out[k] = a
        return out


FLEET_FIELDS = [("inst_state", torch.int32), ("ready", torch.int64), ("billed", torch.int64), ("since", torch.int64),
                ("total_blocks", torch.int32), ("due", torch.int64), ("blocks_cap", torch.int32)]
INST_OFF, INST_STARTING, INST_ACTIVE, INST_DRAINING = 0, 1, 2, 3


class _Fleet(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("inst_state", "ready_ns", "billed_ns", "since_ns", "total_blocks", "due_ns", "blocks_cap")]


class Fleet:
    """Instance records of hfx_scale_apply on the device (fields as FLEET_FIELDS, one entry per instance)."""

    def __init__(self, arrays: Dict[str, np.ndarray], device="cuda"):
        self.t = {k: torch.from_numpy(np.ascontiguousarray(arrays[k])).to(dtype=dt, device=device) for k, dt in FLEET_FIELDS}

    def c_struct(self) -> _Fleet:
        return _Fleet(*[_ptr(self.t[k]) for k, _ in FLEET_FIELDS])

    def to_numpy(self) -> Dict[str, np.ndarray]:
        return {k: v.cpu().numpy() for k, v in self.t.items()}


class DispatchOut:
    """Output buffers of hfx_dispatch_step (allocated once, reused)."""

    def __init__(self, n_rows: int, n_replicas: int, device="cuda"):
        self.t = {k: torch.zeros({"n": max(n_rows, 1), "R": n_replicas, "2": 4}[dim], dtype=dt, device=device)
                  for k, dt, dim in DISPATCH_OUT_FIELDS}
        self.n_rows = n_rows

    def c_struct(self) -> _DispatchOut:
        s = _DispatchOut()
        for k, _, _ in DISPATCH_OUT_FIELDS:
            setattr(s, k, _ptr(self.t[k]))
        return s

    def to_numpy(self) -> Dict[str, np.ndarray]:
        out = {}
        for k, _, dim in DISPATCH_OUT_FIELDS:
            a = self.t[k].cpu().numpy()
            out[k] = a[:self.n_rows] if dim == "n" else (a[:2] if dim == "2" else a)
        return out


class SimOut:
    def __init__(self, n_traces: int, device="cuda"):
        self.t = {k: torch.zeros(max(n_traces, 1), dtype=dt, device=device) for k, dt in SIM_OUT_FIELDS}
        self.n_traces = n_traces

    def c_struct(self) -> _SimOut:
        s = _SimOut()
        for k, _ in SIM_OUT_FIELDS:
            setattr(s, k, _ptr(self.t[k]))
        return s

    def to_numpy(self) -> Dict[str, np.ndarray]:
        return {k: v.cpu().numpy()[:self.n_traces] for k, v in self.t.items()}


class Scheduler:
    """hfx_sched_create / hfx_sched_step / hfx_sim_run / hfx_sched_status on torch tensors."""

    def __init__(self, model: Sequence[int], classes: Sequence[Sequence[int]], replicas, max_rows: int,
                 budget_mode: int = BUDGET_SAFE, weight_max: int = 0, stream: Optional[torch.cuda.Stream] = None,
                 first_fit: bool = False):
        L = load_library()
        self._L = L
        self._h = C.c_void_p()
        m = _Model(*[int(x) for x in model])
        cls = (_SloClass * len(classes))(*[_SloClass(int(a), int(b), int(p), 0) for a, b, p in classes])
        reps_np = np.asarray(replicas, np.int32).reshape(-1, 3)
        reps = (_ReplicaCfg * reps_np.shape[0])(*[_ReplicaCfg(int(r[0]), int(r[1]), int(r[2])) for r in reps_np])
        opts = _Options(int(budget_mode), int(weight_max), 1 if first_fit else 0, 0)
        self.n_replicas = reps_np.shape[0]
        self.stream = stream
        if stream is not None:
            sp = C.c_void_p(stream.cuda_stream)
        elif torch.cuda.is_available():
            sp = C.c_void_p(torch.cuda.current_stream().cuda_stream)
        else:
            sp = C.c_void_p()      # no device: the library reports HFX_E_CUDA
        rc = L.hfx_sched_create(C.byref(self._h), C.byref(m), cls, len(classes), reps, self.n_replicas, int(max_rows),
                                C.byref(opts), sp)
        if rc != 0:
            self._h = C.c_void_p()
            raise HfxError(rc, "hfx_sched_create")

    def step(self, table: DeviceTable, now: torch.Tensor, maturity: torch.Tensor, out: StepOut, commit: bool = False):
        ts, os_ = table.c_struct(), out.c_struct()
        st = _ReplicaState(now.data_ptr(), maturity.data_ptr())
        rc = self._L.hfx_sched_step(self._h, C.byref(ts), C.byref(st), C.byref(os_), COMMIT if commit else 0)
        if rc != 0:
            raise HfxError(rc, "hfx_sched_step")

    def step_raw(self, ts: _Table, st: _ReplicaState, os_: _StepOut, flags: int) -> int:
        """The bare call on prebuilt structs (what a latency-sensitive caller keeps around)."""
        return self._L.hfx_sched_step(self._h, C.byref(ts), C.byref(st), C.byref(os_), flags)

    def sim_run(self, table: DeviceTable, trace_off: np.ndarray, iters: int, out: SimOut):
        off = np.ascontiguousarray(trace_off, np.int32)
        ts, os_ = table.c_struct(), out.c_struct()
        rc = self._L.hfx_sim_run(self._h, C.byref(ts), off.ctypes.data, int(off.shape[0] - 1), int(iters), C.byref(os_))
        if rc != 0:
            raise HfxError(rc, "hfx_sim_run")

    def dispatch_step(self, table: DeviceTable, now_ns: int, maturity: torch.Tensor, out: DispatchOut):
        """hfx_dispatch_step: the dispatching steps over the shared global queue at time now_ns."""
        ts, os_ = table.c_struct(), out.c_struct()
        rc = self._L.hfx_dispatch_step(self._h, C.byref(ts), int(now_ns), _ptr(maturity), C.byref(os_))
        if rc != 0:
            raise HfxError(rc, "hfx_dispatch_step")

    def dispatch_bind(self, table: DeviceTable, now_ns: int, out: DispatchOut, now: torch.Tensor):
        """hfx_dispatch_bind: bind what dispatch_step assigned (table.replica_id, the instance clocks `now`)."""
        ts, os_ = table.c_struct(), out.c_struct()
        rc = self._L.hfx_dispatch_bind(self._h, C.byref(ts), _ptr(table.cols["replica_id"]), int(now_ns), C.byref(os_), _ptr(now))
        if rc != 0:
            raise HfxError(rc, "hfx_dispatch_bind")

    def scale_apply(self, now_ns: int, decision: torch.Tensor, used_blocks: torch.Tensor, cold_start_ns, fleet: "Fleet",
                    now: torch.Tensor, maturity: torch.Tensor, cost: torch.Tensor):
        """hfx_scale_apply: carry out one tick's decisions on `fleet`; cost int64 [3] on the device."""
        cold = (C.c_int64 * 3)(*[int(x) for x in cold_start_ns])
        fs = fleet.c_struct()
        st = _ReplicaState(_ptr(now), _ptr(maturity))
        rc = self._L.hfx_scale_apply(self._h, int(now_ns), _ptr(decision), _ptr(used_blocks), cold, C.byref(fs), C.byref(st), _ptr(cost))
        if rc != 0:
            raise HfxError(rc, "hfx_scale_apply")

    def set_horizon(self, horizon_ns: Optional[int]):
        """hfx_sched_set_horizon (None: no horizon)."""
        rc = self._L.hfx_sched_set_horizon(self._h, int(np.iinfo(np.int64).max if horizon_ns is None else horizon_ns))
        if rc != 0:
            raise HfxError(rc, "hfx_sched_set_horizon")

    def pd_migrate(self, table: DeviceTable, now: torch.Tensor, maturity: torch.Tensor, pair: torch.Tensor,
                   xfer_c0_ns: int, xfer_c1_ns: int, n_moved: Optional[torch.Tensor] = None):
        """hfx_pd_migrate: hand prefilled requests over from the P instances to their partner D instances
        (pair: int32 [n_replicas] on the device); table.replica_id, table.state and now are updated in place."""
        ts = table.c_struct()
        st = _ReplicaState(_ptr(now), _ptr(maturity))
        rc = self._L.hfx_pd_migrate(self._h, C.byref(ts), _ptr(table.cols["replica_id"]), C.byref(st), _ptr(pair),
                                    int(xfer_c0_ns), int(xfer_c1_ns), _ptr(n_moved))
        if rc != 0:
            raise HfxError(rc, "hfx_pd_migrate")

    def attainment(self, table: DeviceTable, out: torch.Tensor):
        """hfx_attainment: out int64 [n_classes + 1, 6] on the device (requests, DONE, attained, REJECTED,
        sum of TTFT, sum of E2E per class; totals in the last row)."""
        ts = table.c_struct()
        rc = self._L.hfx_attainment(self._h, C.byref(ts), _ptr(out))
        if rc != 0:
            raise HfxError(rc, "hfx_attainment")

    def slo_map(self, n_prio: int, window: Dict[str, torch.Tensor], bounds: Dict[str, torch.Tensor],
                last_queue: torch.Tensor, pending: torch.Tensor, new_prio: torch.Tensor, ttft_out: torch.Tensor,
                tpot_out: torch.Tensor):
        """hfx_slo_map: window = {prio int32, ttft_ns, tpot_ns, queue_ns int64} device tensors of w records;
        bounds = the six per-priority int64 device tensors of SLO_BOUND_FIELDS; last_queue int64 [n_prio]
        (updated in place); pending int32 [n_prio]; new_prio int32 [n_new]; outputs int64 [n_new]."""
        w = int(window["prio"].shape[0])
        win = _SloWindow(_ptr(window["prio"]) if w else None, _ptr(window["ttft_ns"]) if w else None,
                         _ptr(window["tpot_ns"]) if w else None, _ptr(window["queue_ns"]) if w else None, w, 0)
        bs = _SloBounds(*[_ptr(bounds[k]) for k in SLO_BOUND_FIELDS])
        n_new = int(new_prio.shape[0])
        rc = self._L.hfx_slo_map(self._h, int(n_prio), C.byref(win), C.byref(bs), _ptr(last_queue), _ptr(pending),
                                 _ptr(new_prio) if n_new else None, n_new, _ptr(ttft_out) if n_new else None,
                                 _ptr(tpot_out) if n_new else None)
        if rc != 0:
            raise HfxError(rc, "hfx_slo_map")

    def scale_tick(self, table: DeviceTable, now_ns: int, total_blocks: torch.Tensor, counts: torch.Tensor,
                   used_blocks: torch.Tensor, decision: torch.Tensor, window_ns: int = 10_000_000_000,
                   block_tokens: int = 16, min_samples: int = 10, eps_out=(7, 10), eps_in=(11, 10), eps_wait=(1, 4)):
        """hfx_scale_tick: counts int64 [3, 4], used_blocks int64 [n_replicas], decision int32 [3, 2] (device)."""
        ts = table.c_struct()
        sp = _ScaleParams(int(window_ns), int(block_tokens), int(min_samples), *eps_out, *eps_in, *eps_wait)
        so = _ScaleOut(counts.data_ptr(), used_blocks.data_ptr(), decision.data_ptr())
        rc = self._L.hfx_scale_tick(self._h, C.byref(ts), int(now_ns), total_blocks.data_ptr(), C.byref(sp), C.byref(so))
        if rc != 0:
            raise HfxError(rc, "hfx_scale_tick")

    def scale_decide(self, total_blocks: torch.Tensor, counts: torch.Tensor, used_blocks: torch.Tensor, decision: torch.Tensor,
                     min_samples: int = 10, eps_out=(7, 10), eps_in=(11, 10), eps_wait=(1, 4)):
        """hfx_scale_decide: the decision from counters that are already there (counts and used_blocks are read)."""
        sp = _ScaleParams(1, 1, int(min_samples), *eps_out, *eps_in, *eps_wait)
        so = _ScaleOut(counts.data_ptr(), used_blocks.data_ptr(), decision.data_ptr())
        rc = self._L.hfx_scale_decide(self._h, total_blocks.data_ptr(), C.byref(sp), C.byref(so))
        if rc != 0:
            raise HfxError(rc, "hfx_scale_decide")

    def status(self) -> int:
        w = C.c_uint32(0)
        rc = self._L.hfx_sched_status(self._h, C.byref(w))
        if rc not in (0, E_TIMEOUT):
            raise HfxError(rc, "hfx_sched_status")
        return int(w.value)

    def set_profiling(self, on: bool):
        rc = self._L.hfx_sched_set_profiling(self._h, int(on))
        if rc != 0:
            raise HfxError(rc, "hfx_sched_set_profiling")

    def set_fused_front(self, on: bool):
        """Run the front end of the following steps as the tile kernel (default) or as the fallback
        kernels with global counters; the results are the same."""
        rc = self._L.hfx_sched_set_fused_front(self._h, int(on))
        if rc != 0:
            raise HfxError(rc, "hfx_sched_set_fused_front")

    def get_profile(self) -> Dict[str, Dict[str, float]]:
        """Per-kernel device time (ms) and launches recorded since the last call."""
        pr = _Profile()
        rc = self._L.hfx_sched_get_profile(self._h, C.byref(pr))
        if rc != 0:
            raise HfxError(rc, "hfx_sched_get_profile")
        out = {}
        for i in range(N_KERNELS):
            name = self._L.hfx_kernel_name(i)
            if name and pr.launches[i]:
                out[name.decode()] = {"ms": float(pr.ms[i]), "launches": int(pr.launches[i])}
        return out

    def launch_count(self) -> int:
        return int(self._L.hfx_sched_launch_count(self._h))

    def close(self):
        if self._h:
            self._L.hfx_sched_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
