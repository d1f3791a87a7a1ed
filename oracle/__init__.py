"""CPU oracle of the scheduler hot path -- TEST INFRASTRUCTURE, not the product.

`hfx_oracle.c` is the oracle (plain single-threaded C written from the paper);
this module compiles it with gcc on first use and wraps it with ctypes + numpy.
Only the tests, the smoke check and the benchmark's CPU-baseline leg import it.
It shares nothing with the CUDA library and never imports it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hfx_oracle.c")
_SO = os.path.join(_HERE, "libhfx_oracle.so")
_lib = None

INF = (1 << 63) - 1
TIME_MAX = 1 << 62
SLACK_MAX = (1 << 39) - 1
SLACK_MIN = -(1 << 39)
CM_WORKED, CM_JUMPED, CM_STUCK = 0, 1, 2
FLAG_COMMIT = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C11, -O2).  Returns the .so path."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-std=gnu11", "-O2", "-fPIC", "-shared", "-Wall", "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


class _Model(C.Structure):
    _fields_ = [(k, C.c_int64) for k in ("c0", "c1", "c2", "d0", "d1", "d2")]


class _Class(C.Structure):
    _fields_ = [("ttft", C.c_int64), ("tpot", C.c_int64), ("prio", C.c_int32), ("pad", C.c_int32)]


class _Replica(C.Structure):
    _fields_ = [("mode", C.c_int32), ("token_cap", C.c_int32), ("batch_cap", C.c_int32)]


class _Config(C.Structure):
    _fields_ = [("model", _Model), ("classes", C.POINTER(_Class)), ("n_classes", C.c_int32),
                ("replicas", C.POINTER(_Replica)), ("n_replicas", C.c_int32),
                ("budget_mode", C.c_int32), ("weight_max", C.c_int32), ("first_fit", C.c_int32),
                ("horizon", C.c_int64)]


_TABLE_COLS = ["replica_id", "class_id", "state", "prompt_len", "output_len", "gen", "arrival_ns",
               "first_token_ns", "last_token_ns", "finish_ns", "req_id", "weight"]


class _Table(C.Structure):
    _fields_ = [("n", C.c_int64)] + [(k, C.c_void_p) for k in _TABLE_COLS]


_STEP_OUT = [("slack", np.int64, "n"), ("pred_ttft", np.int64, "n"), ("pred_tpot", np.int64, "n"),
             ("key", np.uint64, "n"), ("order", np.int32, "n"), ("seg_off", np.int32, "R1"),
             ("admit", np.uint8, "n"), ("admitted_rows", np.int32, "n"), ("budget", np.int64, "R"),
             ("e_d", np.int64, "R"), ("n_run", np.int32, "R"), ("sum_kv", np.int64, "R"),
             ("adm_cost", np.int64, "R"), ("adm_count", np.int32, "R"),
             ("maturity_next", np.int64, "R"), ("epmax", np.int64, "R"), ("n_safe", np.int64, "R")]


class _StepOut(C.Structure):
    _fields_ = [(k, C.c_void_p) for k, _, _ in _STEP_OUT]


_SIM_OUT = [("iters_executed", np.int32), ("finished", np.int32), ("rejected", np.int32),
            ("attained", np.int32), ("ttft_p50", np.int64), ("ttft_p99", np.int64),
            ("tpot_p50", np.int64), ("tpot_p99", np.int64), ("now", np.int64)]


class _SimOut(C.Structure):
    _fields_ = [(k, C.c_void_p) for k, _ in _SIM_OUT]


class _ScaleParams(C.Structure):
    _fields_ = [("window", C.c_int64), ("block_tokens", C.c_int32), ("min_samples", C.c_int32),
                ("eps_out_num", C.c_int32), ("eps_out_den", C.c_int32), ("eps_in_num", C.c_int32),
                ("eps_in_den", C.c_int32), ("eps_wait_num", C.c_int32), ("eps_wait_den", C.c_int32)]


_DISPATCH_OUT = [("assign", np.int32, "n"), ("queue_order", np.int32, "n"), ("n_queue", np.int32, "2"),
                 ("inst_order", np.int32, "R"), ("n_mature", np.int32, "2"), ("slack", np.int64, "n"),
                 ("budget", np.int64, "R"), ("e_d", np.int64, "R"), ("n_run", np.int32, "R"), ("sum_kv", np.int64, "R"),
                 ("adm_cost", np.int64, "R"), ("adm_count", np.int32, "R"), ("maturity_next", np.int64, "R")]


class _DispatchOut(C.Structure):
    _fields_ = [(k, C.c_void_p) for k, _, _ in _DISPATCH_OUT]


class _SloWindow(C.Structure):
    _fields_ = [("w", C.c_int32), ("prio", C.c_void_p), ("ttft", C.c_void_p), ("tpot", C.c_void_p), ("queue", C.c_void_p)]


SLO_BOUND_KEYS = ("ttft_min", "ttft_max", "ttft_min_relaxed", "tpot_min", "tpot_max", "tpot_min_relaxed")


class _SloBounds(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in SLO_BOUND_KEYS]


class _ScaleOut(C.Structure):
    _fields_ = [("counts", C.c_void_p), ("used_blocks", C.c_void_p), ("decision", C.c_void_p)]


class _Fleet(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("inst_state", "ready", "billed", "since", "total_blocks", "due", "blocks_cap")]


FLEET_DTYPES = dict(inst_state=np.int32, ready=np.int64, billed=np.int64, since=np.int64, total_blocks=np.int32,
                    due=np.int64, blocks_cap=np.int32)
INST_OFF, INST_STARTING, INST_ACTIVE, INST_DRAINING = 0, 1, 2, 3
T_NEVER = np.iinfo(np.int64).max


# defaults of the paper: 10 s window, eps_out 0.7, eps_in 1.1, eps_wait 1/4
SCALE_DEFAULTS = dict(window=10_000_000_000, block_tokens=16, min_samples=10, eps_out=(7, 10), eps_in=(11, 10),
                      eps_wait=(1, 4))


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.ora_Ep.restype = C.c_int64
        L.ora_Ep.argtypes = [C.POINTER(_Model), C.c_int64]
        L.ora_Ed.restype = C.c_int64
        L.ora_Ed.argtypes = [C.POINTER(_Model), C.c_int64, C.c_int64]
        L.ora_key.restype = C.c_uint64
        L.ora_key.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int64]
        L.ora_epmax.restype = C.c_int64
        L.ora_epmax.argtypes = [C.c_int64, C.c_int, C.c_int64, C.c_int64]
        L.ora_nsafe.restype = C.c_int64
        L.ora_nsafe.argtypes = [C.POINTER(_Model), C.c_int64, C.c_int64]
        L.ora_step.restype = C.c_uint32
        L.ora_step.argtypes = [C.POINTER(_Config), C.POINTER(_Table), C.c_void_p, C.c_void_p,
                               C.POINTER(_StepOut), C.c_uint32]
        L.ora_sim.restype = C.c_uint32
        L.ora_sim.argtypes = [C.POINTER(_Config), C.POINTER(_Table), C.c_void_p, C.c_int32, C.c_int32,
                              C.c_int32, C.POINTER(_SimOut)]
        L.ora_dispatch.restype = C.c_uint32
        L.ora_dispatch.argtypes = [C.POINTER(_Config), C.POINTER(_Table), C.c_int64, C.c_void_p, C.POINTER(_DispatchOut)]
        L.ora_slo_map.restype = C.c_uint32
        L.ora_slo_map.argtypes = [C.c_int32, C.POINTER(_SloWindow), C.POINTER(_SloBounds), C.c_void_p, C.c_void_p,
                                  C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ora_pd_migrate.restype = C.c_uint32
        L.ora_pd_migrate.argtypes = [C.POINTER(_Config), C.POINTER(_Table), C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                     C.c_void_p]
        L.ora_attainment.restype = C.c_uint32
        L.ora_attainment.argtypes = [C.POINTER(_Config), C.POINTER(_Table), C.c_void_p]
        L.ora_scale_decide.restype = None
        L.ora_scale_decide.argtypes = [C.POINTER(_Config), C.c_void_p, C.POINTER(_ScaleParams), C.POINTER(_ScaleOut)]
        L.ora_dispatch_bind.restype = None
        L.ora_dispatch_bind.argtypes = [C.POINTER(_Config), C.POINTER(_Table), C.c_int64] + [C.c_void_p] * 4
        L.ora_scale_apply.restype = None
        L.ora_scale_apply.argtypes = [C.POINTER(_Config), C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(_Fleet),
                                      C.c_void_p, C.c_void_p, C.c_void_p]
        L.ora_scale.restype = C.c_uint32
        L.ora_scale.argtypes = [C.POINTER(_Config), C.POINTER(_Table), C.c_int64, C.c_void_p, C.POINTER(_ScaleParams),
                                C.POINTER(_ScaleOut)]
        _lib = L
    return _lib


def _model(m) -> _Model:
    return _Model(*[int(x) for x in m])


def Ep(model, t: int) -> int:
    return int(lib().ora_Ep(C.byref(_model(model)), int(t)))


def Ed(model, b: int, kv: int) -> int:
    return int(lib().ora_Ed(C.byref(_model(model)), int(b), int(kv)))


def key(replica: int, phase: int, prio: int, slack: int) -> int:
    return int(lib().ora_key(replica, phase, prio, slack))


def epmax(min_ttft: int, decoding: bool, min_tpot: int, e_d: int) -> int:
    return int(lib().ora_epmax(min_ttft, int(decoding), min_tpot, e_d))


def nsafe(model, epmax_: int, token_cap: int) -> int:
    return int(lib().ora_nsafe(C.byref(_model(model)), epmax_, token_cap))


class _Ctx:
    """Keeps the ctypes structs and the arrays they point to alive together."""

    def __init__(self, wl):
        self.keep = []
        cls = (_Class * len(wl.classes))(*[_Class(int(a), int(b), int(p), 0) for a, b, p in wl.classes])
        reps = (_Replica * wl.n_replicas)(*[_Replica(int(r[0]), int(r[1]), int(r[2])) for r in wl.replicas])
        self.keep += [cls, reps]
        self.cfg = _Config(_model(wl.model), cls, len(wl.classes), reps, wl.n_replicas,
                           int(wl.budget_mode), int(wl.weight_max), int(bool(wl.meta.get("first_fit", False))),
                           int(wl.meta.get("horizon", np.iinfo(np.int64).max)))
        self.table = _Table()
        self.table.n = wl.n_rows
        for k in _TABLE_COLS:
            a = wl.table[k]
            assert a.flags["C_CONTIGUOUS"]
            setattr(self.table, k, a.ctypes.data)


def step(wl, commit: bool = False) -> Dict[str, np.ndarray]:
    """One scheduling iteration over wl (in place on wl.table / wl.now / wl.maturity
    when commit=True).  Returns every output as numpy arrays plus 'status'."""
    L = lib()
    ctx = _Ctx(wl)
    n, R = wl.n_rows, wl.n_replicas
    out = {}
    so = _StepOut()
    for k, dt, dim in _STEP_OUT:
        size = {"n": n, "R": R, "R1": R + 1}[dim]
        out[k] = np.zeros(size, dt)
        setattr(so, k, out[k].ctypes.data)
    now = wl.now if commit else wl.now.copy()
    mat = wl.maturity if commit else wl.maturity.copy()
    st = L.ora_step(C.byref(ctx.cfg), C.byref(ctx.table), now.ctypes.data, mat.ctypes.data,
                    C.byref(so), FLAG_COMMIT if commit else 0)
    out["status"] = int(st)
    return out


def sim(wl, iters: Optional[int] = None, j0: int = 0, j1: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Simulate traces [j0, j1) of wl in place (state, gen and time columns of wl.table
    are overwritten).  Returns per-trace metrics (arrays of n_traces; only [j0, j1) filled)."""
    L = lib()
    ctx = _Ctx(wl)
    T = wl.trace_off.shape[0] - 1
    j1 = T if j1 is None else j1
    out = {}
    so = _SimOut()
    for k, dt in _SIM_OUT:
        out[k] = np.zeros(T, dt)
        setattr(so, k, out[k].ctypes.data)
    off = np.ascontiguousarray(wl.trace_off, np.int32)
    st = L.ora_sim(C.byref(ctx.cfg), C.byref(ctx.table), off.ctypes.data, j0, j1,
                   int(wl.sim_iters if iters is None else iters), C.byref(so))
    out["status"] = int(st)
    return out


def dispatch(wl, now: int) -> Dict[str, np.ndarray]:
    """The dispatching steps over the shared global queue at time `now`: every instance of wl whose
    maturity (wl.maturity) has come takes its turn once, in maturity order; then the same steps for the
    D-stage instances over the queue of prefilled requests.  n_queue and n_mature hold two numbers each
    (the first stage's, the D stage's).  Nothing in wl changes."""
    L = lib()
    ctx = _Ctx(wl)
    n, R = wl.n_rows, wl.n_replicas
    out = {}
    so = _DispatchOut()
    for k, dt, dim in _DISPATCH_OUT:
        out[k] = np.zeros({"n": max(n, 1), "R": R, "2": 2}[dim], dt)
        setattr(so, k, out[k].ctypes.data)
    mat = np.ascontiguousarray(wl.maturity, np.int64)
    st = L.ora_dispatch(C.byref(ctx.cfg), C.byref(ctx.table), int(now), mat.ctypes.data, C.byref(so))
    for k, dt, dim in _DISPATCH_OUT:
        if dim == "n":
            out[k] = out[k][:n]
    out["status"] = int(st)
    return out


def dispatch_bind(wl, now: int, d: Dict[str, np.ndarray]) -> None:
    """Bind the requests that dispatch() assigned (d = its result) to their instances, in place
    (wl.table["replica_id"], wl.now)."""
    L = lib()
    ctx = _Ctx(wl)
    asg = np.ascontiguousarray(d["assign"], np.int32); cnt = np.ascontiguousarray(d["adm_count"], np.int32)
    assert asg.size == wl.n_rows and cnt.size == wl.n_replicas and wl.now.dtype == np.int64
    L.ora_dispatch_bind(C.byref(ctx.cfg), C.byref(ctx.table), int(now), asg.ctypes.data, cnt.ctypes.data,
                        wl.table["replica_id"].ctypes.data, wl.now.ctypes.data)


def pd_migrate(wl, pair: np.ndarray, x0: int, x1: int) -> Dict[str, int]:
    """Hand-off of prefilled requests from the P instances of wl to their partner D instances, in place
    (wl.table["replica_id"], wl.table["state"], wl.now)."""
    L = lib()
    ctx = _Ctx(wl)
    pr = np.ascontiguousarray(pair, np.int32)
    moved = np.zeros(1, np.int32)
    assert wl.table["replica_id"].flags["WRITEABLE"] and wl.now.flags["C_CONTIGUOUS"]
    st = L.ora_pd_migrate(C.byref(ctx.cfg), C.byref(ctx.table), wl.now.ctypes.data, pr.ctypes.data, int(x0), int(x1),
                          moved.ctypes.data)
    return {"status": int(st), "moved": int(moved[0])}


def attainment(wl) -> Dict[str, np.ndarray]:
    """Eq. 2 over wl.table: int64 [n_classes + 1, 6] = requests, DONE, attained, REJECTED, sum of TTFT, sum of
    E2E per class, totals in the last row."""
    L = lib()
    ctx = _Ctx(wl)
    out = np.zeros((len(wl.classes) + 1, 6), np.int64)
    st = L.ora_attainment(C.byref(ctx.cfg), C.byref(ctx.table), out.ctypes.data)
    return {"counts": out, "status": int(st)}


def slo_map(n_prio: int, window: Dict[str, np.ndarray], bounds: Dict[str, np.ndarray], last_queue: np.ndarray,
            pending: np.ndarray, new_prio: np.ndarray) -> Dict[str, np.ndarray]:
    """Priority-based SLO mapping: TTFT / TPOT targets of the requests `new_prio` (row order) from the
    sliding window {prio, ttft, tpot, queue}; returns the targets and the updated last_queue."""
    L = lib()
    wp = np.ascontiguousarray(window["prio"], np.int32)
    wt, wo, wq = (np.ascontiguousarray(window[k], np.int64) for k in ("ttft", "tpot", "queue"))
    win = _SloWindow(int(wp.shape[0]), wp.ctypes.data, wt.ctypes.data, wo.ctypes.data, wq.ctypes.data)
    barr = {k: np.ascontiguousarray(bounds[k], np.int64) for k in SLO_BOUND_KEYS}
    bs = _SloBounds(*[barr[k].ctypes.data for k in SLO_BOUND_KEYS])
    lq = np.ascontiguousarray(last_queue, np.int64).copy()
    pend = np.ascontiguousarray(pending, np.int32)
    npr = np.ascontiguousarray(new_prio, np.int32)
    n = int(npr.shape[0])
    ttft = np.zeros(max(n, 1), np.int64); tpot = np.zeros(max(n, 1), np.int64)
    st = L.ora_slo_map(int(n_prio), C.byref(win), C.byref(bs), lq.ctypes.data, pend.ctypes.data, n, npr.ctypes.data,
                       ttft.ctypes.data, tpot.ctypes.data)
    return {"ttft_slo": ttft[:n], "tpot_slo": tpot[:n], "last_queue": lq, "status": int(st)}


def scale_apply(wl, now: int, decision: np.ndarray, used_blocks: np.ndarray, cold_start, fleet: Dict[str, np.ndarray]) -> np.ndarray:
    """Carry out one tick's decisions on `fleet` (dict of the FLEET_DTYPES arrays, updated in place); of wl the
    replica modes are read and the clocks wl.now / wl.maturity of an instance that comes up are advanced.  Returns
    the cost per pool (instance-time charged so far, Eq. 1 without UnitCost)."""
    L = lib()
    ctx = _Ctx(wl)
    for k, dt in FLEET_DTYPES.items():
        assert fleet[k].dtype == dt and fleet[k].flags["C_CONTIGUOUS"] and fleet[k].shape == (wl.n_replicas,), k
    fl = _Fleet(*[fleet[k].ctypes.data for k in FLEET_DTYPES])
    dec = np.ascontiguousarray(decision, np.int32); used = np.ascontiguousarray(used_blocks, np.int64)
    cold = np.ascontiguousarray(cold_start, np.int64)
    assert dec.size == 6 and used.size == wl.n_replicas and cold.size == 3
    cost = np.zeros(3, np.int64)
    assert wl.now.dtype == np.int64 and wl.maturity.dtype == np.int64
    L.ora_scale_apply(C.byref(ctx.cfg), int(now), dec.ctypes.data, used.ctypes.data, cold.ctypes.data, C.byref(fl),
                      wl.now.ctypes.data, wl.maturity.ctypes.data, cost.ctypes.data)
    return cost


def scale_decide(wl, total_blocks: np.ndarray, counts: np.ndarray, used_blocks: np.ndarray, **kw) -> np.ndarray:
    """The threshold decision per pool from counters and used blocks that are already there (summed over the
    shards of a table, for instance).  Returns decision int32 [3, 2]."""
    L = lib()
    ctx = _Ctx(wl)
    prm = dict(SCALE_DEFAULTS); prm.update(kw)
    sp = _ScaleParams(int(prm["window"]), int(prm["block_tokens"]), int(prm["min_samples"]), *prm["eps_out"],
                      *prm["eps_in"], *prm["eps_wait"])
    cnt = np.ascontiguousarray(counts, np.int64).reshape(3, 4); used = np.ascontiguousarray(used_blocks, np.int64)
    tb = np.ascontiguousarray(total_blocks, np.int32)
    assert used.size == wl.n_replicas and tb.size == wl.n_replicas
    dec = np.zeros((3, 2), np.int32)
    so = _ScaleOut(cnt.ctypes.data, used.ctypes.data, dec.ctypes.data)
    L.ora_scale_decide(C.byref(ctx.cfg), tb.ctypes.data, C.byref(sp), C.byref(so))
    return dec


def scale_tick(wl, now: int, total_blocks: np.ndarray, **kw) -> Dict[str, np.ndarray]:
    """Scaling indicators f1, f2, f3 and the threshold decision per pool at time `now`."""
    L = lib()
    ctx = _Ctx(wl)
    prm = dict(SCALE_DEFAULTS); prm.update(kw)
    sp = _ScaleParams(int(prm["window"]), int(prm["block_tokens"]), int(prm["min_samples"]), *prm["eps_out"],
                      *prm["eps_in"], *prm["eps_wait"])
    out = {"counts": np.zeros((3, 4), np.int64), "used_blocks": np.zeros(wl.n_replicas, np.int64),
           "decision": np.zeros((3, 2), np.int32)}
    so = _ScaleOut(out["counts"].ctypes.data, out["used_blocks"].ctypes.data, out["decision"].ctypes.data)
    tb = np.ascontiguousarray(total_blocks, np.int32)
    out["status"] = int(L.ora_scale(C.byref(ctx.cfg), C.byref(ctx.table), int(now), tb.ctypes.data, C.byref(sp), C.byref(so)))
    return out
