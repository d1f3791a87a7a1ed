"""Seeded synthetic workloads for the scheduler hot path.

This module only draws inputs: request tables, replica configurations and
arrival traces with the shapes, length distributions and SLO mixes of
multi-task serving workloads (short prompts of tens to hundreds of tokens, a
long-prompt task, Poisson or bursty arrivals, several SLO classes; cf. the
paper's Table 1 and Sec. 4 set-up).  It holds none of the scheduler's
arithmetic and is the one module that both the CPU oracle's tests and the CUDA
path's tests read, so both sides see byte-identical inputs.

Floating point appears only here (sampling); every column handed on is an
integer array.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

MS = 1_000_000          # ns per millisecond
SEC = 1_000_000_000     # ns per second

QUEUED, RUNNING, DONE, REJECTED = 0, 1, 2, 3
COLOCATED, PREFILL, DECODE = 0, 1, 2
BUDGET_SAFE, BUDGET_CAP_ONLY = 0, 1

# integer-quantised latency model: E_p(t) = c0 + c1 t + c2 t^2, E_d(b, kv) = d0 + d1 b + d2 kv  (ns)
DEFAULT_MODEL = (5_000_000, 40_000, 2, 8_000_000, 100_000, 20)

CLASSES_3 = [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1), (5000 * MS, 100 * MS, 2)]
CLASSES_4 = CLASSES_3 + [(20000 * MS, 200 * MS, 3)]
CLASSES_5 = [(200 * MS, 30 * MS, 0), (500 * MS, 40 * MS, 1), (1000 * MS, 50 * MS, 2),
             (5000 * MS, 100 * MS, 3), (20000 * MS, 200 * MS, 4)]
CLASSES_PD = CLASSES_3 + [(0, 0, 3)]      # plus a throughput-only batch class (no bounds)


@dataclass
class Workload:
    """Inputs of one scheduler configuration (all integer numpy arrays)."""
    name: str
    model: Tuple[int, int, int, int, int, int]
    classes: List[Tuple[int, int, int]]            # (ttft_slo_ns, tpot_slo_ns, prio)
    replicas: np.ndarray                           # int32 [R, 3]: mode, token_cap, batch_cap
    table: Dict[str, np.ndarray]                   # SoA columns
    now: np.ndarray                                # int64 [R]
    maturity: np.ndarray                           # int64 [R]
    budget_mode: int = BUDGET_SAFE
    weight_max: int = 0
    trace_off: Optional[np.ndarray] = None         # int32 [R+1] (simulator workloads)
    sim_iters: int = 0
    steps: int = 1
    meta: dict = field(default_factory=dict)

    @property
    def n_rows(self) -> int:
        return int(self.table["replica_id"].shape[0])

    @property
    def n_replicas(self) -> int:
        return int(self.replicas.shape[0])

    def copy(self) -> "Workload":
        return Workload(self.name, self.model, list(self.classes), self.replicas.copy(),
                        {k: v.copy() for k, v in self.table.items()}, self.now.copy(),
                        self.maturity.copy(), self.budget_mode, self.weight_max,
                        None if self.trace_off is None else self.trace_off.copy(),
                        self.sim_iters, self.steps, dict(self.meta))


def _lognormal_int(rng, mu, sigma, lo, hi, n):
    return np.clip(np.rint(np.exp(mu + sigma * rng.standard_normal(n))), lo, hi).astype(np.int32)


def _pareto_int(rng, alpha, scale, lo, hi, n):
    # classical Pareto with minimum `scale`: scale * U^(-1/alpha)
    u = 1.0 - rng.random(n)
    return np.clip(np.rint(scale * u ** (-1.0 / alpha)), lo, hi).astype(np.int32)


def _bimodal_int(rng, n):
    short = np.exp(5.0 + 0.7 * rng.standard_normal(n))
    long_ = np.exp(9.0 + 0.5 * rng.standard_normal(n))
    pick = rng.random(n) < 0.7
    return np.clip(np.rint(np.where(pick, short, long_)), 16, 131072).astype(np.int32)


def _empty_table(n) -> Dict[str, np.ndarray]:
    return {
        "replica_id": np.zeros(n, np.int32),
        "class_id": np.zeros(n, np.uint8),
        "state": np.zeros(n, np.uint8),
        "prompt_len": np.zeros(n, np.int32),
        "output_len": np.ones(n, np.int32),
        "gen": np.zeros(n, np.int32),
        "arrival_ns": np.zeros(n, np.int64),
        "first_token_ns": np.zeros(n, np.int64),
        "last_token_ns": np.zeros(n, np.int64),
        "finish_ns": np.zeros(n, np.int64),
        "req_id": np.arange(n, dtype=np.int32),
        "weight": np.ones(n, np.int32),
    }


def _replicas(R, mode, token_cap, batch_cap=0):
    a = np.zeros((R, 3), np.int32)
    a[:, 0] = mode
    a[:, 1] = token_cap
    a[:, 2] = batch_cap
    return a


def _class_arrays(classes):
    ttft = np.array([c[0] for c in classes], np.int64)
    tpot = np.array([c[1] for c in classes], np.int64)
    return ttft, tpot


def _make_inflight(rng, tab, idx, classes, now_rows):
    """Mark rows `idx` RUNNING with a random decode progress: gen ~ U[0, output_len),
    first token gen*tpot*u ago (u in [0.5, 1.2]: some ahead of, some behind their
    token deadlines), arrival a little before the first token."""
    _, tpot = _class_arrays(classes)
    k = idx.size
    out = tab["output_len"][idx].astype(np.int64)
    gen = np.floor(rng.random(k) * out).astype(np.int64)
    tp = tpot[tab["class_id"][idx]]
    tp = np.where(tp > 0, tp, 100 * MS)
    u = 0.5 + 0.7 * rng.random(k)
    first = now_rows - np.rint(gen * tp * u).astype(np.int64) - np.rint(rng.random(k) * 20 * MS).astype(np.int64)
    arrival = first - np.rint((0.05 + 0.95 * rng.random(k)) * SEC).astype(np.int64)
    tab["state"][idx] = RUNNING
    tab["gen"][idx] = gen.astype(np.int32)
    tab["first_token_ns"][idx] = first
    tab["last_token_ns"][idx] = now_rows - np.rint(rng.random(k) * 20 * MS).astype(np.int64)
    tab["arrival_ns"][idx] = arrival


# ----------------------------------------------------------------------------------------------
# config 1: one replica, 256 requests, 3 classes, Poisson 20 req/s; one step + a 2000-iteration run
# ----------------------------------------------------------------------------------------------
def config1(seed: int = 0, n: int = 256, rate: float = 20.0) -> Workload:
    rng = np.random.default_rng(seed)
    tab = _empty_table(n)
    tab["class_id"][:] = rng.integers(0, 3, n).astype(np.uint8)
    tab["prompt_len"][:] = _lognormal_int(rng, 6.0, 1.0, 16, 8192, n)
    tab["output_len"][:] = _lognormal_int(rng, 5.0, 0.8, 1, 2048, n)
    gaps = rng.exponential(1.0 / rate, n)
    tab["arrival_ns"][:] = np.rint(np.cumsum(gaps) * SEC).astype(np.int64)
    now = np.array([tab["arrival_ns"][min(n // 2, n - 1)]], np.int64)
    return Workload("config1", DEFAULT_MODEL, CLASSES_3, _replicas(1, COLOCATED, 8192), tab, now,
                    np.zeros(1, np.int64), trace_off=np.array([0, n], np.int32), sim_iters=2000)


# ----------------------------------------------------------------------------------------------
# config 2: R colocated replicas x rows_per requests, rows grouped by replica, 60 % in flight
# ----------------------------------------------------------------------------------------------
def config2(seed: int = 2, R: int = 64, rows_per: int = 4096, inflight: float = 0.6,
            budget_mode: int = BUDGET_SAFE) -> Workload:
    rng = np.random.default_rng(seed)
    n = R * rows_per
    tab = _empty_table(n)
    tab["replica_id"][:] = np.repeat(np.arange(R, dtype=np.int32), rows_per)
    tab["class_id"][:] = rng.choice(4, n, p=[0.4, 0.3, 0.2, 0.1]).astype(np.uint8)
    tab["prompt_len"][:] = _lognormal_int(rng, 6.0, 1.0, 16, 8192, n)
    tab["output_len"][:] = _lognormal_int(rng, 5.0, 0.8, 1, 2048, n)
    now = (1000 * SEC + rng.integers(0, SEC, R)).astype(np.int64)
    now_rows = now[tab["replica_id"]]
    run = rng.random(n) < inflight
    tab["arrival_ns"][:] = now_rows - np.rint(rng.exponential(2.0, n) * SEC).astype(np.int64)
    _make_inflight(rng, tab, np.nonzero(run)[0], CLASSES_4, now_rows[run])
    maturity = now - rng.integers(0, 100 * MS, R)
    return Workload("config2", DEFAULT_MODEL, CLASSES_4, _replicas(R, COLOCATED, 16384), tab, now,
                    maturity.astype(np.int64), budget_mode=budget_mode,
                    meta={"inflight": inflight})


# ----------------------------------------------------------------------------------------------
# config 3: disaggregated: R/2 prefill replicas + R/2 decode replicas
# ----------------------------------------------------------------------------------------------
def config3(seed: int = 3, R: int = 256, rows_per: int = 16384) -> Workload:
    rng = np.random.default_rng(seed)
    RP = R // 2
    n = R * rows_per
    tab = _empty_table(n)
    tab["replica_id"][:] = np.repeat(np.arange(R, dtype=np.int32), rows_per)
    tab["class_id"][:] = rng.choice(4, n, p=[0.3, 0.3, 0.2, 0.2]).astype(np.uint8)
    tab["prompt_len"][:] = _bimodal_int(rng, n)
    tab["output_len"][:] = _lognormal_int(rng, 5.0, 0.8, 1, 2048, n)
    now = (1000 * SEC + rng.integers(0, SEC, R)).astype(np.int64)
    now_rows = now[tab["replica_id"]]
    tab["arrival_ns"][:] = now_rows - np.rint(rng.exponential(2.0, n) * SEC).astype(np.int64)
    reps = np.concatenate([_replicas(RP, PREFILL, 32768), _replicas(R - RP, DECODE, 32768, 256)])
    # a quarter of the prefill replicas are busy with a batch: maturity in the future
    maturity = now - rng.integers(0, 100 * MS, R)
    busy = rng.random(R) < 0.25
    busy[RP:] = False
    maturity = np.where(busy, now + rng.integers(1 * MS, 400 * MS, R), maturity).astype(np.int64)
    # decode replicas: n_run ~ U[0, 256] running rows; the rest prefilled and waiting to migrate
    dec_rows = tab["replica_id"] >= RP
    ttft, _ = _class_arrays(CLASSES_PD)
    wait = np.rint(rng.exponential(0.05, n) * SEC).astype(np.int64)
    first = now_rows - wait
    pre_lat = np.rint((0.05 + 0.5 * rng.random(n)) * SEC).astype(np.int64)
    tab["first_token_ns"][dec_rows] = first[dec_rows]
    tab["last_token_ns"][dec_rows] = first[dec_rows]
    tab["arrival_ns"][dec_rows] = (first - pre_lat)[dec_rows]
    for r in range(RP, R):
        k = int(rng.integers(0, 257))
        lo = r * rows_per
        idx = lo + rng.choice(rows_per, size=min(k, rows_per), replace=False)
        idx.sort()
        _make_inflight(rng, tab, idx, CLASSES_PD, now_rows[idx])
    return Workload("config3", DEFAULT_MODEL, CLASSES_PD, reps, tab, now, maturity)


# ----------------------------------------------------------------------------------------------
# config 4: one shared arrival-ordered queue of n requests over R replicas (rows interleaved),
#           priority weights, Pareto prompts, several committed steps
# ----------------------------------------------------------------------------------------------
def config4(seed: int = 4, R: int = 1024, n: int = 1 << 20, steps: int = 10,
            budget_mode: int = BUDGET_SAFE) -> Workload:
    rng = np.random.default_rng(seed)
    tab = _empty_table(n)
    tab["replica_id"][:] = rng.integers(0, R, n).astype(np.int32)
    tab["class_id"][:] = rng.integers(0, 5, n).astype(np.uint8)
    tab["weight"][:] = rng.integers(1, 17, n).astype(np.int32)
    tab["prompt_len"][:] = _pareto_int(rng, 1.5, 16.0, 16, 131072, n)
    tab["output_len"][:] = _lognormal_int(rng, 5.0, 0.8, 1, 2048, n)
    tab["arrival_ns"][:] = np.sort(np.rint(rng.random(n) * 60 * SEC).astype(np.int64))
    now = np.full(R, 30 * SEC, np.int64)
    # per replica, its n_run ~ U[0, 192] earliest rows are already in flight
    n_run = rng.integers(0, 193, R)
    order = np.argsort(tab["replica_id"], kind="stable")          # rows of a replica in arrival order
    rid_sorted = tab["replica_id"][order]
    starts = np.searchsorted(rid_sorted, np.arange(R))
    rank = np.arange(n) - starts[rid_sorted]
    inflight_sorted = rank < n_run[rid_sorted]
    idx = np.sort(order[inflight_sorted])
    idx = idx[tab["arrival_ns"][idx] <= 30 * SEC]
    arrival_keep = tab["arrival_ns"][idx].copy()
    _make_inflight(rng, tab, idx, CLASSES_5, np.full(idx.size, 30 * SEC, np.int64))
    # keep the queue's arrival order; the first token cannot precede the arrival
    tab["arrival_ns"][idx] = np.minimum(arrival_keep, tab["first_token_ns"][idx])
    return Workload("config4", DEFAULT_MODEL, CLASSES_5, _replicas(R, COLOCATED, 16384), tab, now,
                    np.full(R, 30 * SEC, np.int64) - rng.integers(0, 50 * MS, R),
                    budget_mode=budget_mode, weight_max=16, steps=steps)


# ----------------------------------------------------------------------------------------------
# config 5: Monte-Carlo batch of traces, each one colocated replica with bursty arrivals
# ----------------------------------------------------------------------------------------------
def _mmpp_arrivals(rng, n, rates=(5.0, 80.0), period=10.0):
    """Two-state modulated Poisson process: the rate is re-drawn (switch with
    probability 1/2) at every `period` boundary."""
    out = np.empty(n, np.float64)
    got = 0
    state = int(rng.integers(0, 2))
    t0 = 0.0
    while got < n:
        k = int(rng.poisson(rates[state] * period))
        ts = np.sort(t0 + rng.random(k) * period)
        take = min(k, n - got)
        out[got:got + take] = ts[:take]
        got += take
        t0 += period
        if rng.random() < 0.5:
            state = 1 - state
    return np.rint(out * SEC).astype(np.int64)


def config5(seed: int = 5, traces: int = 4096, rows_per: int = 2048, iters: int = 10000,
            first_trace: int = 0) -> Workload:
    """Trace j is drawn from seed (seed, first_trace + j): a subset of the batch
    is the same as the corresponding slice of the full batch."""
    n = traces * rows_per
    tab = _empty_table(n)
    tab["replica_id"][:] = np.repeat(np.arange(traces, dtype=np.int32), rows_per)
    for j in range(traces):
        rng = np.random.default_rng([seed, first_trace + j])
        s = slice(j * rows_per, (j + 1) * rows_per)
        tab["class_id"][s] = rng.choice(4, rows_per, p=[0.4, 0.3, 0.2, 0.1]).astype(np.uint8)
        tab["prompt_len"][s] = _lognormal_int(rng, 6.0, 1.0, 16, 8192, rows_per)
        tab["output_len"][s] = _lognormal_int(rng, 5.0, 0.8, 1, 2048, rows_per)
        tab["arrival_ns"][s] = _mmpp_arrivals(rng, rows_per)
    tab["req_id"][:] = np.arange(n, dtype=np.int32)
    off = (np.arange(traces + 1, dtype=np.int64) * rows_per).astype(np.int32)
    return Workload("config5", DEFAULT_MODEL, CLASSES_4, _replicas(traces, COLOCATED, 16384), tab,
                    np.zeros(traces, np.int64), np.zeros(traces, np.int64), trace_off=off,
                    sim_iters=iters)


# ----------------------------------------------------------------------------------------------
# small random tables for property tests and adversarial parity cases
# ----------------------------------------------------------------------------------------------
def random_table(seed: int, n: int, R: int, modes=(COLOCATED,), n_classes: int = 4,
                 grouped: bool = False, permute_ids: bool = True, token_cap: int = 4096,
                 batch_cap: int = 0, tie_heavy: bool = False, weight_max: int = 0,
                 budget_mode: int = BUDGET_SAFE, model=DEFAULT_MODEL,
                 inflight: float = 0.3, done: float = 0.1, future: float = 0.2) -> Workload:
    """A mixed-state table: running, visible queued, future, done and rejected rows;
    `tie_heavy` draws every field from a handful of values so that every key field ties."""
    rng = np.random.default_rng(seed)
    tab = _empty_table(n)
    rid = rng.integers(0, R, n).astype(np.int32)
    if grouped:
        rid.sort()
    tab["replica_id"][:] = rid
    base = [(200 * MS, 30 * MS), (1000 * MS, 50 * MS), (5000 * MS, 100 * MS), (0, 0),
            (20000 * MS, 200 * MS), (300 * MS, 0), (0, 40 * MS), (50 * MS, 20 * MS)]
    classes = [(base[i % len(base)][0], base[i % len(base)][1], int(rng.integers(0, 4)) if tie_heavy else i % 63)
               for i in range(n_classes)]
    tab["class_id"][:] = rng.integers(0, n_classes, n).astype(np.uint8)
    if tie_heavy:
        tab["prompt_len"][:] = rng.choice([16, 64, 64, 256], n).astype(np.int32)
        tab["output_len"][:] = rng.choice([1, 2, 8], n).astype(np.int32)
    else:
        tab["prompt_len"][:] = _lognormal_int(rng, 5.0, 1.2, 1, 3 * token_cap // 2, n)
        tab["output_len"][:] = _lognormal_int(rng, 3.0, 1.0, 1, 512, n)
    tab["weight"][:] = rng.integers(0, max(weight_max, 1) + 3, n).astype(np.int32)
    now = (100 * SEC + rng.integers(0, 2, R) * 7 * MS).astype(np.int64)
    now_rows = now[np.clip(rid, 0, R - 1)]
    u = rng.random(n)
    if tie_heavy:
        tab["arrival_ns"][:] = now_rows - rng.choice([0, 10 * MS, 10 * MS, 3 * SEC], n)
    else:
        tab["arrival_ns"][:] = now_rows - np.rint(rng.exponential(1.0, n) * SEC).astype(np.int64)
    fut = u < future
    tab["arrival_ns"][fut] = now_rows[fut] + 1 + np.rint(rng.random(int(fut.sum())) * SEC).astype(np.int64)
    run = (u >= future) & (u < future + inflight)
    idx = np.nonzero(run)[0]
    if idx.size:
        _make_inflight(rng, tab, idx, classes, now_rows[idx])
        if tie_heavy:
            tab["gen"][idx] = rng.choice([0, 1, 5], idx.size).astype(np.int32)
            tab["first_token_ns"][idx] = now_rows[idx] - rng.choice([0, 30 * MS, 100 * MS], idx.size)
    dn = (u >= future + inflight) & (u < future + inflight + done)
    tab["state"][dn] = rng.choice([DONE, REJECTED], int(dn.sum())).astype(np.uint8)
    # queued rows of decode replicas are prefilled: they carry a first-token time
    q = tab["state"] == QUEUED
    tab["first_token_ns"][q] = tab["arrival_ns"][q] + np.rint(rng.random(int(q.sum())) * 300 * MS).astype(np.int64)
    if permute_ids:
        tab["req_id"][:] = rng.permutation(n).astype(np.int32) * 3 - n   # unique, unordered, some negative
    reps = np.zeros((R, 3), np.int32)
    reps[:, 0] = rng.choice(np.array(modes, np.int32), R)
    reps[:, 1] = token_cap
    reps[:, 2] = batch_cap
    maturity = now - rng.integers(0, 50 * MS, R)
    late = rng.random(R) < 0.15
    maturity = np.where(late, now + rng.integers(1, 200 * MS, R), maturity).astype(np.int64)
    return Workload(f"random{seed}", model, classes, reps, tab, now, maturity,
                    budget_mode=budget_mode, weight_max=weight_max)


def random_traces(seed: int, traces: int, rows_lo: int, rows_hi: int, iters: int,
                  rate: float = 30.0, token_cap: int = 8192, model=DEFAULT_MODEL,
                  classes=None, out_hi: int = 256) -> Workload:
    """Ragged batch of short traces for simulator parity tests."""
    rng = np.random.default_rng(seed)
    lens = rng.integers(rows_lo, rows_hi + 1, traces)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    n = int(off[-1])
    classes = classes or CLASSES_PD
    tab = _empty_table(n)
    tab["replica_id"][:] = np.repeat(np.arange(traces, dtype=np.int32), lens)
    tab["class_id"][:] = rng.integers(0, len(classes), n).astype(np.uint8)
    tab["prompt_len"][:] = _lognormal_int(rng, 6.0, 1.2, 1, 3 * token_cap // 2, n)
    tab["output_len"][:] = _lognormal_int(rng, 3.5, 1.0, 1, out_hi, n)
    for j in range(traces):
        m = int(lens[j])
        if m:
            r = rate * (0.2 + 2.0 * rng.random())
            tab["arrival_ns"][off[j]:off[j + 1]] = np.rint(np.cumsum(rng.exponential(1.0 / r, m)) * SEC).astype(np.int64)
    tab["req_id"][:] = rng.permutation(n).astype(np.int32)
    return Workload(f"traces{seed}", model, classes, _replicas(traces, COLOCATED, token_cap), tab,
                    np.zeros(traces, np.int64), np.zeros(traces, np.int64), trace_off=off,
                    sim_iters=iters)


def pd_pairs(seed: int, pairs: int, rows_per: int, rate: float = 40.0, token_cap: int = 8192, batch_cap: int = 64,
             out_hi: int = 24, classes=None, permute_ids: bool = True) -> Workload:
    """Disaggregated deployment for the coupled P/D tests: `pairs` P instances (replicas 0 .. pairs-1) and
    their partner D instances (replicas pairs .. 2 pairs-1).  Every request starts QUEUED on a P instance
    (Poisson arrivals from time 0, short outputs so that requests finish within a few dozen rounds); all
    clocks start at 0.  The partner table is `np.arange(pairs, 2 pairs)` for the P instances, -1 for the rest."""
    rng = np.random.default_rng(seed)
    classes = classes or CLASSES_PD
    n = pairs * rows_per
    tab = _empty_table(n)
    tab["replica_id"][:] = rng.integers(0, pairs, n).astype(np.int32)
    tab["class_id"][:] = rng.integers(0, len(classes), n).astype(np.uint8)
    tab["prompt_len"][:] = _lognormal_int(rng, 5.5, 1.0, 1, token_cap // 2, n)
    tab["output_len"][:] = rng.integers(1, out_hi + 1, n).astype(np.int32)
    tab["arrival_ns"][:] = np.rint(np.sort(rng.exponential(1.0 / (rate * pairs), n).cumsum()) * SEC).astype(np.int64)
    if permute_ids:          # ids in arrival order otherwise (the table is sorted by arrival)
        tab["req_id"][:] = rng.permutation(n).astype(np.int32)
    reps = np.concatenate([_replicas(pairs, PREFILL, token_cap), _replicas(pairs, DECODE, token_cap, batch_cap)])
    return Workload(f"pd{seed}", DEFAULT_MODEL, classes, reps, tab, np.zeros(2 * pairs, np.int64),
                    np.zeros(2 * pairs, np.int64))


def pd_partner_table(pairs: int) -> np.ndarray:
    return np.concatenate([np.arange(pairs, 2 * pairs), -np.ones(pairs)]).astype(np.int32)


def elastic(seed: int, R: int, n: int, rates=(10.0, 120.0), period: float = 2.0, token_cap: int = 8192,
            batch_cap: int = 64, out_hi: int = 24, prompt_hi: int = 2000) -> Workload:
    """Colocated fleet of up to R instances fed from one global queue, for the scaling loop: n requests, unbound
    (replica_id -1), arriving as a two-state modulated Poisson process (quiet / burst, re-drawn every `period`
    seconds) so that load rises above and falls below what a fixed fleet serves; short outputs, all clocks 0.
    Prompts stay below the safe budget of an idle instance under the strictest TTFT (2144 tokens with the default
    model), so every request can be dispatched at some time."""
    rng = np.random.default_rng(seed)
    tab = _empty_table(n)
    tab["replica_id"][:] = -1
    tab["class_id"][:] = rng.choice(4, n, p=[0.4, 0.3, 0.2, 0.1]).astype(np.uint8)
    tab["prompt_len"][:] = _lognormal_int(rng, 6.0, 1.0, 16, prompt_hi, n)
    tab["output_len"][:] = rng.integers(1, out_hi + 1, n).astype(np.int32)
    tab["arrival_ns"][:] = _mmpp_arrivals(rng, n, rates, period)
    tab["req_id"][:] = np.arange(n, dtype=np.int32)
    return Workload(f"elastic{seed}", DEFAULT_MODEL, CLASSES_4, _replicas(R, COLOCATED, token_cap, batch_cap), tab,
                    np.zeros(R, np.int64), np.zeros(R, np.int64))


INST_OFF, INST_STARTING, INST_ACTIVE, INST_DRAINING = 0, 1, 2, 3
T_NEVER = np.iinfo(np.int64).max


def new_fleet(blocks_cap, active) -> Dict[str, np.ndarray]:
    """Instance records for the scaling loop: the instances listed in `active` are ACTIVE since time 0 and due
    for dispatching at once, the others are OFF (never due)."""
    cap = np.ascontiguousarray(blocks_cap, np.int32)
    R = cap.size
    f = dict(inst_state=np.zeros(R, np.int32), ready=np.zeros(R, np.int64), billed=np.zeros(R, np.int64),
             since=np.zeros(R, np.int64), total_blocks=np.zeros(R, np.int32), due=np.full(R, T_NEVER, np.int64),
             blocks_cap=cap.copy())
    a = np.asarray(list(active), np.int64)
    f["inst_state"][a] = INST_ACTIVE
    f["due"][a] = 0
    f["total_blocks"][a] = cap[a]
    return f


def by_name(name: str, **kw) -> Workload:
    return {"config1": config1, "config2": config2, "config3": config3, "config4": config4,
            "config5": config5}[name](**kw)
