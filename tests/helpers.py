"""Small helpers shared by the tests (no scheduler arithmetic)."""
import os

import numpy as np

import gen
from gen.workloads import Workload, _empty_table, MS, SEC  # noqa: F401

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def load_pins():
    pins = {}
    with open(os.path.join(GOLDEN, "pins.txt")) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            k, v = line.split()
            pins[k] = int(v, 0)
    return pins


def make_wl(rows, classes, replicas=((gen.COLOCATED, 8192, 0),), now=(0,), maturity=(0,),
            model=gen.DEFAULT_MODEL, budget_mode=gen.BUDGET_SAFE, weight_max=0, trace_off=None,
            sim_iters=0):
    """rows: list of dicts with any of the table's column names (missing = default)."""
    n = len(rows)
    tab = _empty_table(n)
    for i, r in enumerate(rows):
        for k, v in r.items():
            tab[k][i] = v
    return Workload("hand", tuple(model), list(classes), np.array(replicas, np.int32).reshape(-1, 3), tab,
                    np.array(now, np.int64), np.array(maturity, np.int64), budget_mode, weight_max,
                    None if trace_off is None else np.array(trace_off, np.int32), sim_iters)


def permute_rows(wl, perm):
    out = wl.copy()
    for k in out.table:
        out.table[k] = np.ascontiguousarray(out.table[k][perm])
    return out


def oracle_sim_config5_range(args):
    """Worker of a process pool (importable under `spawn`): the single-threaded oracle on traces
    [first, first + count) of config 5, drawn afresh from their seeds (a subset of the batch equals
    the same slice of the full batch).  Returns the per-trace metrics and the table columns the
    simulator writes."""
    first, count, iters = args
    import oracle
    wl = gen.config5(traces=count, first_trace=first, iters=iters)
    res = oracle.sim(wl)
    cols = {k: wl.table[k] for k in ("state", "gen", "first_token_ns", "last_token_ns", "finish_ns")}
    return first, count, res, cols
