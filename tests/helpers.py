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


# ---- inputs of the D stage of the dispatching call (shared by the tests of the oracle and the parity tests) ----
def migrator_case(seed, **kw):
    modes = (gen.PREFILL, gen.DECODE, gen.DECODE, gen.COLOCATED, gen.DECODE)[: 2 + seed % 4]
    wl = gen.random_table(200 + seed, 80 + 41 * seed, len(modes), modes=modes, inflight=0.7, **kw)
    wl.replicas[:, 0] = modes          # (the generator draws the modes; here every instance has the one listed)
    now = int(wl.now.max())
    t = wl.table
    run_on_p = (t["state"] == gen.RUNNING) & (wl.replicas[np.clip(t["replica_id"], 0, wl.n_replicas - 1), 0] == gen.PREFILL)
    # prefill batches that ended up to 40 ms ago, a few that have not ended yet
    rng = np.random.default_rng(seed)
    t["first_token_ns"][run_on_p] = now - rng.integers(-3 * MS, 40 * MS, int(run_on_p.sum()))
    wl.maturity[:] = now - rng.integers(-2 * MS, 20 * MS, wl.n_replicas)
    return wl, now


def migrator_hand_case():
    # model with a decode iteration of 8 ms + 2 ms per request + 0.2 us per token of context
    now = 1000 * MS
    model = (5_000_000, 40_000, 2, 8_000_000, 2_000_000, 200)
    classes = [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1)]
    rows = [dict(state=1, replica_id=2, class_id=1, prompt_len=10_000, gen=100, output_len=500, first_token_ns=now - 6000 * MS),   # in flight on D instance 2
            dict(state=1, replica_id=2, class_id=1, prompt_len=10_000, gen=100, output_len=500, first_token_ns=now - 6000 * MS),
            dict(state=1, replica_id=0, class_id=1, prompt_len=70_000, gen=0, output_len=50, first_token_ns=now - 20 * MS),      # A  row 2
            dict(state=1, replica_id=0, class_id=0, prompt_len=5000, gen=0, output_len=50, first_token_ns=now - 25 * MS),       # B  row 3
            dict(state=1, replica_id=0, class_id=0, prompt_len=40_000, gen=0, output_len=50, first_token_ns=now - 1 * MS),       # C  row 4
            dict(state=1, replica_id=0, class_id=0, prompt_len=100, gen=0, output_len=50, first_token_ns=now + 1)]             # its prefill batch has not ended
    wl = make_wl(rows, classes, replicas=[(gen.PREFILL, 8192, 0), (gen.DECODE, 8192, 0), (gen.DECODE, 8192, 3)],
                 now=[now] * 3, maturity=[now + 1, now - 5 * MS, now - 10 * MS], model=model)
    return wl, now
