"""Run a workload through the CUDA library and through the oracle, and compare bit for bit."""
import numpy as np
import torch

import oracle
import paper_2508_15919_b200 as hfx

STEP_KEYS = {"slack": "slack_ns", "pred_ttft": "pred_ttft_ns", "pred_tpot": "pred_tpot_ns", "key": "key",
             "order": "order", "seg_off": "seg_off", "admit": "admit", "admitted_rows": "admitted_rows",
             "budget": "budget", "e_d": "e_d_ns", "n_run": "n_run", "sum_kv": "sum_kv", "adm_cost": "adm_cost",
             "adm_count": "adm_count", "maturity_next": "maturity_next"}
STATE_COLS = ["state", "gen", "first_token_ns", "last_token_ns", "finish_ns"]
SIM_KEYS = {"iters_executed": "iters_executed", "finished": "finished", "rejected": "rejected", "attained": "attained",
            "ttft_p50": "ttft_p50_ns", "ttft_p99": "ttft_p99_ns", "tpot_p50": "tpot_p50_ns", "tpot_p99": "tpot_p99_ns",
            "now": "now_ns"}


def make_sched(wl, max_rows=None):
    return hfx.Scheduler(wl.model, wl.classes, wl.replicas, max_rows or max(wl.n_rows, 1),
                         budget_mode=wl.budget_mode, weight_max=wl.weight_max, first_fit=bool(wl.meta.get("first_fit", False)))


def assert_step_parity(wl, steps=1, commit=False, optional=True, sched=None):
    """Run `steps` iterations on both sides from the same inputs; every output and (with commit)
    every table / clock column must agree exactly after each step.  Returns the last GPU outputs."""
    cpu = wl.copy()
    own = sched is None
    sched = sched or make_sched(wl)
    sched.set_horizon(wl.meta.get("horizon"))
    tab = hfx.DeviceTable.from_numpy(wl.table)
    now = torch.from_numpy(wl.now.copy()).cuda()
    mat = torch.from_numpy(wl.maturity.copy()).cuda()
    out = hfx.StepOut(wl.n_rows, wl.n_replicas, optional=optional)
    g = None
    for s in range(steps):
        sched.step(tab, now, mat, out, commit=commit)
        st_gpu = sched.status()
        g = out.to_numpy()
        c = oracle.step(cpu, commit=commit)
        assert st_gpu == c["status"], (s, st_gpu, c["status"])
        for ko, kg in STEP_KEYS.items():
            if kg not in g:
                continue
            assert np.array_equal(g[kg], c[ko]), f"step {s}: {kg} differs at {np.nonzero(g[kg] != c[ko])[0][:8]}"
        if commit:
            tg = tab.to_numpy()
            for k in STATE_COLS:
                assert np.array_equal(tg[k], cpu.table[k]), f"step {s}: column {k} differs at {np.nonzero(tg[k] != cpu.table[k])[0][:8]}"
            assert np.array_equal(now.cpu().numpy(), cpu.now), f"step {s}: now"
            assert np.array_equal(mat.cpu().numpy(), cpu.maturity), f"step {s}: maturity"
        else:
            assert np.array_equal(now.cpu().numpy(), wl.now) and np.array_equal(mat.cpu().numpy(), wl.maturity)
    if own:
        sched.close()
    return g


def run_sim_gpu(wl, iters=None, sched=None):
    own = sched is None
    sched = sched or make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    T = wl.trace_off.shape[0] - 1
    out = hfx.SimOut(T)
    sched.sim_run(tab, wl.trace_off, wl.sim_iters if iters is None else iters, out)
    st = sched.status()
    res = out.to_numpy()
    cols = tab.to_numpy()
    if own:
        sched.close()
    return res, cols, st


def assert_sim_parity(wl, iters=None, traces=None):
    """GPU simulation of every trace against the oracle on `traces` (default: all)."""
    res, cols, st = run_sim_gpu(wl, iters)
    T = wl.trace_off.shape[0] - 1
    traces = list(range(T)) if traces is None else list(traces)
    cpu = wl.copy()
    st_cpu = 0
    for j in traces:
        c = oracle.sim(cpu, iters=iters, j0=j, j1=j + 1)
        st_cpu |= c["status"]
        a, b = wl.trace_off[j], wl.trace_off[j + 1]
        for ko, kg in SIM_KEYS.items():
            assert res[kg][j] == c[ko][j], f"trace {j}: {kg}: gpu {res[kg][j]} oracle {c[ko][j]}"
        for k in STATE_COLS:
            assert np.array_equal(cols[k][a:b], cpu.table[k][a:b]), f"trace {j}: column {k} differs at {np.nonzero(cols[k][a:b] != cpu.table[k][a:b])[0][:8]}"
    if len(traces) == T:
        assert st == st_cpu, (st, st_cpu)
    return res


DISPATCH_KEYS = {"assign": "assign", "queue_order": "queue_order", "n_queue": "n_queue", "inst_order": "inst_order",
                 "n_mature": "n_mature", "slack": "slack_ns", "budget": "budget", "e_d": "e_d_ns", "n_run": "n_run",
                 "sum_kv": "sum_kv", "adm_cost": "adm_cost", "adm_count": "adm_count", "maturity_next": "maturity_next"}


def assert_dispatch_parity(wl, now, sched=None, calls=1):
    """hfx_dispatch_step against the oracle's dispatch on the same table, every output bit for bit."""
    own = sched is None
    sched = sched or make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    mat = torch.from_numpy(wl.maturity.copy()).cuda()
    out = hfx.DispatchOut(wl.n_rows, wl.n_replicas)
    c = oracle.dispatch(wl, now)
    g = None
    for _ in range(calls):
        sched.dispatch_step(tab, now, mat, out)
        st = sched.status()
        g = out.to_numpy()
        assert st == c["status"], (st, c["status"])
        for ko, kg in DISPATCH_KEYS.items():
            assert np.array_equal(g[kg], c[ko]), f"{kg} differs at {np.nonzero(g[kg] != c[ko])[0][:8]}: gpu {g[kg][np.nonzero(g[kg] != c[ko])[0][:4]]} oracle {c[ko][np.nonzero(g[kg] != c[ko])[0][:4]]}"
    if own:
        sched.close()
    return g
