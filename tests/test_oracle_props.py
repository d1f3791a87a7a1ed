"""Invariants, brute force and permutation tests of the oracle (CPU only)."""
import itertools

import numpy as np
import pytest

import gen
import oracle
from helpers import MS, SEC, make_wl, permute_rows, migrator_case

MODES3 = (gen.COLOCATED, gen.PREFILL, gen.DECODE)


def _cases():
    for seed in range(12):
        yield gen.random_table(seed, 300 + 37 * seed, 1 + seed % 5, modes=MODES3, tie_heavy=seed % 3 == 0,
                               batch_cap=(0, 7)[seed % 2], weight_max=(0, 16)[seed % 4 == 1],
                               budget_mode=(gen.BUDGET_SAFE, gen.BUDGET_CAP_ONLY)[seed % 5 == 2])


@pytest.mark.parametrize("wl", list(_cases()), ids=lambda w: w.name)
def test_step_invariants(wl):
    o = oracle.step(wl)
    t = wl.table
    R = wl.n_replicas
    assert o["status"] == 0
    assert o["seg_off"][0] == 0 and o["seg_off"][R] == wl.n_rows
    assert sorted(o["order"]) == list(range(wl.n_rows))            # a permutation
    ttft = np.array([c[0] for c in wl.classes]); tpot = np.array([c[1] for c in wl.classes])
    for r in range(R):
        rows = o["order"][o["seg_off"][r]:o["seg_off"][r + 1]]
        assert np.all(t["replica_id"][rows] == r)
        mode, cap, bcap = wl.replicas[r]
        running = t["state"][rows] == gen.RUNNING
        visible = (t["state"][rows] == gen.QUEUED) & (t["arrival_ns"][rows] <= wl.now[r])
        # in-flight requests are protected: always in the batch, and ordered first
        assert np.all(o["admit"][rows][running] == 1)
        nrun = int(running.sum())
        assert np.all(running[:nrun]) and o["n_run"][r] == nrun
        assert np.all(visible[nrun:nrun + int(visible.sum())])
        inactive = ~(running | visible)
        assert np.all(o["admit"][rows][inactive] == 0) and np.all(o["slack"][rows][inactive] == 0)
        assert o["sum_kv"][r] == int((t["prompt_len"][rows][running].astype(np.int64) + t["gen"][rows][running]).sum())
        # the order is ascending in (key, req_id)
        keys = [(int(k), int(q)) for k, q in zip(o["key"][rows], t["req_id"][rows])]
        assert keys == sorted(keys)
        assert all((k >> 48) == r for k, _ in keys)
        # admitted tokens never exceed the budget; the batch cap holds
        newly = visible & (o["admit"][rows] == 1)
        n_eff = 0 if mode == gen.PREFILL else nrun
        if mode == gen.DECODE:
            cost = wl.model[4] + wl.model[5] * (t["prompt_len"][rows].astype(np.int64) + t["gen"][rows])
        else:
            cost = t["prompt_len"][rows].astype(np.int64)
            assert o["budget"][r] <= max(0, cap - n_eff)
        assert o["adm_cost"][r] == int(cost[newly].sum()) <= o["budget"][r]
        assert o["adm_count"][r] == int(newly.sum())
        if bcap:
            assert o["adm_count"][r] == 0 or n_eff + o["adm_count"][r] <= bcap
        # before maturity the instance is protected
        if wl.now[r] < wl.maturity[r]:
            assert o["budget"][r] == 0 and o["adm_count"][r] == 0
            assert o["maturity_next"][r] == wl.maturity[r]
        # admission is prefix-closed among the rows that fit alone
        elig = visible & (cost <= o["budget"][r])
        adm_seq = o["admit"][rows][elig]
        assert list(adm_seq) == sorted(adm_seq, reverse=True)
        # the compacted admitted list
        lst = o["admitted_rows"][o["seg_off"][r]:o["seg_off"][r + 1]]
        assert list(lst[:o["adm_count"][r]]) == list(rows[newly]) and np.all(lst[o["adm_count"][r]:] == -1)
        # slack of a visible queued row with a TTFT bound on a colocated / prefill replica
        if mode != gen.DECODE:
            start = max(wl.now[r], wl.maturity[r])
            for i in rows[visible][:20]:
                c = t["class_id"][i]
                want = (ttft[c] - (start - t["arrival_ns"][i]) - oracle.Ep(wl.model, int(t["prompt_len"][i]))
                        if ttft[c] > 0 else oracle.SLACK_MAX)
                assert o["slack"][i] == want
                assert o["pred_ttft"][i] == start - t["arrival_ns"][i] + oracle.Ep(wl.model, int(t["prompt_len"][i]))
        else:
            # D stage: a prefilled request's slack runs from its token deadline, first token + (gen+1) TPOT,
            # to the earliest start, net of the step latency the enlarged batch is predicted to have
            start = max(wl.now[r], wl.maturity[r])
            d0, d1, d2 = wl.model[3:]
            for i in rows[visible][:20]:
                c = t["class_id"][i]
                kv_i = int(t["prompt_len"][i]) + int(t["gen"][i])
                ptpot = d0 + d1 * (nrun + 1) + d2 * (int(o["sum_kv"][r]) + kv_i)
                want = (int(t["first_token_ns"][i]) + (int(t["gen"][i]) + 1) * int(tpot[c]) - int(start) - ptpot
                        if tpot[c] > 0 else oracle.SLACK_MAX)
                assert o["slack"][i] == want and o["pred_tpot"][i] == ptpot
                assert o["pred_ttft"][i] == t["first_token_ns"][i] - t["arrival_ns"][i]


@pytest.mark.parametrize("seed", range(6))
def test_outputs_invariant_under_row_permutation(seed):
    wl = gen.random_table(seed + 50, 400, 3, modes=MODES3, tie_heavy=seed % 2 == 0)
    o1 = oracle.step(wl)
    perm = np.random.default_rng(seed).permutation(wl.n_rows)
    wl2 = permute_rows(wl, perm)
    o2 = oracle.step(wl2)
    for k in ("budget", "e_d", "n_run", "sum_kv", "adm_cost", "adm_count", "maturity_next", "seg_off"):
        assert np.array_equal(o1[k], o2[k]), k
    # per-request outputs keyed by req_id
    id1, id2 = wl.table["req_id"], wl2.table["req_id"]
    for k in ("slack", "admit", "key", "pred_ttft", "pred_tpot"):
        a = dict(zip(id1.tolist(), o1[k].tolist())); b = dict(zip(id2.tolist(), o2[k].tolist()))
        assert a == b, k
    assert id1[o1["order"]].tolist() == id2[o2["order"]].tolist()


def _brute_force_best_prefix(costs, budget, count_room):
    """Over all subsets of the rows (given in priority order) that are prefix-closed among the
    rows that fit alone and feasible, the largest one."""
    elig = [j for j, c in enumerate(costs) if c <= budget]
    best = []
    for k in range(len(elig) + 1):
        sub = elig[:k]
        if sum(costs[j] for j in sub) <= budget and (count_room is None or len(sub) <= count_room):
            best = sub
        # feasibility is monotone in k for non-negative costs, but do not assume it here
    return best


@pytest.mark.parametrize("seed", range(40))
def test_admission_against_brute_force(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 9))
    rows = [dict(prompt_len=int(rng.integers(1, 1500)), arrival_ns=int(rng.integers(0, 50 * MS)), req_id=i,
                 class_id=int(rng.integers(0, 2))) for i in range(n)]
    bcap = int(rng.integers(0, 4))
    wl = make_wl(rows, [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1)],
                 replicas=[(gen.COLOCATED, 8192, bcap)], now=[60 * MS])
    o = oracle.step(wl)
    order = list(o["order"])
    costs = [rows[i]["prompt_len"] for i in order]
    best = _brute_force_best_prefix(costs, int(o["budget"][0]), bcap if bcap else None)
    assert sorted(order[j] for j in best) == sorted(np.nonzero(o["admit"])[0].tolist())
    # with equal costs the greedy set also has the maximum count over all feasible subsets
    for r in rows:
        r["prompt_len"] = 300
    wl = make_wl(rows, [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1)],
                 replicas=[(gen.COLOCATED, 8192, bcap)], now=[60 * MS])
    o = oracle.step(wl)
    b = int(o["budget"][0])
    best_count = 0
    for mask in itertools.product([0, 1], repeat=n):
        k = sum(mask)
        if 300 * k <= b and (not bcap or k <= bcap):
            best_count = max(best_count, k)
    assert o["adm_count"][0] == best_count


def test_budget_monotone_in_load():
    cls = [(200 * MS, 30 * MS, 0)]
    prev = None
    for n_run in range(0, 240, 7):
        rows = [dict(state=gen.RUNNING, prompt_len=300, gen=10, first_token_ns=0, req_id=i) for i in range(n_run)]
        rows.append(dict(prompt_len=16, req_id=10_000))
        o = oracle.step(make_wl(rows, cls, now=[MS]))
        if prev is not None:
            assert o["budget"][0] <= prev
        prev = o["budget"][0]
    assert prev == 0            # E_d has passed the TPOT SLO: nothing is safe
    prev = None
    for kv in range(0, 900_000, 50_000):
        rows = [dict(state=gen.RUNNING, prompt_len=kv // 4, gen=0, first_token_ns=0, req_id=i) for i in range(4)]
        rows.append(dict(prompt_len=16, req_id=10_000))
        o = oracle.step(make_wl(rows, cls, now=[MS], replicas=[(gen.COLOCATED, 1 << 20, 0)]))
        if prev is not None:
            assert o["budget"][0] <= prev
        prev = o["budget"][0]


def test_queued_slack_falls_one_for_one_with_time():
    wl = gen.random_table(99, 200, 1, inflight=0.0, done=0.0, future=0.0)
    wl.maturity[:] = 0
    o1 = oracle.step(wl)
    wl.now += 12345
    o2 = oracle.step(wl)
    bounded = np.array([wl.classes[c][0] > 0 for c in wl.table["class_id"]])
    assert np.all((o1["slack"] - o2["slack"])[bounded] == 12345)
    assert np.all(o2["slack"][~bounded] == oracle.SLACK_MAX)


def test_larger_batch_later_maturity():
    cls = [(5000 * MS, 100 * MS, 0)]
    base = [dict(state=gen.RUNNING, prompt_len=300, gen=10, first_token_ns=0, req_id=i) for i in range(8)]
    prev = 0
    for p in (16, 64, 256, 1024, 4096):
        o = oracle.step(make_wl(base + [dict(prompt_len=p, req_id=100)], cls, now=[MS]))
        assert o["adm_count"][0] == 1 and o["maturity_next"][0] > prev
        prev = o["maturity_next"][0]


@pytest.mark.parametrize("seed", range(4))
def test_simulator_conservation(seed):
    wl = gen.random_traces(seed, 6, 0, 120, iters=3000)
    s = oracle.sim(wl)
    t = wl.table
    for j in range(6):
        a, b = wl.trace_off[j], wl.trace_off[j + 1]
        st = t["state"][a:b]
        assert np.all(st <= 3)
        done = st == gen.DONE
        assert s["finished"][j] == int(done.sum()) and s["rejected"][j] == int((st == gen.REJECTED).sum())
        assert s["attained"][j] <= s["finished"][j]
        # a finished request emitted exactly output_len tokens; times are ordered
        assert np.all(t["gen"][a:b][done] + 1 == t["output_len"][a:b][done])
        served = (st == gen.DONE) | (st == gen.RUNNING)
        assert np.all(t["first_token_ns"][a:b][served] >= t["arrival_ns"][a:b][served])
        assert np.all(t["last_token_ns"][a:b][served] >= t["first_token_ns"][a:b][served])
        assert np.all(t["finish_ns"][a:b][done] == t["last_token_ns"][a:b][done])
        assert np.all(t["first_token_ns"][a:b][~served] == -1)
        assert np.all(t["prompt_len"][a:b][st == gen.REJECTED] > 8192)
        assert 0 <= s["iters_executed"][j] <= 3000
        if b > a and s["iters_executed"][j] < 3000:     # ran to completion: nothing is left waiting
            assert not np.any(st == gen.RUNNING)
            left = np.nonzero(st == gen.QUEUED)[0] + a
            if left.size:
                # what is left could never fit: the idle budget set by the strictest TTFT still
                # waiting is smaller than every waiting prompt
                ttfts = [wl.classes[c][0] for c in t["class_id"][left] if wl.classes[c][0] > 0]
                assert ttfts
                n_safe = oracle.nsafe(wl.model, min(ttfts) // 2, 8192)
                assert np.all(t["prompt_len"][left] > n_safe)
        if b == a:
            assert s["iters_executed"][j] == 0 and s["ttft_p50"][j] == -1


def test_simulator_equals_repeated_step_commit():
    wl = gen.random_traces(11, 1, 60, 60, iters=400)
    w1 = wl.copy()
    s = oracle.sim(w1)
    w2 = wl.copy()
    t = w2.table
    t["state"][:] = 0; t["gen"][:] = 0
    for k in ("first_token_ns", "last_token_ns", "finish_ns"):
        t[k][:] = -1
    clocks = []
    for it in range(int(s["iters_executed"][0])):
        oracle.step(w2, commit=True)
        clocks.append(int(w2.now[0]))
    assert clocks == sorted(clocks)
    for k in ("state", "gen", "first_token_ns", "last_token_ns", "finish_ns"):
        assert np.array_equal(w1.table[k], t[k]), k
    assert s["now"][0] == w2.now[0]


def test_percentiles_nearest_rank_against_numpy():
    wl = gen.random_traces(5, 3, 100, 200, iters=20000)
    s = oracle.sim(wl)
    t = wl.table
    for j in range(3):
        a, b = wl.trace_off[j], wl.trace_off[j + 1]
        served = (t["state"][a:b] == gen.DONE) | (t["state"][a:b] == gen.RUNNING)
        v = np.sort((t["first_token_ns"][a:b] - t["arrival_ns"][a:b])[served])
        for p, k in ((50, "ttft_p50"), (99, "ttft_p99")):
            want = np.percentile(v, p, method="inverted_cdf") if v.size else -1
            assert s[k][j] == want


def test_configs_smoke():
    for wl in (gen.config1(), gen.config2(R=4, rows_per=256), gen.config3(R=4, rows_per=512),
               gen.config4(R=8, n=4096), gen.config2(R=4, rows_per=256, inflight=0.02)):
        o = oracle.step(wl)
        assert o["status"] == 0 and sorted(o["order"]) == list(range(wl.n_rows))
    wl = gen.config5(traces=2, rows_per=256, iters=3000)
    s = oracle.sim(wl)
    assert np.all(s["finished"] > 0)
    full = gen.config5(traces=3, rows_per=64, iters=10)
    part = gen.config5(traces=1, rows_per=64, iters=10, first_trace=2)
    assert np.array_equal(full.table["arrival_ns"][128:], part.table["arrival_ns"])


# ---- dispatching over the shared global queue -------------------------------------------------------
def _dispatch_case(seed, **kw):
    wl = gen.random_table(seed, 60 + 37 * seed, 1 + seed % 6, modes=(gen.COLOCATED,), token_cap=(4096, 600)[seed % 2], **kw)
    return wl, int(wl.now.max())


@pytest.mark.parametrize("seed", range(12))
def test_dispatch_invariants(seed):
    wl, now = _dispatch_case(seed, batch_cap=(0, 12)[seed % 3 == 1], tie_heavy=seed % 4 == 2,
                             budget_mode=(gen.BUDGET_SAFE, gen.BUDGET_CAP_ONLY)[seed % 5 == 3])
    o = oracle.dispatch(wl, now)
    t, R = wl.table, wl.n_replicas
    nq, nm = int(o["n_queue"][0]), int(o["n_mature"][0])
    cap_max = int(wl.replicas[:, 1].max())
    queue = o["queue_order"][:nq]
    # the queue is exactly the visible, valid, servable QUEUED rows
    vis = (t["state"] == 0) & (t["arrival_ns"] <= now) & (t["prompt_len"] <= cap_max) & (t["class_id"] < len(wl.classes))
    assert sorted(queue.tolist()) == np.nonzero(vis)[0].tolist() and np.all(o["queue_order"][nq:] == -1)
    # instances take their turn in maturity order, only once matured
    mature = np.nonzero(wl.maturity <= now)[0]
    assert nm == mature.size and sorted(o["inst_order"][:nm].tolist()) == mature.tolist()
    mo = wl.maturity[o["inst_order"][:nm]]
    assert np.all(np.diff(mo) >= 0)
    # consecutive runs of the queue's entries that fit some instance, in instance order; each run within
    # budget and batch cap, each maximal; entries larger than every budget of the call are passed over
    bmax = int(o["budget"][o["inst_order"][:nm]].max()) if nm else 0
    fits = t["prompt_len"][queue] <= bmax
    assert np.all(o["assign"][queue[~fits]] == -1)
    queue = queue[fits]
    cursor = 0
    for r in o["inst_order"][:nm]:
        cnt, cost = int(o["adm_count"][r]), int(o["adm_cost"][r])
        rows = queue[cursor:cursor + cnt]
        assert np.all(o["assign"][rows] == r) and int(t["prompt_len"][rows].sum()) == cost
        assert cost <= o["budget"][r] <= wl.replicas[r, 1]
        cap = int(wl.replicas[r, 2])
        assert cap == 0 or cnt == 0 or o["n_run"][r] + cnt <= cap
        cursor += cnt
        if cursor < queue.size:
            nxt = int(t["prompt_len"][queue[cursor]])
            assert cost + nxt > o["budget"][r] or (cap != 0 and o["n_run"][r] + cnt + 1 > cap)
        assert (o["maturity_next"][r] > now) == (cnt > 0) or cnt == 0
    assert np.all(o["assign"][queue[cursor:]] == -1)
    for r in range(R):
        if wl.maturity[r] > now:
            assert o["budget"][r] == 0 and o["adm_count"][r] == 0 and o["maturity_next"][r] == wl.maturity[r]
    assert np.count_nonzero(o["assign"] >= 0) == int(o["adm_count"].sum())


@pytest.mark.parametrize("seed", range(6))
def test_dispatch_invariant_under_row_permutation(seed):
    wl, now = _dispatch_case(seed, tie_heavy=seed % 2 == 1)
    a = oracle.dispatch(wl, now)
    perm = np.random.default_rng(100 + seed).permutation(wl.n_rows)
    wp = permute_rows(wl, perm)
    b = oracle.dispatch(wp, now)
    ida, idb = wl.table["req_id"], wp.table["req_id"]
    nq = int(a["n_queue"][0])
    assert nq == int(b["n_queue"][0]) and np.array_equal(ida[a["queue_order"][:nq]], idb[b["queue_order"][:nq]])
    assert dict(zip(ida.tolist(), a["assign"].tolist())) == dict(zip(idb.tolist(), b["assign"].tolist()))
    assert dict(zip(ida.tolist(), a["slack"].tolist())) == dict(zip(idb.tolist(), b["slack"].tolist()))
    for k in ("budget", "adm_cost", "adm_count", "maturity_next", "inst_order", "n_run", "sum_kv", "e_d"):
        assert np.array_equal(a[k], b[k]), k


def test_dispatch_single_instance_equals_the_per_replica_step_without_skips():
    # one matured instance, every queued prompt small enough to fit alone, all rows bound to it:
    # the per-replica step admits the same prefix of the same order with the same budget and maturity
    wl = gen.random_table(5, 300, 1, modes=(gen.COLOCATED,), token_cap=4096)
    wl.table["prompt_len"][:] = np.minimum(wl.table["prompt_len"], 40)
    wl.maturity[:] = wl.now - 1
    now = int(wl.now[0])
    d = oracle.dispatch(wl, now)
    s = oracle.step(wl)
    assert d["budget"][0] == s["budget"][0] and d["adm_count"][0] == s["adm_count"][0] > 0
    assert d["adm_cost"][0] == s["adm_cost"][0] and d["maturity_next"][0] == s["maturity_next"][0]
    queued = (wl.table["state"] == 0) & (wl.table["arrival_ns"] <= now)
    assert np.array_equal(d["assign"][queued] == 0, s["admit"][queued] == 1)
    assert np.array_equal(d["slack"][queued], s["slack"][queued])


# ---- first-fit admission variant ---------------------------------------------------------------------------
def test_first_fit_admission_hand_case_and_properties():
    # budget 2144 (idle instance, TTFT 200 ms); queue in priority order: 1144, 1100 (does not fit behind the
    # first), 900 (fits: 2044), 100 (fits exactly: 2144), 16 (nothing left).  The prefix rule stops at the second.
    cls = [(200 * MS, 30 * MS, 0)]
    rows = [dict(prompt_len=pl, arrival_ns=-(5 - k) * MS, req_id=k) for k, pl in enumerate([1144, 1100, 900, 100, 16])]
    wl = make_wl(rows, cls, now=[0])
    o = oracle.step(wl)
    assert o["budget"][0] == 2144 and list(o["admit"]) == [1, 0, 0, 0, 0] and o["adm_cost"][0] == 1144
    wl.meta["first_fit"] = True
    o = oracle.step(wl)
    assert list(o["order"]) == [0, 1, 2, 3, 4] and list(o["admit"]) == [1, 0, 1, 1, 0]
    assert o["adm_cost"][0] == 2144 and o["adm_count"][0] == 3 and list(o["admitted_rows"][:4]) == [0, 2, 3, -1]
    # batch cap 2: the third fitting request is refused
    wl.replicas[0, 2] = 2
    o = oracle.step(wl)
    assert list(o["admit"]) == [1, 0, 1, 0, 0] and o["adm_count"][0] == 2


@pytest.mark.parametrize("seed", range(8))
def test_first_fit_invariants_and_dominance(seed):
    wl = gen.random_table(seed, 400 + 57 * seed, 1 + seed % 5, modes=MODES3 if seed % 2 else (gen.COLOCATED,),
                          batch_cap=(0, 9)[seed % 3 == 1], tie_heavy=seed % 4 == 3)
    a = oracle.step(wl)
    wf = wl.copy(); wf.meta["first_fit"] = True
    b = oracle.step(wf)
    t = wl.table
    # same budgets, same order; first fit admits at least what the prefix rule admits, within the same limits
    assert np.array_equal(a["budget"], b["budget"]) and np.array_equal(a["order"], b["order"])
    assert np.all(b["admit"] >= a["admit"]) and np.all(b["adm_count"] >= a["adm_count"])
    for r in range(wl.n_replicas):
        seg = b["order"][b["seg_off"][r]:b["seg_off"][r + 1]]
        mode, cap, bcap = wl.replicas[r]
        queued = seg[(t["state"][seg] == 0) & (t["arrival_ns"][seg] <= wl.now[r]) & (t["class_id"][seg] < len(wl.classes))]
        cost = t["prompt_len"][queued].astype(np.int64) if mode != gen.DECODE else None
        if cost is None:
            continue
        adm = b["admit"][queued] == 1
        assert cost[adm].sum() == b["adm_cost"][r] <= b["budget"][r]
        # walking the order, a request is refused only if it does not fit what is left at its turn
        used, cnt = 0, 0
        n_eff = 0 if mode == gen.PREFILL else int(b["n_run"][r])
        for k in range(queued.size):
            fits = used + cost[k] <= b["budget"][r] and (bcap == 0 or n_eff + cnt + 1 <= bcap)
            assert bool(adm[k]) == bool(fits)
            if fits:
                used += int(cost[k]); cnt += 1


def test_scaling_loop_invariants():
    # global queue -> dispatcher -> instances, with the Scaler switching instances on and off between ticks
    from oracle.elastic_loop import oracle_round
    R = 8
    wl = gen.elastic(1, R, 1500)
    f = gen.new_fleet([2000] * R, [0, 1])
    on_max, on_later_min, prev_cost, seen = 2, R, 0, set()
    for k in range(330):
        before = f["inst_state"].copy()
        o = oracle_round(wl, f, k)
        st, d = f["inst_state"], o["dispatch"]
        sel = d["assign"] >= 0
        assert np.all(st[d["assign"][sel]] == gen.INST_ACTIVE)                   # only ACTIVE instances are given work
        assert np.all(wl.now[np.unique(d["assign"][sel])] >= o["now"])           # and not before the call was made
        assert np.count_nonzero(st == gen.INST_STARTING) <= 1                    # capacity is not ordered twice
        assert np.array_equal(f["due"] == gen.T_NEVER, st != gen.INST_ACTIVE)
        assert np.array_equal(f["total_blocks"], np.where(st == gen.INST_ACTIVE, 2000, 0))
        assert o["cost"][0] == f["billed"].sum() and o["cost"][0] >= prev_cost and np.all(f["billed"] <= o["now"])
        assert o["cost"][0] - prev_cost <= R * 50 * MS                            # at most every instance for one tick
        for r in range(R):                                                        # the life cycle has no other edges
            assert (before[r], st[r]) in {(0, 0), (0, 1), (1, 1), (1, 2), (2, 2), (2, 3), (3, 3), (3, 2), (3, 0)}, (k, r)
            seen.add((before[r], st[r]))
        off = np.flatnonzero(st == gen.INST_OFF)
        assert not np.any(np.isin(wl.table["replica_id"], off) & np.isin(wl.table["state"], (gen.QUEUED, gen.RUNNING)))
        prev_cost = o["cost"][0]
        n_on = int(np.count_nonzero(st != gen.INST_OFF))
        on_max = max(on_max, n_on)
        if on_max >= 6:
            on_later_min = min(on_later_min, n_on)
    assert on_max >= 6 and on_later_min <= 3, (on_max, on_later_min)             # the fleet grew with the burst and shrank after it
    assert {(0, 1), (1, 2), (2, 3), (3, 0)} <= seen
    assert np.count_nonzero(wl.table["state"] == gen.DONE) > 700
    # every instance's clock stays within one iteration of the global clock once it has work
    busy = np.isin(np.arange(R), wl.table["replica_id"][wl.table["state"] == gen.RUNNING])
    assert np.all(wl.now[busy] <= o["now"] + 1100 * MS)      # one iteration: a prefill batch up to the token cap, then a decode iteration


# ---- the D stage of the dispatching call (the Migrator) ----------------------------------------------
@pytest.mark.parametrize("seed", range(12))
def test_migrator_invariants(seed):
    wl, now = migrator_case(seed, batch_cap=(0, 6)[seed % 3 == 1], tie_heavy=seed % 4 == 2,
                             budget_mode=(gen.BUDGET_SAFE, gen.BUDGET_CAP_ONLY)[seed % 5 == 3])
    o = oracle.dispatch(wl, now)
    t, R, M = wl.table, wl.n_replicas, wl.model
    nq, ndq = int(o["n_queue"][0]), int(o["n_queue"][1])
    nm, nmd = int(o["n_mature"][0]), int(o["n_mature"][1])
    mode = wl.replicas[:, 0]
    ok = (t["class_id"] < len(wl.classes)) & (t["replica_id"] >= 0) & (t["replica_id"] < R)
    on_p = ok & (mode[np.clip(t["replica_id"], 0, R - 1)] == gen.PREFILL)
    pre = (t["state"] == gen.RUNNING) & on_p & (t["first_token_ns"] <= now)
    dqueue = o["queue_order"][nq:nq + ndq]
    assert sorted(dqueue.tolist()) == np.nonzero(pre)[0].tolist() and np.all(o["queue_order"][nq + ndq:] == -1)
    # its order: (priority, clamped slack, request id), the slack being the time to the next-token deadline net
    # of a decode iteration of the request alone
    kv = t["prompt_len"].astype(np.int64) + t["gen"]
    keys = []
    for i in dqueue:
        ttft, tpot, prio = wl.classes[t["class_id"][i]]
        sl = int(t["first_token_ns"][i]) + (int(t["gen"][i]) + 1) * tpot - now - oracle.Ed(M, 1, int(kv[i])) if tpot > 0 else oracle.SLACK_MAX
        assert o["slack"][i] == sl
        keys.append((prio, min(max(sl, oracle.SLACK_MIN), oracle.SLACK_MAX), int(t["req_id"][i])))
    assert keys == sorted(keys)
    # D instances take their turn in maturity order behind the instances of the first stage
    dmat = np.nonzero((mode == gen.DECODE) & (wl.maturity <= now))[0]
    dorder = o["inst_order"][nm:nm + nmd]
    assert sorted(dorder.tolist()) == dmat.tolist() and np.all(np.diff(wl.maturity[dorder]) >= 0)
    assert np.all(o["inst_order"][nm + nmd:] == -1)
    # budgets: a time, from the strictest TPOT in flight or, for an idle instance, of the queue of prefilled requests
    tpot_of = np.array([c[1] for c in wl.classes], np.int64)
    qt = tpot_of[t["class_id"][dqueue]]
    tq = int(qt[qt > 0].min()) if np.any(qt > 0) else oracle.INF
    for r in dorder:
        mine = ok & (t["state"] == gen.RUNNING) & (t["replica_id"] == r)
        rt = tpot_of[t["class_id"][mine]]
        T = int(rt[rt > 0].min()) if np.any(rt > 0) else tq
        if wl.budget_mode == gen.BUDGET_CAP_ONLY or T == oracle.INF:
            assert o["budget"][r] == oracle.INF
        else:
            assert o["budget"][r] == max(T - oracle.Ed(M, int(mine.sum()), int(kv[mine].sum())), 0)
    # consecutive runs of the entries that fit some D instance; within budget and batch room; maximal
    cost_of = M[4] + M[5] * kv
    bmax = int(o["budget"][dorder].max()) if nmd else 0
    fits = cost_of[dqueue] <= bmax
    assert np.all(o["assign"][dqueue[~fits]] == -1)
    queue = dqueue[fits]
    cursor = 0
    for r in dorder:
        cnt, cost = int(o["adm_count"][r]), int(o["adm_cost"][r])
        rows = queue[cursor:cursor + cnt]
        assert np.all(o["assign"][rows] == r) and int(cost_of[rows].sum()) == cost and cost <= o["budget"][r]
        cap = int(wl.replicas[r, 2])
        assert cap == 0 or cnt == 0 or o["n_run"][r] + cnt <= cap
        cursor += cnt
        if cursor < queue.size:
            assert cost + int(cost_of[queue[cursor]]) > o["budget"][r] or (cap != 0 and o["n_run"][r] + cnt + 1 > cap)
        if o["n_run"][r] + cnt > 0:
            assert o["maturity_next"][r] == now + oracle.Ed(M, int(o["n_run"][r]) + cnt, int(o["sum_kv"][r]) + int(kv[rows].sum()))
        else:
            assert o["maturity_next"][r] == wl.maturity[r]
    assert np.all(o["assign"][queue[cursor:]] == -1)
    for r in np.nonzero((mode == gen.DECODE) & (wl.maturity > now))[0]:
        assert o["budget"][r] == 0 and o["adm_count"][r] == 0 and o["maturity_next"][r] == wl.maturity[r]
    assert np.count_nonzero(o["assign"] >= 0) == int(o["adm_count"].sum())


def test_migrator_single_instance_equals_the_per_replica_decode_step():
    # One matured D instance and prefilled requests that each fit alone: handing them to that instance's own queue
    # (what the partner-table hand-off does) and running the per-replica step must admit the same requests with
    # the same budget, cost and maturity -- the two slacks differ by a constant, the order does not.
    for seed in range(6):
        wl = gen.random_table(300 + seed, 200, 2, modes=(gen.PREFILL, gen.DECODE), inflight=0.8, done=0.0, future=0.0, batch_cap=(0, 25)[seed % 2])
        wl.replicas[:, 0] = (gen.PREFILL, gen.DECODE)
        if seed in (0, 4):
            wl.model = wl.model[:4] + (400_000, 200)                    # dearer decode steps: the budget ends the run
        now = int(wl.now.max())
        wl.now[:] = now
        wl.maturity[:] = [now + 1, now - 1]
        t = wl.table
        on_p = t["replica_id"] == 0
        t["state"][on_p] = gen.RUNNING
        t["first_token_ns"][on_p] = now - 5 * MS
        t["gen"][on_p] = 0
        t["state"][(t["replica_id"] == 1) & (t["state"] == gen.QUEUED)] = gen.DONE      # the D instance has no queue of its own
        if seed >= 4:
            t["state"][t["replica_id"] == 1] = gen.DONE                 # an idle D instance: the queue's strictest TPOT
        d = oracle.dispatch(wl, now)
        assert d["n_queue"][1] == int(on_p.sum()) and d["n_mature"][1] == 1
        w2 = wl.copy()
        w2.table["replica_id"][on_p] = 1
        w2.table["state"][on_p] = gen.QUEUED
        s = oracle.step(w2)
        assert d["budget"][1] == s["budget"][1] and d["e_d"][1] == s["e_d"][1]
        cost_of = wl.model[4] + wl.model[5] * (t["prompt_len"].astype(np.int64) + t["gen"])
        if np.all(cost_of[on_p] <= d["budget"][1]):                     # nothing is skipped by either
            nq = int(d["n_queue"][0])
            order_d = d["queue_order"][nq:nq + int(on_p.sum())]
            order_s = [i for i in s["order"] if on_p[i]]
            assert order_d.tolist() == order_s
            assert np.array_equal(np.nonzero(d["assign"] == 1)[0], np.nonzero(s["admit"].astype(bool) & on_p)[0])
            assert d["adm_cost"][1] == s["adm_cost"][1] and d["adm_count"][1] == s["adm_count"][1]
            assert d["maturity_next"][1] == s["maturity_next"][1]
            assert seed not in (0, 4) or 0 < d["adm_count"][1] < d["n_queue"][1]
