"""The oracle against what the paper and the mathematics fix: hand-worked values
(tests/golden/pins.txt), the closed form of Eq. 3 in exact rationals, single-request
closed forms of the simulator and a two-request case worked out by hand."""
from fractions import Fraction

import numpy as np
import pytest

import gen
import oracle
from helpers import MS, load_pins, make_wl, migrator_hand_case

PINS = load_pins()
M = gen.DEFAULT_MODEL
C200 = [(200 * MS, 30 * MS, 0)]


def test_prefill_model_values():
    for t in (16, 1000, 8192, 32768, 131072, 1281, 1282):
        assert oracle.Ep(M, t) == PINS[f"Ep_{t}"]
    assert oracle.Ed(M, 80, 64000) == PINS["Ed_80_64000"]


def test_key_layout():
    assert oracle.key(3, 1, 0, PINS["slack_queued"]) == PINS["key_queued"]
    assert oracle.key(0, 0, 0, -1) & ((1 << 40) - 1) == PINS["key_low40_slack_minus1"]
    # saturation of the 40-bit slack field
    assert oracle.key(0, 0, 0, -(1 << 50)) & ((1 << 40) - 1) == 0
    assert oracle.key(0, 0, 0, 1 << 50) & ((1 << 40) - 1) == (1 << 40) - 1
    # field order: replica > phase > prio > slack
    assert oracle.key(1, 0, 0, oracle.SLACK_MIN) > oracle.key(0, 3, 63, oracle.SLACK_MAX)
    assert oracle.key(0, 1, 0, oracle.SLACK_MIN) > oracle.key(0, 0, 62, oracle.SLACK_MAX)
    assert oracle.key(0, 1, 1, oracle.SLACK_MIN) > oracle.key(0, 1, 0, oracle.SLACK_MAX)


def test_epmax_and_nsafe_pins():
    ed = PINS["Ed_80_64000"]
    ep = oracle.epmax(200 * MS, True, 30 * MS, ed)
    assert ep == PINS["Epmax_busy"]
    assert oracle.nsafe(M, ep, 8192) == PINS["nsafe_busy"]
    lin = (M[0], M[1], 0) + M[3:]
    assert oracle.nsafe(lin, ep, 8192) == PINS["nsafe_linear"]
    assert oracle.epmax(200 * MS, False, oracle.INF, 0) == PINS["Epmax_idle"]
    assert oracle.nsafe(M, PINS["Epmax_idle"], 8192) == PINS["nsafe_idle"]
    # no TTFT bound in the queue -> capacity only; TPOT <= E_d -> nothing is safe
    assert oracle.epmax(oracle.INF, True, 30 * MS, ed) == oracle.INF
    assert oracle.nsafe(M, oracle.INF, 777) == 777
    assert oracle.epmax(200 * MS, True, ed, ed) == -1
    assert oracle.nsafe(M, -1, 8192) == 0
    assert oracle.nsafe(M, M[0] - 1, 8192) == 0 and oracle.nsafe(M, M[0], 8192) == 0
    assert oracle.nsafe(M, oracle.Ep(M, 1), 8192) == 1


def test_eq3_closed_form_in_exact_rationals():
    """With the paper's linear model E_p = a + b n, the budget must equal floor(Eq. 3)."""
    rng = np.random.default_rng(7)
    for _ in range(3000):
        a = int(rng.integers(0, 20_000_000))
        b = int(rng.integers(1, 200_000))
        lin = (a, b, 0, 8_000_000, 100_000, 20)
        tpot = int(rng.integers(1 * MS, 300 * MS))
        ttft = int(rng.integers(1 * MS, 20_000 * MS))
        ed = int(rng.integers(0, tpot))          # TPOT > E_d
        cap = 1 << 24
        rhs = Fraction((tpot - ed) * ttft, (2 * tpot - ed) * b) - Fraction(a, b)   # Eq. 3
        ep = oracle.epmax(ttft, True, tpot, ed)
        got = oracle.nsafe(lin, ep, cap)
        want = max(0, min(cap, rhs.numerator // rhs.denominator)) if rhs >= 0 else 0
        assert got == want, (a, b, tpot, ttft, ed)


def test_eq3_quadratic_generalisation_brackets():
    rng = np.random.default_rng(8)
    for _ in range(500):
        tpot = int(rng.integers(10 * MS, 300 * MS)); ttft = int(rng.integers(50 * MS, 20_000 * MS))
        ed = int(rng.integers(0, tpot))
        ep = oracle.epmax(ttft, True, tpot, ed)
        # E_p (2 TPOT - E_d)/(TPOT - E_d) <= TTFT holds at ep and fails at ep + 1
        assert Fraction(ep * (2 * tpot - ed), tpot - ed) <= ttft < Fraction((ep + 1) * (2 * tpot - ed), tpot - ed)
        n = oracle.nsafe(M, ep, 16384)
        if n == 0:
            assert oracle.Ep(M, 1) > ep
        else:
            assert oracle.Ep(M, n) <= ep
        if n < 16384:
            assert oracle.Ep(M, n + 1) > ep


def test_queued_slack_closed_form_single_row():
    wl = make_wl([dict(prompt_len=1000, arrival_ns=0)], C200, replicas=[(gen.COLOCATED, 8192, 0)] * 4,
                 now=[10 * MS] * 4, maturity=[0] * 4)
    wl.table["replica_id"][0] = 3
    o = oracle.step(wl)
    assert o["slack"][0] == PINS["slack_queued"]
    assert o["key"][0] == PINS["key_queued"]
    assert o["pred_ttft"][0] == 10 * MS + PINS["Ep_1000"]
    assert o["pred_tpot"][0] == 8_000_000 + 100_000 + 20 * 1000
    assert list(o["seg_off"]) == [0, 0, 0, 0, 1]
    # maturity in the future delays the earliest start
    wl.maturity[3] = 25 * MS
    o = oracle.step(wl)
    assert o["slack"][0] == 200 * MS - 25 * MS - PINS["Ep_1000"]
    assert o["admit"][0] == 0 and o["budget"][3] == 0 and o["adm_count"][3] == 0


def _busy_replica(queued_prompt):
    rows = [dict(state=gen.RUNNING, prompt_len=700, gen=100, first_token_ns=0, arrival_ns=-MS, req_id=i)
            for i in range(80)]                      # n_run = 80, sum_kv = 80 * 800 = 64000
    rows.append(dict(prompt_len=queued_prompt, arrival_ns=0, req_id=1000))
    return make_wl(rows, C200, now=[5 * MS], maturity=[0])


def test_busy_replica_budget_and_maturity():
    wl = _busy_replica(1281)
    o = oracle.step(wl)
    assert o["n_run"][0] == 80 and o["sum_kv"][0] == 64000
    assert o["e_d"][0] == PINS["Ed_80_64000"]
    assert o["epmax"][0] == PINS["Epmax_busy"] and o["n_safe"][0] == PINS["nsafe_busy"]
    assert o["budget"][0] == PINS["nsafe_busy"]
    assert o["admit"][80] == 1 and o["adm_count"][0] == 1 and o["adm_cost"][0] == 1281
    assert o["maturity_next"][0] - wl.now[0] == PINS["maturity_busy_delta"]
    # one token more does not fit
    o = oracle.step(_busy_replica(1282))
    assert o["admit"][80] == 0 and o["adm_count"][0] == 0 and o["maturity_next"][0] == 0
    # running rows: slack = first_token + (gen+1) TPOT - now - E_d
    assert o["slack"][0] == 0 + 101 * 30 * MS - 5 * MS - PINS["Ed_80_64000"]
    assert o["pred_tpot"][0] == PINS["Ed_80_64000"] and o["pred_ttft"][0] == MS
    assert all(o["admit"][:80] == 1)


def test_idle_replica_budget():
    wl = make_wl([dict(prompt_len=2144, arrival_ns=0), dict(prompt_len=2145, arrival_ns=0, req_id=1)],
                 C200, now=[0])
    o = oracle.step(wl)
    assert o["epmax"][0] == PINS["Epmax_idle"] and o["budget"][0] == PINS["nsafe_idle"]
    # equal slack order: shorter prompt has more slack, so the 2145-token row is more urgent but
    # cannot fit alone and is skipped; the 2144-token row is admitted
    assert list(o["order"]) == [1, 0]
    assert list(o["admit"]) == [1, 0]
    assert o["maturity_next"][0] == oracle.Ep(M, 2144)   # k = 0 without a running batch


def test_simulator_single_request_closed_form():
    wl = make_wl([dict(prompt_len=1000, output_len=101, arrival_ns=0)], C200, trace_off=[0, 1], sim_iters=500)
    s = oracle.sim(wl)
    t = wl.table
    assert t["first_token_ns"][0] == PINS["sim1_ttft"]
    assert t["finish_ns"][0] == PINS["sim1_finish"] == PINS["sim1_ttft"] + PINS["sim1_decode_sum"]
    assert t["last_token_ns"][0] == PINS["sim1_finish"]
    assert t["state"][0] == gen.DONE and t["gen"][0] == 100
    assert s["iters_executed"][0] == PINS["sim1_iters"]
    assert s["tpot_p50"][0] == s["tpot_p99"][0] == PINS["sim1_tpot"]
    assert s["ttft_p50"][0] == PINS["sim1_ttft"]
    assert s["attained"][0] == 1 and s["finished"][0] == 1 and s["rejected"][0] == 0
    assert s["now"][0] == PINS["sim1_finish"]


def test_simulator_iteration_limit_and_late_arrival():
    # the request arrives at 1 s: iteration 0 only advances the clock
    wl = make_wl([dict(prompt_len=1000, output_len=101, arrival_ns=1000 * MS)], C200, trace_off=[0, 1], sim_iters=50)
    s = oracle.sim(wl)
    assert s["iters_executed"][0] == 50
    assert wl.table["state"][0] == gen.RUNNING and wl.table["gen"][0] == 48   # 1 jump + 1 prefill + 48 decodes
    assert wl.table["first_token_ns"][0] == 1000 * MS + PINS["sim1_ttft"]
    assert s["finished"][0] == 0 and s["attained"][0] == 0
    assert s["ttft_p50"][0] == PINS["sim1_ttft"] and s["tpot_p50"][0] == -1


def test_simulator_two_requests_hand_worked():
    rows = [dict(prompt_len=1000, output_len=3, arrival_ns=0, req_id=0),
            dict(prompt_len=500, output_len=2, arrival_ns=10 * MS, req_id=1)]
    # replay iteration by iteration with step+commit to check the intermediate values
    wl = make_wl(rows, C200, now=[0], maturity=[0])
    o = oracle.step(wl, commit=True)
    assert list(o["admit"]) == [1, 0] and wl.now[0] == 47 * MS and wl.maturity[0] == 47 * MS
    o = oracle.step(wl, commit=True)
    assert o["epmax"][0] == PINS["sim2_epmax_it1"] and o["n_safe"][0] == PINS["sim2_nsafe_it1"]
    assert o["slack"][1] == PINS["sim2_slackB_it1"] and o["slack"][0] == PINS["sim2_slackA_it1"]
    assert list(o["order"]) == [0, 1] and list(o["admit"]) == [1, 1]
    assert wl.maturity[0] == PINS["sim2_maturity_it1"] and wl.now[0] == PINS["sim2_now_after_it1"]
    assert wl.table["first_token_ns"][1] == 72_500_000 and wl.table["gen"][0] == 1
    o = oracle.step(wl, commit=True)
    assert o["e_d"][0] == 8_230_020 and wl.now[0] == PINS["sim2_finish"]
    assert list(wl.table["state"]) == [gen.DONE, gen.DONE]
    # and the same through the simulator
    wl = make_wl(rows, C200, trace_off=[0, 2], sim_iters=100)
    s = oracle.sim(wl)
    t = wl.table
    assert list(t["finish_ns"]) == [PINS["sim2_finish"]] * 2
    assert t["first_token_ns"][0] - t["arrival_ns"][0] == PINS["sim2_ttft_A"]
    assert t["first_token_ns"][1] - t["arrival_ns"][1] == PINS["sim2_ttft_B"]
    assert s["iters_executed"][0] == PINS["sim2_iters"]
    assert s["ttft_p50"][0] == PINS["sim2_ttft_A"] and s["ttft_p99"][0] == PINS["sim2_ttft_B"]
    assert s["tpot_p50"][0] == PINS["sim2_tpot_B"] and s["tpot_p99"][0] == PINS["sim2_tpot_A"]
    assert s["attained"][0] == 2 and s["finished"][0] == 2


def test_prefill_and_decode_stage_budgets():
    # P-stage: budget from the strictest TTFT of the queue alone (E_d = 0), running rows ignored
    rows = [dict(state=gen.RUNNING, prompt_len=4000, gen=3, first_token_ns=0, class_id=0, req_id=9),
            dict(prompt_len=100, class_id=1, req_id=1), dict(prompt_len=100, class_id=0, req_id=2)]
    cls = [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1)]
    wl = make_wl(rows, cls, replicas=[(gen.PREFILL, 32768, 0)], now=[MS])
    o = oracle.step(wl)
    assert o["epmax"][0] == 100 * MS and o["budget"][0] == 2144 and o["e_d"][0] == 0
    assert o["adm_count"][0] == 2 and o["maturity_next"][0] == MS + oracle.Ep(M, 200)
    # D-stage: budget = strictest in-flight TPOT - E_d(batch), in ns; cost of a request d1 + d2 kv
    rows = [dict(state=gen.RUNNING, prompt_len=900, gen=100, first_token_ns=0, class_id=1, req_id=9),
            dict(prompt_len=500, gen=0, first_token_ns=0, class_id=0, req_id=1),
            dict(prompt_len=2000, gen=0, first_token_ns=0, class_id=0, req_id=2)]
    wl = make_wl(rows, cls, replicas=[(gen.DECODE, 32768, 2)], now=[MS])
    o = oracle.step(wl)
    ed1 = 8_000_000 + 100_000 + 20 * 1000
    assert o["e_d"][0] == ed1 and o["budget"][0] == 50 * MS - ed1
    assert o["adm_count"][0] == 1          # batch cap 2: one running + one migrated
    # the longer prefilled request predicts the larger TPOT, so it has less slack and goes first
    assert list(o["order"]) == [0, 2, 1]
    assert o["adm_cost"][0] == 100_000 + 20 * 2000
    assert o["maturity_next"][0] == MS + 8_000_000 + 2 * 100_000 + 20 * 3000
    # idle D-stage instance: strictest TPOT of the prefilled queue
    rows[0]["state"] = gen.DONE
    wl = make_wl(rows, cls, replicas=[(gen.DECODE, 32768, 0)], now=[MS])
    o = oracle.step(wl)
    assert o["budget"][0] == 30 * MS - 8_000_000 and o["adm_count"][0] == 2
    assert o["maturity_next"][0] == MS + 8_000_000 + 2 * 100_000 + 20 * 2500


def test_decode_stage_queued_slack_hand_worked():
    """D stage, prefilled request waiting in the queue: slack = first token + (gen+1) TPOT - earliest start -
    predicted TPOT of the enlarged batch, with the earliest start at the maturity time while the instance is busy."""
    cls = [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1)]
    rows = [dict(state=gen.RUNNING, prompt_len=900, gen=100, first_token_ns=20 * MS, arrival_ns=5 * MS, class_id=1, req_id=7),
            dict(prompt_len=500, gen=3, first_token_ns=60 * MS, arrival_ns=10 * MS, class_id=0, req_id=1),
            dict(prompt_len=2000, gen=0, first_token_ns=90 * MS, arrival_ns=40 * MS, class_id=1, req_id=2)]
    wl = make_wl(rows, cls, replicas=[(gen.DECODE, 32768, 0)], now=[100 * MS], maturity=[130 * MS])
    o = oracle.step(wl)
    assert o["e_d"][0] == PINS["dq_ed"] and o["n_run"][0] == 1 and o["sum_kv"][0] == 1000
    assert o["slack"][0] == PINS["dq_slack_R0"] and o["pred_tpot"][0] == PINS["dq_ed"]
    assert o["slack"][1] == PINS["dq_slack_Q1"] and o["pred_tpot"][1] == PINS["dq_ptpot_Q1"]
    assert o["slack"][2] == PINS["dq_slack_Q2"] and o["pred_tpot"][2] == PINS["dq_ptpot_Q2"]
    assert o["pred_ttft"][1] == PINS["dq_pttft_Q1"] and o["pred_ttft"][2] == 50 * MS
    assert o["key"][1] == PINS["dq_key_Q1"] and o["key"][2] == PINS["dq_key_Q2"]
    assert list(o["order"]) == [0, 1, 2]
    # busy until maturity: no decision, the maturity time stands
    assert o["budget"][0] == 0 and o["adm_count"][0] == 0 and o["maturity_next"][0] == 130 * MS
    assert list(o["admit"]) == [1, 0, 0]
    # the same instance once matured: the earliest start is now
    wl = make_wl(rows, cls, replicas=[(gen.DECODE, 32768, 0)], now=[100 * MS], maturity=[90 * MS])
    o = oracle.step(wl)
    assert o["slack"][1] == PINS["dq_slack_Q1_matured"] and o["slack"][2] == PINS["dq_slack_Q2_matured"]
    assert o["slack"][0] == PINS["dq_slack_R0"]
    assert o["budget"][0] == PINS["dq_budget_matured"] and o["adm_count"][0] == 2
    assert o["adm_cost"][0] == PINS["dq_adm_cost_matured"] and o["maturity_next"][0] == PINS["dq_maturity_matured"]
    assert list(o["admit"]) == [1, 1, 1]
    # a class without a TPOT bound: the slack saturates high and the request goes last in its priority
    cls2 = cls + [(0, 0, 0)]
    rows2 = rows + [dict(prompt_len=10, gen=0, first_token_ns=1, arrival_ns=0, class_id=2, req_id=0)]
    o = oracle.step(make_wl(rows2, cls2, replicas=[(gen.DECODE, 32768, 0)], now=[100 * MS], maturity=[130 * MS]))
    assert o["slack"][3] == oracle.SLACK_MAX and list(o["order"]) == [0, 1, 3, 2]


def test_cap_only_mode_and_batch_cap():
    rows = [dict(prompt_len=3000, req_id=i, arrival_ns=i) for i in range(5)]
    wl = make_wl(rows, C200, replicas=[(gen.COLOCATED, 8192, 2)], now=[MS], budget_mode=gen.BUDGET_CAP_ONLY)
    o = oracle.step(wl)
    assert o["budget"][0] == 8192 and o["adm_count"][0] == 2 and o["adm_cost"][0] == 6000
    wl = make_wl(rows, C200, replicas=[(gen.COLOCATED, 8192, 0)], now=[MS], budget_mode=gen.BUDGET_CAP_ONLY)
    o = oracle.step(wl)
    assert o["adm_count"][0] == 2          # third request would make 9000 > 8192


def test_oversize_prompt_rejected_on_commit_and_bad_rows_flagged():
    rows = [dict(prompt_len=9000, req_id=0), dict(prompt_len=100, req_id=1, output_len=5), dict(prompt_len=100, class_id=7, req_id=2),
            dict(prompt_len=-5, req_id=3), dict(prompt_len=10, req_id=4, replica_id=5)]
    wl = make_wl(rows, C200, now=[MS])
    o = oracle.step(wl, commit=True)
    assert o["status"] == 1 | 2 | 4
    assert list(wl.table["state"]) == [gen.REJECTED, gen.RUNNING, gen.QUEUED, gen.QUEUED, gen.QUEUED]
    assert list(o["seg_off"]) == [0, 4] and o["order"][4] == 4
    assert list(o["admit"]) == [0, 1, 0, 0, 0]


def test_commit_of_the_disaggregated_stages_hand_worked():
    cls = [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1)]
    # D-stage: the enlarged batch advances one token; t2 = now + E_d(2, 1000 + 2000)
    rows = [dict(state=gen.RUNNING, prompt_len=900, gen=100, first_token_ns=0, class_id=1, req_id=9, output_len=102),
            dict(prompt_len=500, gen=0, first_token_ns=0, class_id=0, req_id=1, output_len=5),
            dict(prompt_len=2000, gen=0, first_token_ns=0, class_id=0, req_id=2, output_len=5)]
    wl = make_wl(rows, cls, replicas=[(gen.DECODE, 32768, 2)], now=[MS])
    oracle.step(wl, commit=True)
    t2 = MS + 8_000_000 + 2 * 100_000 + 20 * 3000
    t = wl.table
    assert list(t["state"]) == [gen.DONE, gen.QUEUED, gen.RUNNING]
    assert list(t["gen"]) == [101, 0, 1] and t["finish_ns"][0] == t2
    assert t["last_token_ns"][0] == t2 and t["last_token_ns"][2] == t2 and t["first_token_ns"][2] == 0
    assert wl.now[0] == t2 and wl.maturity[0] == t2
    # P-stage: the admitted batch completes at t1 = now + E_p(200); the instance does not decode
    rows = [dict(state=gen.RUNNING, prompt_len=4000, gen=3, first_token_ns=0, class_id=0, req_id=9, output_len=50),
            dict(prompt_len=100, class_id=1, req_id=1, output_len=1), dict(prompt_len=100, class_id=0, req_id=2, output_len=3)]
    wl = make_wl(rows, cls, replicas=[(gen.PREFILL, 32768, 0)], now=[MS])
    oracle.step(wl, commit=True)
    t1 = MS + 5_000_000 + 40_000 * 200 + 2 * 200 * 200
    t = wl.table
    assert list(t["state"]) == [gen.RUNNING, gen.DONE, gen.RUNNING] and list(t["gen"]) == [3, 0, 0]
    assert t["finish_ns"][1] == t1 and t["first_token_ns"][2] == t1 and t["last_token_ns"][2] == t1
    assert wl.now[0] == t1 and wl.maturity[0] == t1


def test_idle_replica_jumps_to_its_next_event():
    rows = [dict(prompt_len=10, arrival_ns=900 * MS, req_id=0), dict(prompt_len=10, arrival_ns=700 * MS, req_id=1),
            dict(prompt_len=10, arrival_ns=100 * MS, req_id=2, state=gen.DONE)]
    wl = make_wl(rows, C200, now=[500 * MS], maturity=[0])
    o = oracle.step(wl, commit=True)
    assert wl.now[0] == 700 * MS and o["adm_count"][0] == 0 and list(wl.table["state"]) == [0, 0, gen.DONE]
    wl = make_wl(rows, C200, now=[500 * MS], maturity=[600 * MS])
    oracle.step(wl, commit=True)
    assert wl.now[0] == 600 * MS and wl.maturity[0] == 600 * MS
    wl = make_wl(rows[2:], C200, now=[500 * MS], maturity=[0])       # nothing left to happen: the clock stays
    oracle.step(wl, commit=True)
    assert wl.now[0] == 500 * MS


def test_scaling_indicators_hand_worked():
    # two colocated instances, tick at 20 s, 10 s window, 16-token KV blocks (Sec. 3.3.3)
    S = 1000 * MS
    rows = [dict(replica_id=0, arrival_ns=5 * S, state=gen.DONE, finish_ns=12 * S, req_id=0),      # completed in the window
            dict(replica_id=1, arrival_ns=11 * S, state=gen.DONE, finish_ns=19 * S, req_id=1),     # arrived and completed in it
            dict(replica_id=0, arrival_ns=15 * S, state=gen.RUNNING, prompt_len=100, gen=28, req_id=2),
            dict(replica_id=1, arrival_ns=20 * S - 100 * MS, prompt_len=33, req_id=3),             # waits 100 ms of 200 ms
            dict(replica_id=1, arrival_ns=20 * S - 20 * MS, prompt_len=16, req_id=4),              # waits 20 ms of 200 ms
            dict(replica_id=0, arrival_ns=25 * S, prompt_len=500, req_id=5)]                       # not arrived yet
    wl = make_wl(rows, C200, replicas=[(gen.COLOCATED, 8192, 0)] * 2, now=[0, 0], maturity=[0, 0])
    o = oracle.scale_tick(wl, 20 * S, np.array([100, 100]), min_samples=2)
    assert list(o["counts"][0]) == [4, 2, 2, 32768 + 6553]        # 0.5 and floor(0.1 * 65536) in 16.16
    assert list(o["used_blocks"]) == [8, 3 + 1]                   # ceil(128/16); ceil(33/16) + ceil(16/16)
    assert list(o["decision"][0]) == [1, -1]                      # f1 = 2/4 < 0.7 (and f2 = 0.3 > 1/4): scale out
    assert np.all(o["counts"][1:] == 0) and np.all(o["decision"][1:] == [0, -1])
    # too few arrivals seen: f1 is suppressed, f2 alone decides (0.3 > 1/4 still scales out; 1/2 does not)
    assert list(oracle.scale_tick(wl, 20 * S, np.array([100, 100]), min_samples=5)["decision"][0]) == [1, -1]
    assert list(oracle.scale_tick(wl, 20 * S, np.array([100, 100]), min_samples=5, eps_wait=(1, 2))["decision"][0]) == [0, -1]
    # completions outpace arrivals and nobody waits: scale in, removing the emptier instance
    for r in rows[3:5]:
        r.update(state=gen.DONE, finish_ns=20 * S - 1)
    wl = make_wl(rows, C200, replicas=[(gen.COLOCATED, 8192, 0)] * 2, now=[0, 0], maturity=[0, 0])
    o = oracle.scale_tick(wl, 20 * S, np.array([100, 100]), min_samples=2)
    assert list(o["counts"][0]) == [4, 4, 0, 0] and list(o["used_blocks"]) == [8, 0]
    assert list(o["decision"][0]) == [0, -1]                      # f1 = 1.0: between the thresholds, hold
    rows[2].update(state=gen.DONE, finish_ns=18 * S)
    rows.append(dict(replica_id=0, arrival_ns=2 * S, state=gen.DONE, finish_ns=17 * S, req_id=6))
    rows.append(dict(replica_id=0, arrival_ns=3 * S, state=gen.RUNNING, prompt_len=40, gen=0, req_id=7))
    wl = make_wl(rows, C200, replicas=[(gen.COLOCATED, 8192, 0)] * 2, now=[0, 0], maturity=[0, 0])
    o = oracle.scale_tick(wl, 20 * S, np.array([100, 100]), min_samples=2)
    assert list(o["counts"][0]) == [4, 6, 0, 0] and list(o["decision"][0]) == [-1, 1]     # f1 = 1.5 > 1.1; instance 1 holds 0 blocks
    o = oracle.scale_tick(wl, 20 * S, np.array([100, 0]), min_samples=2)
    assert list(o["decision"][0]) == [0, -1]                      # a single active instance is never removed
    o = oracle.scale_tick(wl, 20 * S, np.array([1, 100]), min_samples=2)
    assert list(o["decision"][0]) == [-1, 1]
    o = oracle.scale_tick(wl, 20 * S, np.array([1000, 100]), min_samples=2)     # 3/1000 vs 0/100: still instance 1
    assert list(o["used_blocks"]) == [3, 0] and list(o["decision"][0]) == [-1, 1]


# ---- dispatching over the shared global queue -------------------------------------------------------
def _dispatch_hand_case():
    now = 1000 * MS
    classes = [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1)]
    rows = [dict(state=1, replica_id=0, prompt_len=800, gen=0, output_len=500, arrival_ns=0, first_token_ns=now - 30 * MS)
            for _ in range(80)]
    rows += [dict(replica_id=-1, class_id=0, prompt_len=1000, arrival_ns=now - 10 * MS),    # q1  row 80
             dict(replica_id=-1, class_id=0, prompt_len=1144, arrival_ns=now - 50 * MS),    # q2  row 81
             dict(replica_id=-1, class_id=1, prompt_len=281, arrival_ns=now - 900 * MS),    # q3  row 82
             dict(replica_id=-1, class_id=0, prompt_len=16, arrival_ns=now - 1 * MS),       # q4  row 83
             dict(replica_id=-1, class_id=1, prompt_len=2000, arrival_ns=now - 100 * MS),   # q5  row 84
             dict(replica_id=-1, class_id=0, prompt_len=16, arrival_ns=now + 1)]            # not arrived yet
    wl = make_wl(rows, classes, replicas=[(gen.COLOCATED, 8192, 0)] * 3, now=[now] * 3,
                 maturity=[now - 5, now - 10, now + 1])
    return wl, now


def test_dispatch_global_queue_hand_worked():
    wl, now = _dispatch_hand_case()
    o = oracle.dispatch(wl, now)
    assert o["status"] == 0
    assert o["n_queue"][0] == 5 and list(o["queue_order"][:5]) == [81, 80, 83, 82, 84] and o["queue_order"][5] == -1
    assert o["slack"][80] == PINS["slack_queued"] and o["slack"][81] == PINS["disp_slack_q2"]
    assert o["slack"][82] == PINS["disp_slack_q3"] and o["slack"][83] == PINS["disp_slack_q4"]
    assert o["slack"][84] == PINS["disp_slack_q5"] and o["slack"][85] == 0 and o["slack"][0] == 0
    assert o["n_mature"][0] == 2 and list(o["inst_order"]) == [1, 0, -1]
    assert list(o["budget"]) == [PINS["nsafe_busy"], PINS["nsafe_idle"], 0]
    assert list(o["n_run"]) == [80, 0, 0] and o["e_d"][0] == PINS["Ed_80_64000"] and o["e_d"][1] == 0
    assert list(o["assign"][80:86]) == [1, 1, 0, 0, -1, -1] and np.all(o["assign"][:80] == -1)
    assert list(o["adm_cost"]) == [297, 2144, 0] and list(o["adm_count"]) == [2, 2, 0]
    assert o["maturity_next"][1] - now == PINS["disp_mat1_delta"]
    assert o["maturity_next"][0] - now == PINS["disp_mat0_delta"]
    assert o["maturity_next"][2] == now + 1


def test_dispatch_batch_cap_stops_a_run_and_oversize_prompts_leave_the_queue():
    wl, now = _dispatch_hand_case()
    wl.replicas[1, 2] = 1                      # the idle instance may hold one request
    wl.table["prompt_len"][84] = 9000          # longer than every token cap: can never be served
    o = oracle.dispatch(wl, now)
    assert o["n_queue"][0] == 4 and list(o["queue_order"][:4]) == [81, 80, 83, 82]
    # instance 1 takes q2 and is full; instance 0 (budget 1281) takes q1 + q4 = 1016, q3 would make 1297
    assert list(o["assign"][80:86]) == [0, 1, -1, 0, -1, -1]
    assert list(o["adm_cost"]) == [1016, 1144, 0] and list(o["adm_count"]) == [2, 1, 0]


def test_dispatch_entry_that_fits_nowhere_is_passed_over():
    wl, now = _dispatch_hand_case()
    wl.table["prompt_len"][80] = 3000
    o = oracle.dispatch(wl, now)
    assert o["slack"][80] == PINS["disp_slack_q1_long"]
    assert list(o["queue_order"][:5]) == [80, 81, 83, 82, 84]
    assert list(o["assign"][80:86]) == [-1, 1, 1, 1, -1, -1]
    assert list(o["adm_cost"]) == [0, 1441, 0] and list(o["adm_count"]) == [0, 3, 0]
    assert o["maturity_next"][1] - now == PINS["disp_mat1_delta_long"] and o["maturity_next"][0] == now - 5


# ---- priority-based SLO mapping -------------------------------------------------------------------------
def _slo_hand_case():
    win = {"prio": np.array([0, 1, 0, 2, 1, 2]), "ttft": np.array([100, 300, 150, 900, 250, 700]) * MS,
           "tpot": np.array([20, 40, 25, 80, 35, 60]) * MS, "queue": np.array([10, 50, 30, 400, 20, 200]) * MS}
    bounds = {"ttft_min": np.array([150, 200, 700]) * MS, "ttft_max": np.array([200, 1000, 5000]) * MS,
              "ttft_min_relaxed": np.array([50, 100, 200]) * MS, "tpot_min": np.array([30, 30, 50]) * MS,
              "tpot_max": np.array([30, 50, 100]) * MS, "tpot_min_relaxed": np.array([10, 20, 30]) * MS}
    return win, bounds, np.array([10, 30, 100]) * MS, np.array([1, 2, 1, 0])


def test_slo_mapping_hand_worked():
    win, bounds, last, new = _slo_hand_case()
    o = oracle.slo_map(3, win, bounds, last, np.array([0, 3, 0]), new)
    assert o["status"] == 0
    assert list(o["ttft_slo"]) == [PINS["slo_req0_ttft_ms"] * MS, PINS["slo_req1_ttft_ms_contended"] * MS,
                                   PINS["slo_req2_ttft_ms"] * MS, PINS["slo_req3_ttft_ms"] * MS]
    assert list(o["tpot_slo"]) == [40 * MS, 80 * MS, 40 * MS, 20 * MS]
    assert list(o["last_queue"]) == [10 * MS, 50 * MS, 400 * MS]
    o = oracle.slo_map(3, win, bounds, last, np.array([0, 0, 0]), new)
    assert o["ttft_slo"][1] == PINS["slo_req1_ttft_ms_free"] * MS
    # strict bounds when the highest priority is pending: p=1 TPOT 40 stays, p=2 TTFT 600 -> 700; p=0 never has a higher one
    o = oracle.slo_map(3, win, bounds, last, np.array([5, 0, 0]), new)
    assert list(o["ttft_slo"]) == [280 * MS, 700 * MS, 300 * MS, 100 * MS] and o["tpot_slo"][3] == 20 * MS
    # an empty window: the loosest targets of each range; last_queue untouched
    empty = {k: v[:0] for k, v in win.items()}
    o = oracle.slo_map(3, empty, bounds, last, np.array([0, 0, 0]), new)
    assert list(o["ttft_slo"]) == [1000 * MS, 5000 * MS, 1000 * MS, 200 * MS] and list(o["last_queue"]) == list(last)
    # a priority outside [0, N): flagged, no targets
    o = oracle.slo_map(3, win, bounds, last, np.array([0, 0, 0]), np.array([7, 0]))
    assert o["status"] == 2 and o["ttft_slo"][0] == 0 and o["ttft_slo"][1] == 100 * MS


def test_slo_mapping_quantiles_against_numpy():
    # with one priority level the index is floor(C/2): the upper median of the window; ranges wide open
    rng = np.random.default_rng(3)
    for w in (1, 2, 7, 100, 1001):
        win = {"prio": np.zeros(w, np.int64), "ttft": rng.integers(1, 10**9, w), "tpot": rng.integers(1, 10**8, w),
               "queue": np.zeros(w, np.int64)}
        big = np.array([1 << 60])
        bounds = {"ttft_min": -big, "ttft_max": big, "ttft_min_relaxed": -big, "tpot_min": -big, "tpot_max": big,
                  "tpot_min_relaxed": -big}
        o = oracle.slo_map(1, win, bounds, np.array([0]), np.array([0]), np.array([0]))
        assert o["ttft_slo"][0] == np.sort(win["ttft"])[w // 2] and o["tpot_slo"][0] == np.sort(win["tpot"])[w // 2]


# ---- hand-off between the stages of the disaggregated mode ----------------------------------------------
def test_pd_handoff_hand_worked():
    cls = [(200 * MS, 30 * MS, 0)]
    rows = [dict(replica_id=0, prompt_len=1000, output_len=3, arrival_ns=0),
            dict(replica_id=0, prompt_len=64, output_len=1, arrival_ns=0)]          # finishes at its first token
    wl = make_wl(rows, cls, replicas=[(gen.PREFILL, 32768, 0), (gen.DECODE, 32768, 8)], now=[0, 0], maturity=[0, 0])
    pair = np.array([1, -1])
    o = oracle.step(wl, commit=True)
    assert o["budget"][0] == PINS["nsafe_idle"] and list(o["admit"]) == [1, 1]
    ft = 5_000_000 + 40_000 * 1064 + 2 * 1064 * 1064          # both prompts form one prefill batch of 1064 tokens
    assert wl.table["first_token_ns"][0] == ft and list(wl.table["state"]) == [gen.RUNNING, gen.DONE]
    # the single-request figures of the pin file: the batch is request A alone
    wl = make_wl(rows[:1], cls, replicas=[(gen.PREFILL, 32768, 0), (gen.DECODE, 32768, 8)], now=[0, 0], maturity=[0, 0])
    oracle.step(wl, commit=True)
    assert wl.table["first_token_ns"][0] == PINS["pd_first_token"] and wl.now[0] == PINS["pd_first_token"]
    r = oracle.pd_migrate(wl, pair, 1_000_000, 1000)
    assert r == {"status": 0, "moved": 0} and wl.table["replica_id"][0] == 0 and wl.table["state"][0] == gen.RUNNING
    assert wl.now[1] == PINS["pd_ready"] and wl.now[0] == PINS["pd_first_token"]
    r = oracle.pd_migrate(wl, pair, 1_000_000, 1000)
    assert r["moved"] == 1 and wl.table["replica_id"][0] == 1 and wl.table["state"][0] == gen.QUEUED
    o = oracle.step(wl, commit=True)
    assert o["budget"][1] == 22_000_000 and o["admit"][0] == 1 and o["adm_cost"][1] == 120_000
    assert wl.now[1] == PINS["pd_d_iteration_end"] and wl.table["gen"][0] == 1 and wl.table["state"][0] == gen.RUNNING
    assert wl.table["first_token_ns"][0] == PINS["pd_first_token"] and wl.table["last_token_ns"][0] == PINS["pd_d_iteration_end"]
    # a busy D instance is not woken, a request whose transfer is still under way stays on the P instance
    rows = [dict(replica_id=0, state=gen.RUNNING, prompt_len=1000, output_len=9, first_token_ns=100 * MS),
            dict(replica_id=1, state=gen.RUNNING, prompt_len=10, gen=2, output_len=99, first_token_ns=0),
            dict(replica_id=0, state=gen.RUNNING, prompt_len=0, output_len=9, first_token_ns=9 * MS)]
    wl = make_wl(rows, cls, replicas=[(gen.PREFILL, 32768, 0), (gen.DECODE, 32768, 8)], now=[200 * MS, 10 * MS], maturity=[0, 0])
    r = oracle.pd_migrate(wl, pair, 1_000_000, 1000)
    assert r["moved"] == 1 and list(wl.table["replica_id"]) == [0, 1, 1] and list(wl.now) == [200 * MS, 10 * MS]
    # a partner that is not a D instance is an error of the data: flagged, nothing moves
    r = oracle.pd_migrate(wl, np.array([0, -1]), 0, 0)
    assert r["status"] == 1 and r["moved"] == 0


# ---- SLO attainment (Eq. 2) -------------------------------------------------------------------------------
def _attainment_hand_case():
    cls = [(200 * MS, 30 * MS, 0), (1000 * MS, 0, 1)]
    rows = [dict(state=gen.DONE, class_id=0, prompt_len=1000, output_len=101, gen=100, arrival_ns=0,
                 first_token_ns=PINS["sim1_ttft"], last_token_ns=PINS["sim1_finish"], finish_ns=PINS["sim1_finish"]),
            dict(state=gen.DONE, class_id=0, output_len=11, gen=10, arrival_ns=100 * MS, first_token_ns=350 * MS,
                 last_token_ns=850 * MS, finish_ns=850 * MS),
            dict(state=gen.RUNNING, class_id=0, output_len=50, gen=3, arrival_ns=5 * MS, first_token_ns=15 * MS, last_token_ns=99 * MS),
            dict(state=gen.REJECTED, class_id=1, prompt_len=100000, arrival_ns=0),
            dict(state=gen.DONE, class_id=1, output_len=1, arrival_ns=MS, first_token_ns=1000 * MS, last_token_ns=1000 * MS,
                 finish_ns=1000 * MS),
            dict(state=gen.QUEUED, class_id=1, arrival_ns=7 * MS)]
    return make_wl(rows, cls, replicas=[(gen.COLOCATED, 8192, 0)])


def test_attainment_hand_worked():
    o = oracle.attainment(_attainment_hand_case())
    c = o["counts"]
    assert o["status"] == 0
    assert list(c[0]) == [3, 2, 1, 0, PINS["att_A_ttft_sum"], PINS["att_A_e2e_sum"]]
    assert list(c[1]) == [3, 1, 1, 1, PINS["att_B_ttft_sum"], 999 * MS]
    assert list(c[2]) == [6, 3, 2, 1, PINS["att_A_ttft_sum"] + PINS["att_B_ttft_sum"], PINS["att_A_e2e_sum"] + 999 * MS]


def test_attainment_agrees_with_the_simulator():
    # the simulator reports finished / attained / rejected per trace; the table it leaves gives the same by Eq. 2
    wl = gen.random_traces(3, 5, 30, 60, 400)
    sim = oracle.sim(wl)
    c = oracle.attainment(wl)["counts"][-1]
    assert c[1] == sim["finished"].sum() and c[2] == sim["attained"].sum() and c[3] == sim["rejected"].sum()


def test_dispatch_serves_the_p_stage():
    # the hand-worked case with instance 0 as a P-stage instance: its 80 resident requests do not decode there, so
    # it has the budget of an empty instance (2144), no E_d, and matures when its prefill batch ends:
    # E_p(297) = 17056418.
    wl, now = _dispatch_hand_case()
    wl.replicas[0, 0] = gen.PREFILL
    wl.replicas[2, 0] = gen.DECODE
    wl.maturity[2] = now - 100
    o = oracle.dispatch(wl, now)
    assert list(o["inst_order"]) == [1, 0, 2] and list(o["n_mature"]) == [2, 1]
    assert list(o["budget"][:2]) == [2144, 2144] and list(o["e_d"]) == [0, 0, 0] and list(o["n_run"]) == [80, 0, 0]
    assert list(o["assign"][80:86]) == [1, 1, 0, 0, -1, -1] and list(o["adm_cost"][:2]) == [297, 2144]
    assert o["maturity_next"][0] - now == 17_056_418
    # The D stage in the same call (Sec. 3.3.1, "D-stage Migrator"): the 80 residents got their first token 30 ms ago
    # and are the queue of prefilled requests; TPOT 30 ms, 800 tokens of context each.  Slack = (now - 30 ms) + 30 ms
    # - now - E_d(1, 800) = -(8000000 + 100000 + 16000); all equal, so they queue by request id behind the 5
    # entries of the global queue.  The idle D instance 2 takes the strictest TPOT of that queue: budget = 30 ms -
    # E_d(0, 0) = 22000000 ns; a request costs d1 + d2 * 800 = 116000 ns, all 80 fit (9280000); its maturity is
    # the end of the first decode iteration of the 80: E_d(80, 64000).
    assert list(o["n_queue"]) == [5, 80] and list(o["queue_order"][5:85]) == list(range(80)) and o["queue_order"][85] == -1
    assert np.all(o["slack"][:80] == -8_116_000)
    assert o["budget"][2] == 22_000_000 and o["adm_cost"][2] == 80 * 116_000 and o["adm_count"][2] == 80
    assert np.all(o["assign"][:80] == 2)
    assert o["maturity_next"][2] - now == PINS["Ed_80_64000"] == 17_280_000


def test_migrator_selects_the_d_instance_hand_worked():
    # Sec. 3.3.1, "Disaggregated Mode": the four steps once more for the D stage.  E_d(n, kv) = 8 ms + 2 ms n + 0.2 us kv.
    # Queue of prefilled requests (first token produced): slack = first_token + TPOT - now - E_d(1, kv)
    #   A (class 1, 50 ms, 70000 tokens) 30 ms - 24 ms =  6 ms   cost 2 ms + 14 ms = 16 ms
    #   B (class 0, 30 ms,  5000 tokens)  5 ms - 11 ms = -6 ms   cost 2 ms +  1 ms =  3 ms
    #   C (class 0, 30 ms, 40000 tokens) 29 ms - 18 ms = 11 ms   cost 2 ms +  8 ms = 10 ms
    # order: priority 0 first (B, C), then A.  Instance 2 matured first (10 ms ago): two requests in flight with
    # 20200 tokens, E_d = 8 + 4 + 4.04 = 16.04 ms, strictest TPOT in flight 50 ms: budget 33.96 ms; its batch cap of 3
    # leaves room for one request: it takes B and stops at C.  Instance 1 is idle: strictest TPOT of the queue as
    # the call began (30 ms) minus E_d(0, 0) = 22 ms; it takes C (10 ms), A (16 ms more) does not fit and waits.
    wl, now = migrator_hand_case()
    o = oracle.dispatch(wl, now)
    assert o["status"] == 0
    assert list(o["n_queue"]) == [0, 3] and list(o["queue_order"][:4]) == [3, 4, 2, -1]
    assert o["slack"][2] == PINS["mig_slack_A"] and o["slack"][3] == PINS["mig_slack_B"] and o["slack"][4] == PINS["mig_slack_C"]
    assert o["slack"][5] == 0 and o["slack"][0] == 0
    assert list(o["n_mature"]) == [0, 2] and list(o["inst_order"]) == [2, 1, -1]
    assert list(o["n_run"]) == [4, 0, 2] and list(o["e_d"]) == [0, 0, PINS["mig_ed_inst2"]]
    assert list(o["budget"]) == [0, PINS["mig_budget_inst1"], PINS["mig_budget_inst2"]]
    assert list(o["assign"]) == [-1, -1, -1, 2, 1, -1]
    assert list(o["adm_cost"]) == [0, PINS["mig_cost_C"], PINS["mig_cost_B"]] and list(o["adm_count"]) == [0, 1, 1]
    assert o["maturity_next"][2] - now == PINS["mig_mat_inst2"] and o["maturity_next"][1] - now == PINS["mig_mat_inst1"]
    assert o["maturity_next"][0] == now + 1
    # a D instance before its maturity takes no part; the other then takes its share: room for B only stands, so
    # with instance 2 protected instance 1 takes B and C (13 ms) and A (29 ms) still does not fit
    wl.maturity[2] = now + 1
    o = oracle.dispatch(wl, now)
    assert list(o["n_mature"]) == [0, 1] and list(o["inst_order"]) == [1, -1, -1] and o["budget"][2] == 0
    assert list(o["assign"]) == [-1, -1, -1, 1, 1, -1] and o["adm_cost"][1] == 13_000_000
    assert o["maturity_next"][1] - now == 8_000_000 + 2 * 2_000_000 + 200 * 45_000 and o["maturity_next"][2] == now + 1
    # binding: a dispatched prefilled request stays in flight, now on its D instance
    wl.maturity[2] = now - 10 * MS
    o = oracle.dispatch(wl, now)
    oracle.dispatch_bind(wl, now, o)
    assert list(wl.table["replica_id"]) == [2, 2, 0, 2, 1, 0] and list(wl.table["state"]) == [1] * 6


def test_scale_apply_hand_worked():
    S = 1_000_000_000
    rows = [dict(replica_id=0, prompt_len=1, output_len=1)]
    wl = make_wl(rows, [(200 * MS, 30 * MS, 0)], replicas=[(gen.COLOCATED, 4096, 0)] * 4 + [(gen.PREFILL, 4096, 0)],
                 now=[0] * 5, maturity=[0] * 5)
    f = gen.new_fleet([100] * 5, [0, 1, 4])
    NEVER = gen.T_NEVER
    hold = [0, -1]

    def tick(t, dec0, used, dec1=hold):
        return oracle.scale_apply(wl, t * S, np.array([dec0, dec1, hold]), np.array(used), [2 * S, 5 * S, 7 * S], f)

    cost = tick(10, [1, -1], [50, 20, 0, 0, 10])
    assert list(f["inst_state"]) == [2, 2, 1, 0, 2] and f["ready"][2] == 12 * S and list(cost) == [20 * S, 10 * S, 0]
    assert list(f["total_blocks"]) == [100, 100, 0, 0, 100] and list(f["due"]) == [0, 0, NEVER, NEVER, 0]
    cost = tick(11, [1, -1], [50, 20, 0, 0, 10])
    assert list(f["inst_state"]) == [2, 2, 1, 0, 2] and cost[0] == 23 * S
    wl.maturity[0] = 14 * S                                              # instance 0 is busy until 14 s
    cost = tick(13, hold, [50, 20, 0, 0, 10], dec1=[1, -1])
    assert list(f["inst_state"]) == [2, 2, 2, 0, 2] and f["total_blocks"][2] == 100
    assert list(f["due"]) == [14 * S, 0, 12 * S, NEVER, 0] and list(wl.now) == [0, 0, 12 * S, 0, 0] and wl.maturity[2] == 12 * S
    assert cost[0] == PINS["fleet_cost_s_t13"] * S and cost[1] == 13 * S
    cost = tick(20, [-1, 1], [50, 20, 5, 0, 10])
    assert list(f["inst_state"]) == [2, 3, 2, 0, 2] and f["due"][1] == NEVER and f["total_blocks"][1] == 0 and cost[0] == 50 * S
    cost = tick(21, hold, [50, 20, 5, 0, 10])
    assert f["inst_state"][1] == 3 and cost[0] == 53 * S
    wl.maturity[1] = 25 * S
    cost = tick(22, [1, -1], [50, 7, 5, 0, 10])
    assert list(f["inst_state"]) == [2, 2, 2, 0, 2] and f["due"][1] == 25 * S and cost[0] == PINS["fleet_cost_s_t22"] * S
    cost = tick(30, [-1, 0], [9, 7, 5, 0, 10])
    assert f["inst_state"][0] == 3 and cost[0] == 80 * S
    cost = tick(31, hold, [0, 7, 5, 0, 10])
    assert f["inst_state"][0] == 0 and f["due"][0] == NEVER and cost[0] == PINS["fleet_cost_s_t31"] * S
    cost = tick(40, [1, -1], [0, 7, 5, 0, 10])
    assert list(f["inst_state"]) == [1, 2, 2, 0, 2] and f["ready"][0] == 42 * S and f["billed"][0] == 31 * S and cost[0] == 101 * S
    cost = tick(41, [-1, 0], [0, 7, 5, 0, 10], dec1=[-1, 0])          # the second names an instance of another pool
    assert list(f["inst_state"]) == [1, 2, 2, 0, 2]
    assert cost[0] == PINS["fleet_cost_s_t41"] * S and cost[1] == PINS["fleet_prefill_cost_s_t41"] * S and cost[2] == 0
    assert list(f["billed"]) == [32 * S, 41 * S, 31 * S, 0, 41 * S]
    # an instance whose clock is already past its ready time keeps it
    wl.now[0] = 50 * S; wl.maturity[0] = 55 * S
    tick(43, hold, [0, 7, 5, 0, 10])
    assert f["inst_state"][0] == 2 and wl.now[0] == 50 * S and f["due"][0] == 55 * S


def test_horizon_gate_and_binding():
    # a replica whose clock is past the horizon reports its decisions and changes nothing
    rows = [dict(replica_id=0, prompt_len=1000, output_len=3, arrival_ns=0), dict(replica_id=1, prompt_len=1000, output_len=3, arrival_ns=0)]
    wl = make_wl(rows, [(200 * MS, 30 * MS, 0)], replicas=[(gen.COLOCATED, 32768, 0)] * 2, now=[10 * MS, 30 * MS], maturity=[0, 0])
    wl.meta["horizon"] = 20 * MS
    o = oracle.step(wl, commit=True)
    assert list(o["admit"]) == [1, 1]
    assert list(wl.table["state"]) == [gen.RUNNING, gen.QUEUED] and list(wl.now) == [10 * MS + PINS["pd_first_token"], 30 * MS]
    assert wl.table["first_token_ns"][0] == 10 * MS + PINS["pd_first_token"] and wl.maturity[1] == 0
    wl.meta["horizon"] = 30 * MS                      # a clock exactly at the horizon still acts
    oracle.step(wl, commit=True)
    assert wl.table["state"][1] == gen.RUNNING and wl.now[1] == 30 * MS + PINS["pd_first_token"]
    # binding: the request moves to its instance, whose clock cannot stay behind the time of the call
    wl = make_wl([dict(replica_id=-1, prompt_len=10, output_len=3), dict(replica_id=-1, prompt_len=10, output_len=3)],
                 [(200 * MS, 30 * MS, 0)], replicas=[(gen.COLOCATED, 32768, 0)] * 3, now=[5, 500, 7], maturity=[0, 0, 0])
    oracle.dispatch_bind(wl, 100, dict(assign=np.array([1, -1], np.int32), adm_count=np.array([1, 1, 0], np.int32)))
    assert list(wl.table["replica_id"]) == [1, -1] and list(wl.now) == [100, 500, 7]


def test_unbound_queued_rows_are_the_global_queue_not_an_error():
    rows = [dict(prompt_len=100, req_id=0, output_len=5), dict(prompt_len=100, req_id=1, replica_id=-1, output_len=5),
            dict(prompt_len=100, req_id=2, replica_id=-1, output_len=5), dict(prompt_len=100, req_id=3, output_len=5)]
    wl = make_wl(rows, C200, now=[MS])
    o = oracle.step(wl, commit=True)
    assert o["status"] == 0 and list(o["seg_off"]) == [0, 2] and list(o["order"]) == [0, 3, 1, 2]
    assert list(o["admit"]) == [1, 0, 0, 1] and list(wl.table["state"]) == [gen.RUNNING, gen.QUEUED, gen.QUEUED, gen.RUNNING]
    # the same id on a request that is running somewhere is bad data; so is any other id out of range
    wl.table["replica_id"][0] = -1
    assert oracle.step(wl)["status"] == 1
    wl.table["replica_id"][0] = 0; wl.table["replica_id"][1] = -2
    assert oracle.step(wl)["status"] == 1
    # the hand-off between the stages leaves the global queue alone too
    wl = make_wl(rows[:2], [(200 * MS, 30 * MS, 0)], replicas=[(gen.PREFILL, 32768, 0), (gen.DECODE, 32768, 8)], now=[0, 0], maturity=[0, 0])
    r = oracle.pd_migrate(wl, np.array([1, -1]), 1_000_000, 1000)
    assert r == {"status": 0, "moved": 0}
