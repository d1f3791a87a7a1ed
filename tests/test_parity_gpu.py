"""Parity of the CUDA path with the oracle, bit for bit, through the C ABI (needs a GPU)."""
import numpy as np
import pytest
import torch

import gen
import oracle
from helpers import MS, SEC, make_wl
from gpu_helpers import assert_dispatch_parity, assert_step_parity, assert_sim_parity, make_sched, run_sim_gpu

pytestmark = pytest.mark.gpu
MODES3 = (gen.COLOCATED, gen.PREFILL, gen.DECODE)


# ---- the five configurations ---------------------------------------------------------------------
def test_config1_step_and_simulation():
    wl = gen.config1()
    assert_step_parity(wl)
    assert_step_parity(wl, steps=5, commit=True)
    assert_sim_parity(wl)


@pytest.mark.parametrize("mode", [gen.BUDGET_SAFE, gen.BUDGET_CAP_ONLY])
@pytest.mark.parametrize("inflight", [0.6, 0.02])
def test_config2_full(mode, inflight):
    g = assert_step_parity(gen.config2(inflight=inflight, budget_mode=mode))
    if mode == gen.BUDGET_CAP_ONLY or inflight < 0.1:
        assert g["adm_count"].sum() > 0


def test_config2_committed_steps():
    assert_step_parity(gen.config2(R=16, rows_per=4096, inflight=0.02), steps=4, commit=True)


def test_config3_full():
    g = assert_step_parity(gen.config3(), optional=False)
    assert g["adm_count"][:128].sum() > 0 and g["adm_count"][128:].sum() > 0


def test_config3_small_committed():
    assert_step_parity(gen.config3(R=8, rows_per=3000), steps=4, commit=True)


def test_config4_full_ten_committed_steps():
    wl = gen.config4()
    g = assert_step_parity(wl, steps=wl.steps, commit=True, optional=False)


def test_config4_small_all_outputs():
    assert_step_parity(gen.config4(R=32, n=50_001, steps=3), steps=3, commit=True)


def test_config5_subset_of_traces():
    wl = gen.config5(traces=6)
    assert_sim_parity(wl)


def test_config5_full_batch_sampled_traces():
    # the whole 4096-trace batch in one call (the launch the benchmark times); 256 traces spread evenly
    # over the batch (every 16th) are compared with the oracle, which runs as a pool of single-threaded
    # worker processes over disjoint trace ranges; the rest through properties that hold for every trace
    import multiprocessing as mp
    import os
    from gpu_helpers import SIM_KEYS, STATE_COLS
    from helpers import oracle_sim_config5_range
    wl = gen.config5()
    T = wl.trace_off.shape[0] - 1
    picked = list(range(0, T, 16))
    workers = max(1, min(len(picked), (os.cpu_count() or 1) - 1, 64))
    # the pool is started with `spawn`: this process may hold a CUDA context already, and a forked child of it hangs
    with mp.get_context("spawn").Pool(workers) as pool:
        pending = pool.map_async(oracle_sim_config5_range, [(j, 1, wl.sim_iters) for j in picked], chunksize=1)
        res, cols, st = run_sim_gpu(wl)
        done = pending.get(timeout=900)
    print(f"oracle: {len(picked)} traces on {workers} worker processes of {os.cpu_count()} cores")
    assert st == 0
    for first, count, c, ccols in done:
        a, b = wl.trace_off[first], wl.trace_off[first + count]
        for ko, kg in SIM_KEYS.items():
            assert np.array_equal(res[kg][first:first + count], c[ko][:count]), f"trace {first}: {kg}"
        for k in STATE_COLS:
            assert np.array_equal(cols[k][a:b], ccols[k]), f"trace {first}: column {k}"
        assert c["status"] == 0
    assert np.all(res["iters_executed"] <= wl.sim_iters) and np.all(res["iters_executed"] > 0)
    assert np.all(res["attained"] <= res["finished"]) and np.all(res["finished"] + res["rejected"] <= 2048)
    assert np.all(res["ttft_p50_ns"] <= res["ttft_p99_ns"]) and np.all(res["tpot_p50_ns"] <= res["tpot_p99_ns"])


# ---- random and adversarial step cases -----------------------------------------------------------
@pytest.mark.parametrize("seed", range(16))
def test_random_tables(seed):
    wl = gen.random_table(seed, 1000 + 997 * seed, 1 + (seed * 7) % 23, modes=MODES3, tie_heavy=seed % 3 == 0,
                          batch_cap=(0, 7)[seed % 2], weight_max=(0, 16)[seed % 4 == 1],
                          budget_mode=(gen.BUDGET_SAFE, gen.BUDGET_CAP_ONLY)[seed % 5 == 2], grouped=seed % 4 == 3)
    assert_step_parity(wl, steps=3, commit=True)
    assert_step_parity(wl)


@pytest.mark.parametrize("n", [0, 1, 2, 3, 5, 255, 257, 2047, 2048, 2049, 4099])
def test_ragged_sizes_single_replica(n):
    wl = gen.random_table(100 + n, n, 1, modes=(gen.COLOCATED,))
    assert_step_parity(wl, steps=2, commit=True)


@pytest.mark.parametrize("seed", [0, 3, 5, 9])
def test_separate_front_end_kernels(seed):
    # the front end as separate kernels (what tables with more tiles than resident blocks use) gives
    # the same results as the fused cooperative kernel that the other tests run
    wl = gen.random_table(seed, 1000 + 997 * seed, 1 + (seed * 7) % 23, modes=MODES3, tie_heavy=seed % 3 == 0,
                          batch_cap=(0, 7)[seed % 2], weight_max=(0, 16)[seed % 4 == 1], grouped=seed % 4 == 3)
    sched = make_sched(wl)
    sched.set_fused_front(False)
    assert_step_parity(wl, steps=3, commit=True, sched=sched)
    sched.set_fused_front(True)
    assert_step_parity(wl, steps=2, commit=True, sched=sched)
    sched.close()
    wl = gen.config4(R=64, n=200_000, steps=3)
    sched = make_sched(wl)
    sched.set_fused_front(False)
    assert_step_parity(wl, steps=3, commit=True, optional=False, sched=sched)
    sched.close()


def test_medium_and_oversize_segments():
    # 2048 < rows <= 16384: medium path; > 16384: global-sort path
    assert_step_parity(gen.random_table(7, 9000, 1, tie_heavy=True), steps=2, commit=True)
    assert_step_parity(gen.random_table(8, 16384 + 16385 + 100, 3, grouped=True, modes=MODES3), steps=2, commit=True)
    wl = gen.random_table(9, 40_001, 1)
    assert_step_parity(wl, steps=2, commit=True)
    wl = gen.random_table(10, 70_000, 2, tie_heavy=True, modes=(gen.DECODE, gen.COLOCATED))
    assert_step_parity(wl)


def test_many_replicas_atomic_regroup_and_natural_ids():
    # more replicas than fit the shared-memory counters: global-counter regroup
    wl = gen.random_table(40, 30_000, 9000, modes=MODES3)
    assert_step_parity(wl, steps=2, commit=True)
    # request ids rising with the row index, interleaved replicas: the order of equal keys comes from positions
    for R, n in ((300, 40_000), (3, 5000), (64, 20_000)):
        wl = gen.random_table(41 + R, n, R, modes=MODES3, permute_ids=False, tie_heavy=R == 64)
        assert_step_parity(wl, steps=3, commit=True)
    # one id out of order anywhere must switch every replica to the general order
    wl = gen.random_table(44, 20_000, 50, permute_ids=False)
    wl.table["req_id"][12_345] = -5
    assert_step_parity(wl, steps=2, commit=True)
    wl = gen.random_table(45, 20_001, 50, permute_ids=False, grouped=True)
    wl.table["req_id"][20_000] = 7
    assert_step_parity(wl)


@pytest.mark.parametrize("R", [4095, 4096])
def test_replica_count_at_the_counter_limit(R):
    # 4095 replicas still use the tile histograms, 4096 the global counters
    for ids in (True, False):
        wl = gen.random_table(60 + R % 7, 60_000, R, modes=MODES3, permute_ids=ids)
        assert_step_parity(wl, steps=2, commit=True)


@pytest.mark.parametrize("n", [1023, 1024, 1025, 296 * 1024 - 1, 296 * 1024, 296 * 1024 + 5])
def test_sizes_at_tile_boundaries(n):
    wl = gen.config4(seed=n % 100, R=64, n=n, steps=2)
    assert_step_parity(wl, steps=2, commit=True, optional=n < 5000)


def test_scheduler_on_its_own_stream():
    import paper_2508_15919_b200 as hfx
    wl = gen.config4(seed=77, R=32, n=30_000, steps=3)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        sched = hfx.Scheduler(wl.model, wl.classes, wl.replicas, wl.n_rows, budget_mode=wl.budget_mode,
                              weight_max=wl.weight_max, stream=st)
        assert_step_parity(wl, steps=3, commit=True, sched=sched)
        sched.close()
    st.synchronize()


def test_two_schedulers_interleaved():
    a = gen.config4(seed=78, R=16, n=20_000, steps=2)
    b = gen.random_table(79, 5000, 7, modes=MODES3)
    sa, sb = make_sched(a), make_sched(b)
    assert_step_parity(a, steps=1, commit=True, sched=sa)
    assert_step_parity(b, steps=2, commit=True, sched=sb)
    assert_step_parity(a, steps=2, commit=True, sched=sa)
    sa.close(); sb.close()


def test_empty_replicas_and_all_inactive():
    wl = gen.random_table(11, 500, 40)
    wl.table["replica_id"][:] = wl.table["replica_id"] % 3 * 13        # most replicas have no rows
    assert_step_parity(wl, steps=2, commit=True)
    wl = gen.random_table(12, 700, 4)
    wl.table["state"][:] = gen.DONE
    assert_step_parity(wl, steps=2, commit=True)
    wl = gen.random_table(13, 700, 4)
    wl.table["arrival_ns"][:] = wl.now.max() + SEC                     # everything in the future
    wl.table["state"][:] = gen.QUEUED
    assert_step_parity(wl, steps=3, commit=True)


def test_bad_rows_are_flagged_not_fatal():
    wl = gen.random_table(14, 3000, 5, modes=MODES3)
    t = wl.table
    t["replica_id"][::17] = 5
    t["replica_id"][5::31] = -1
    t["class_id"][3::29] = 200
    t["prompt_len"][7::37] = -1
    t["gen"][11::41] = (1 << 24) + 1
    g = assert_step_parity(wl, steps=2, commit=True)
    sched = make_sched(wl)
    assert sched.status() == 0
    sched.close()
    # -1 on a QUEUED row is the global queue, not an error: a table whose only oddity is that raises nothing
    wl = gen.random_table(15, 3000, 5, modes=MODES3)
    q = np.flatnonzero(wl.table["state"] == gen.QUEUED)
    wl.table["replica_id"][q[::3]] = -1
    cpu = wl.copy()
    assert oracle.step(cpu)["status"] == 0
    assert_step_parity(wl, steps=2, commit=True)
    wl.table["replica_id"][np.flatnonzero(wl.table["state"] == gen.RUNNING)[:1]] = -1
    assert oracle.step(wl.copy())["status"] == 1
    assert_step_parity(wl, steps=1)


def test_ties_in_every_key_field():
    rows = []
    for i in range(600):
        rows.append(dict(prompt_len=64, arrival_ns=0, class_id=i % 2, req_id=(i * 7919) % 600 - 300,
                         state=gen.RUNNING if i % 3 == 0 else gen.QUEUED, first_token_ns=MS, gen=2))
    wl = make_wl(rows, [(200 * MS, 30 * MS, 1), (200 * MS, 30 * MS, 1)], now=[50 * MS],
                 replicas=[(gen.COLOCATED, 8192, 0)])
    assert_step_parity(wl, steps=2, commit=True)


def test_slack_saturation_and_budget_zero():
    # waits far beyond 2^39 ns saturate the key's slack field: order falls back to req_id
    rows = [dict(prompt_len=100 + i, arrival_ns=-(i % 5) * 700 * SEC, req_id=1000 - i, class_id=i % 3) for i in range(300)]
    cls = [(200 * MS, 30 * MS, 0), (0, 0, 0), (1 << 44, 1 << 34, 0)]
    wl = make_wl(rows, cls, now=[5 * SEC])
    g = assert_step_parity(wl, steps=2, commit=True)
    # TPOT <= E_d: nothing is safe
    rows = [dict(state=gen.RUNNING, prompt_len=4000, gen=50, first_token_ns=0, req_id=i, output_len=900) for i in range(260)]
    rows += [dict(prompt_len=16, req_id=500 + i) for i in range(50)]
    g = assert_step_parity(make_wl(rows, [(200 * MS, 30 * MS, 0)], now=[SEC]), steps=2, commit=True)
    assert g["budget"][0] == 0 and g["adm_count"][0] == 0
    # zero-token prompts fit a zero budget
    rows += [dict(prompt_len=0, req_id=900 + i) for i in range(3)]
    g = assert_step_parity(make_wl(rows, [(200 * MS, 30 * MS, 0)], now=[SEC]), steps=2, commit=True)


def test_maturity_saturates():
    # k * E_d beyond 64 bits: one running request whose TPOT leaves 1 ns of slack per step, a slow prefill
    model = (1 << 40, 40_000, 2, 1 << 33, 100_000, 20)
    tpot = (1 << 33) + 100_000 + 20 * 1000 + 1
    rows = [dict(state=gen.RUNNING, prompt_len=1000, gen=0, first_token_ns=0, req_id=0, output_len=50),
            dict(prompt_len=64, req_id=1, output_len=50)]
    wl = make_wl(rows, [(1 << 44, tpot, 0)], now=[SEC], model=model, budget_mode=gen.BUDGET_CAP_ONLY)
    g = assert_step_parity(wl, steps=2, commit=True)
    wl = make_wl(rows, [(1 << 44, tpot, 0)], now=[SEC], model=model, budget_mode=gen.BUDGET_CAP_ONLY)
    g = assert_step_parity(wl)
    assert g["maturity_next"][0] == 1 << 62 and g["adm_count"][0] == 1
    # and just below the 64-bit product limit / the saturation point
    for c0 in (1 << 20, 1 << 28, 1 << 29, 1 << 30):
        wl = make_wl(rows, [(1 << 44, tpot, 0)], now=[SEC], model=(c0,) + model[1:], budget_mode=gen.BUDGET_CAP_ONLY)
        assert_step_parity(wl)


def test_oversize_prompts_and_batch_cap():
    wl = gen.random_table(15, 2500, 6, token_cap=512, batch_cap=3, modes=MODES3)
    assert_step_parity(wl, steps=4, commit=True)


def test_scheduler_reuse_and_capacity():
    wl = gen.random_table(16, 1200, 4)
    sched = make_sched(wl, max_rows=5000)
    assert_step_parity(wl, sched=sched)
    wl2 = gen.random_table(17, 4999, 4)
    wl2.classes, wl2.replicas = wl.classes, wl.replicas
    assert_step_parity(wl2, steps=2, commit=True, sched=sched)
    assert sched.launch_count() > 0
    sched.close()


# ---- simulator ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(4))
def test_simulator_ragged_traces(seed):
    wl = gen.random_traces(seed, 40, 0, 300, iters=4000, token_cap=(8192, 600)[seed % 2])
    assert_sim_parity(wl)


def test_simulator_iteration_limits():
    wl = gen.random_traces(20, 12, 50, 200, iters=0)
    for iters in (0, 1, 7, 150):
        assert_sim_parity(wl, iters=iters)


def test_simulator_traces_beyond_shared_memory():
    # 20,000 rows do not fit a block's shared memory: the trace's rows work in device scratch (same code)
    wl = gen.random_traces(23, 2, 20_000, 20_000, iters=1200, rate=400.0, out_hi=64)
    assert_sim_parity(wl)
    # 9,000 rows: still in shared memory, one trace per SM
    wl = gen.random_traces(24, 2, 9000, 9000, iters=1500, rate=300.0, out_hi=64)
    assert_sim_parity(wl)


def test_simulator_trace_length_limit():
    # rows of a trace are numbered with 16 bits inside the simulator: 65,536 rows are refused before anything is launched
    import paper_2508_15919_b200 as hfx
    wl = gen.random_traces(25, 1, 65_536, 65_536, iters=1)
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    with pytest.raises(hfx.HfxError) as e:
        sched.sim_run(tab, wl.trace_off, 1, hfx.SimOut(1))
    assert e.value.code == -3
    sched.close()


def test_simulator_long_trace_and_weights():
    wl = gen.random_traces(21, 3, 3000, 4096, iters=6000, rate=60.0)
    wl.weight_max = 8
    wl.table["weight"][:] = np.random.default_rng(0).integers(0, 12, wl.n_rows).astype(np.int32)
    assert_sim_parity(wl)


def test_simulator_saturated_slack_and_zero_prompts():
    # a slow model makes waits exceed the 40-bit slack field; zero-token prompts are admitted at budget 0
    model = (200 * SEC, 40_000, 2, 8_000_000, 100_000, 20)
    cls = [(1 << 44, 30 * MS, 0), (200 * MS, 30 * MS, 0), (0, 0, 0)]
    wl = gen.random_traces(22, 6, 20, 60, iters=3000, model=model, classes=cls, out_hi=8)
    wl.table["prompt_len"][::9] = 0
    assert_sim_parity(wl)


def test_simulator_bad_rows():
    wl = gen.random_traces(23, 5, 50, 100, iters=2000)
    wl.table["class_id"][::13] = 99
    wl.table["prompt_len"][5::17] = -3
    res, cols, st = run_sim_gpu(wl)
    assert st == 2 | 4
    assert_sim_parity(wl)


# ---- argument errors ---------------------------------------------------------------------------------
def test_argument_errors():
    import paper_2508_15919_b200 as hfx
    wl = gen.random_table(30, 64, 2)
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    now = torch.from_numpy(wl.now).cuda(); mat = torch.from_numpy(wl.maturity).cuda()
    out = hfx.StepOut(64, 2)
    bad = hfx.StepOut(64, 2)
    bad.t["order"] = torch.zeros(65, dtype=torch.int32, device="cuda")[1:]
    with pytest.raises(hfx.HfxError) as e:
        sched.step(tab, now, mat, bad)
    assert e.value.code == -2
    bad = hfx.StepOut(64, 2)
    bad.t["admit"] = None
    with pytest.raises(hfx.HfxError) as e:
        sched.step(tab, now, mat, bad)
    assert e.value.code == -1
    big = hfx.DeviceTable.from_numpy(gen.random_table(31, 65, 2).table)
    with pytest.raises(hfx.HfxError) as e:
        sched.step(big, now, mat, out)
    assert e.value.code == -3
    tab.cols["output_len"] = None
    with pytest.raises(hfx.HfxError) as e:
        sched.step(tab, now, mat, out, commit=True)
    assert e.value.code == -1
    sched.step(tab, now, mat, out)          # still usable, and output_len is optional without commit
    assert sched.status() == 0
    with pytest.raises(hfx.HfxError):
        hfx.Scheduler((1, 1, 1 << 13, 1, 1, 1), wl.classes, wl.replicas, 10)
    with pytest.raises(hfx.HfxError):
        hfx.Scheduler(wl.model, wl.classes, [(3, 100, 0)], 10)
    sched.close()


# ---- scaler tick -----------------------------------------------------------------------------------------
def _scale_parity(wl, now, total_blocks, **kw):
    import paper_2508_15919_b200 as hfx
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    tb = torch.from_numpy(np.ascontiguousarray(total_blocks, np.int32)).cuda()
    counts = torch.full((3, 4), -1, dtype=torch.int64, device="cuda")
    used = torch.full((wl.n_replicas,), -1, dtype=torch.int64, device="cuda")
    dec = torch.full((3, 2), 9, dtype=torch.int32, device="cuda")
    for _ in range(2):      # twice: the outputs must not accumulate
        sched.scale_tick(tab, now, tb, counts, used, dec, **{("window_ns" if k == "window" else k): v for k, v in kw.items()})
    st = sched.status()
    c = oracle.scale_tick(wl, now, total_blocks, **kw)
    assert st == c["status"]
    assert np.array_equal(counts.cpu().numpy(), c["counts"]), (counts.cpu().numpy(), c["counts"])
    assert np.array_equal(used.cpu().numpy(), c["used_blocks"])
    assert np.array_equal(dec.cpu().numpy(), c["decision"]), (dec.cpu().numpy(), c["decision"])
    sched.close()
    return c


def test_scaler_tick_parity():
    rng = np.random.default_rng(3)
    wl = gen.config4(R=64, n=200_001, steps=1)
    wl.table["state"][::7] = gen.DONE
    wl.table["finish_ns"][::7] = wl.table["arrival_ns"][::7] + rng.integers(0, 20 * SEC, wl.table["finish_ns"][::7].shape)
    tb = rng.integers(0, 4000, 64)
    seen = set()
    for now, kw in ((30 * SEC, {}), (12 * SEC, dict(min_samples=100_000)),
                    (30 * SEC, dict(eps_out=(1, 1000), eps_wait=(1000, 1), eps_in=(1, 100))),
                    (30 * SEC, dict(eps_out=(1, 1000), eps_wait=(1000, 1), eps_in=(1000, 1))),
                    (30 * SEC, dict(window=SEC, block_tokens=1, eps_out=(1, 1000)))):
        c = _scale_parity(wl, now, tb, **kw)
        seen.add(int(c["decision"][0][0]))
    assert seen == {1, 0, -1}
    # all three pools, bad rows, ties for the emptiest instance, more replicas than fit the shared counters
    wl = gen.random_table(5, 30_000, 40, modes=MODES3, future=0.1, done=0.4)
    wl.table["finish_ns"][:] = wl.now.max() - rng.integers(0, 3 * SEC, wl.n_rows)
    wl.table["replica_id"][::31] = 77
    wl.table["class_id"][5::29] = 200
    tb = np.full(40, 1000); tb[::5] = 0
    _scale_parity(wl, int(wl.now.max()), tb, window=2 * SEC, eps_in=(1, 50), eps_wait=(50, 1), min_samples=1)
    wl = gen.random_table(6, 20_000, 9000)
    _scale_parity(wl, int(wl.now.max()), np.full(9000, 5), window=2 * SEC)
    wl = gen.random_table(7, 0, 3)
    _scale_parity(wl, 5, np.full(3, 5))
    # requests still in the global queue (QUEUED, bound to no instance) count for the colocated pool and the P stage
    wl = gen.random_table(8, 30_001, 12, modes=MODES3, future=0.1, done=0.3)
    wl.table["replica_id"][::3] = -1
    c = _scale_parity(wl, int(wl.now.max()), np.full(12, 500), window=2 * SEC, min_samples=1)
    assert c["counts"][0][2] > 1000 and c["counts"][1][2] > 1000 and c["status"] != 0


# ---- dispatching over the shared global queue -------------------------------------------------------
def _colocated(wl):
    wl.replicas[:, 0] = gen.COLOCATED
    return wl


@pytest.mark.parametrize("seed", range(10))
def test_dispatch_random_tables(seed):
    wl = gen.random_table(seed, 500 + 1777 * seed, 1 + (seed * 5) % 19, modes=(gen.COLOCATED,), tie_heavy=seed % 3 == 0,
                          batch_cap=(0, 9)[seed % 2], weight_max=(0, 16)[seed % 4 == 1], token_cap=(4096, 700)[seed % 3 == 1],
                          budget_mode=(gen.BUDGET_SAFE, gen.BUDGET_CAP_ONLY)[seed % 5 == 2])
    assert_dispatch_parity(wl, int(wl.now.max()), calls=2)


def test_dispatch_hand_worked_case_and_degenerate_tables():
    now = 1000 * MS
    classes = [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1)]
    rows = [dict(state=1, replica_id=0, prompt_len=800, output_len=500, first_token_ns=now - 30 * MS) for _ in range(80)]
    rows += [dict(replica_id=-1, class_id=0, prompt_len=1000, arrival_ns=now - 10 * MS),
             dict(replica_id=-1, class_id=0, prompt_len=1144, arrival_ns=now - 50 * MS),
             dict(replica_id=-1, class_id=1, prompt_len=281, arrival_ns=now - 900 * MS),
             dict(replica_id=-1, class_id=0, prompt_len=16, arrival_ns=now - 1 * MS),
             dict(replica_id=-1, class_id=1, prompt_len=2000, arrival_ns=now - 100 * MS),
             dict(replica_id=-1, class_id=0, prompt_len=16, arrival_ns=now + 1)]
    wl = make_wl(rows, classes, replicas=[(gen.COLOCATED, 8192, 0)] * 3, now=[now] * 3, maturity=[now - 5, now - 10, now + 1])
    g = assert_dispatch_parity(wl, now)
    assert list(g["assign"][80:86]) == [1, 1, 0, 0, -1, -1] and list(g["adm_cost"]) == [297, 2144, 0]
    # nothing queued; nothing matured; an empty table; zero-token prompts against a zero budget
    wl2 = wl.copy(); wl2.table["state"][80:] = 2
    assert_dispatch_parity(wl2, now)
    wl3 = wl.copy(); wl3.maturity[:] = now + 7
    assert_dispatch_parity(wl3, now)
    assert_dispatch_parity(make_wl([], classes, replicas=[(gen.COLOCATED, 8192, 0)] * 2, now=[now] * 2, maturity=[0, 0]), now)
    wl4 = wl.copy(); wl4.table["prompt_len"][80:84] = 0; wl4.replicas[:, 1] = 80
    assert_dispatch_parity(wl4, now)
    # the most urgent entry is larger than every budget of the call: passed over, the rest is served
    wl5 = wl.copy(); wl5.table["prompt_len"][80] = 3000
    g = assert_dispatch_parity(wl5, now)
    assert list(g["assign"][80:86]) == [-1, 1, 1, 1, -1, -1]


def test_dispatch_shared_queue_workload():
    # the shared-queue workload at reduced and at full size: many tiles, ragged tail, 1024 instances
    wl = gen.config4(R=64, n=200_001, steps=1)
    assert_dispatch_parity(wl, int(wl.now[0]))
    wl = gen.config4(steps=1)
    wl.maturity[::7] = wl.now[0] + 5            # some instances have not matured
    g = assert_dispatch_parity(wl, int(wl.now[0]))
    assert g["n_queue"][0] > 300_000 and g["adm_count"].sum() > 10_000


def test_dispatch_argument_errors_and_bad_rows():
    import paper_2508_15919_b200 as hfx
    wl = gen.random_table(40, 300, 3, modes=(gen.COLOCATED,))
    now = int(wl.now.max())
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    mat = torch.from_numpy(wl.maturity).cuda()
    out = hfx.DispatchOut(300, 3)
    bad = hfx.DispatchOut(300, 3)
    bad.t["assign"] = torch.zeros(304, dtype=torch.int32, device="cuda")[1:]
    with pytest.raises(hfx.HfxError) as e:
        sched.dispatch_step(tab, now, mat, bad)
    assert e.value.code == -2
    bad = hfx.DispatchOut(300, 3)
    bad.t["n_queue"] = None
    with pytest.raises(hfx.HfxError) as e:
        sched.dispatch_step(tab, now, mat, bad)
    assert e.value.code == -1
    big = hfx.DeviceTable.from_numpy(gen.random_table(41, 301, 3).table)
    with pytest.raises(hfx.HfxError) as e:
        sched.dispatch_step(big, now, mat, out)
    assert e.value.code == -3
    sched.dispatch_step(tab, now, mat, out)          # still usable
    assert sched.status() == 0
    sched.close()
    # P-stage instances are served like colocated ones, D-stage instances by the second stage of the call
    for seed in (42, 44, 45):
        wl2 = gen.random_table(seed, 3000, 7, modes=MODES3, batch_cap=(0, 5)[seed % 2])
        assert_dispatch_parity(wl2, int(wl2.now.max()))
    # rows with ids or lengths outside the domain are flagged and take no part
    wl3 = gen.random_table(43, 2000, 5, modes=(gen.COLOCATED,))
    wl3.table["class_id"][::97] = 200
    wl3.table["prompt_len"][5::131] = -3
    wl3.table["replica_id"][7::53] = 99
    assert_dispatch_parity(wl3, int(wl3.now.max()))


def test_migrator_selects_d_instances():
    # the D stage of the dispatching call (Sec. 3.3.1, "D-stage Migrator"): the hand-worked case, then seeded tables
    from helpers import migrator_case, migrator_hand_case
    wl, now = migrator_hand_case()
    g = assert_dispatch_parity(wl, now, calls=2)
    assert list(g["assign"]) == [-1, -1, -1, 2, 1, -1] and list(g["n_queue"]) == [0, 3] and list(g["inst_order"]) == [2, 1, -1]
    for seed in range(12):
        wl, now = migrator_case(seed, batch_cap=(0, 6)[seed % 3 == 1], tie_heavy=seed % 4 == 2,
                                budget_mode=(gen.BUDGET_SAFE, gen.BUDGET_CAP_ONLY)[seed % 5 == 3], permute_ids=seed % 2 == 0)
        assert_dispatch_parity(wl, now)
    # D instances only (no P stage: the queue of prefilled requests is empty, the budgets and maturities stand)
    wl = gen.random_table(77, 5000, 4, modes=(gen.DECODE,), inflight=0.5)
    assert_dispatch_parity(wl, int(wl.now.max()))


def test_migrator_many_tiles_and_binding():
    # a table whose two queues span many tiles; both stages dispatch; binding puts the prefilled requests in flight
    # on their D instances, and the per-replica step that follows agrees with the oracle's
    import paper_2508_15919_b200 as hfx
    R = 48
    wl = gen.random_table(88, 150_001, R, modes=MODES3, inflight=0.6, permute_ids=False)
    wl.replicas[:, 0] = np.arange(R) % 3                      # colocated, P, D in turn
    now = int(wl.now.max())
    wl.now[:] = now
    t = wl.table
    on_p = (t["state"] == gen.RUNNING) & (wl.replicas[np.clip(t["replica_id"], 0, R - 1), 0] == gen.PREFILL)
    rng = np.random.default_rng(5)
    t["first_token_ns"][on_p] = now - rng.integers(-2 * MS, 30 * MS, int(on_p.sum()))
    on_d = np.nonzero((t["state"] == gen.RUNNING) & (wl.replicas[np.clip(t["replica_id"], 0, R - 1), 0] == gen.DECODE))[0]
    t["state"][on_d[on_d % 100 != 0]] = gen.DONE            # small decode batches: the D instances have room
    wl.maturity[:] = now - rng.integers(-1 * MS, 10 * MS, R)
    g = assert_dispatch_parity(wl, now)
    assert g["n_queue"][0] > 10_000 and g["n_queue"][1] > 10_000 and g["n_mature"][1] > 0
    d_inst = np.nonzero(wl.replicas[:, 0] == gen.DECODE)[0]
    assert g["adm_count"][d_inst].sum() > 0 and set(np.unique(g["assign"][on_p])) <= set(d_inst.tolist()) | {-1}
    # bind on both sides, then one per-replica step
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    out = hfx.DispatchOut(wl.n_rows, R)
    mat = torch.from_numpy(wl.maturity.copy()).cuda()
    clock = torch.from_numpy(wl.now.copy()).cuda()
    sched.dispatch_step(tab, now, mat, out)
    sched.dispatch_bind(tab, now, out, clock)
    c = oracle.dispatch(wl, now)
    oracle.dispatch_bind(wl, now, c)
    assert np.array_equal(tab.to_numpy()["replica_id"], wl.table["replica_id"]) and np.array_equal(clock.cpu().numpy(), wl.now)
    sched.close()
    wl.maturity[:] = c["maturity_next"]
    assert_step_parity(wl, steps=2, commit=True)


# ---- priority-based SLO mapping ---------------------------------------------------------------------------
def _slo_parity(n_prio, win, bounds, last, pending, new, calls=2):
    import paper_2508_15919_b200 as hfx
    wl = gen.random_table(1, 16, 1)
    sched = make_sched(wl)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a, dt)).cuda()
    w = {"prio": dev(win["prio"], np.int32), "ttft_ns": dev(win["ttft"], np.int64), "tpot_ns": dev(win["tpot"], np.int64),
         "queue_ns": dev(win["queue"], np.int64)}
    b = {k + "_ns": dev(bounds[k], np.int64) for k in oracle.SLO_BOUND_KEYS}
    lq = dev(last, np.int64)
    lq_cpu = np.ascontiguousarray(last, np.int64)
    pend = dev(pending, np.int32)
    npr = dev(new, np.int32)
    n = int(npr.shape[0])
    t_out = torch.full((max(n, 1),), -7, dtype=torch.int64, device="cuda")
    p_out = torch.full((max(n, 1),), -7, dtype=torch.int64, device="cuda")
    for _ in range(calls):       # the second call starts from the delays the first one left behind
        sched.slo_map(n_prio, w, b, lq, pend, npr, t_out, p_out)
        st = sched.status()
        c = oracle.slo_map(n_prio, win, bounds, lq_cpu, pending, new)
        lq_cpu = c["last_queue"]
        assert st == c["status"]
        assert np.array_equal(t_out.cpu().numpy()[:n], c["ttft_slo"]), (t_out.cpu().numpy()[:8], c["ttft_slo"][:8])
        assert np.array_equal(p_out.cpu().numpy()[:n], c["tpot_slo"])
        assert np.array_equal(lq.cpu().numpy(), c["last_queue"])
    sched.close()
    return c


def test_slo_mapping_hand_worked_and_edges():
    win = {"prio": np.array([0, 1, 0, 2, 1, 2]), "ttft": np.array([100, 300, 150, 900, 250, 700]) * MS,
           "tpot": np.array([20, 40, 25, 80, 35, 60]) * MS, "queue": np.array([10, 50, 30, 400, 20, 200]) * MS}
    bounds = {"ttft_min": np.array([150, 200, 700]) * MS, "ttft_max": np.array([200, 1000, 5000]) * MS,
              "ttft_min_relaxed": np.array([50, 100, 200]) * MS, "tpot_min": np.array([30, 30, 50]) * MS,
              "tpot_max": np.array([30, 50, 100]) * MS, "tpot_min_relaxed": np.array([10, 20, 30]) * MS}
    last = np.array([10, 30, 100]) * MS
    c = _slo_parity(3, win, bounds, last, np.array([0, 3, 0]), np.array([1, 2, 1, 0]))
    _slo_parity(3, win, bounds, last, np.array([0, 0, 0]), np.array([1, 2, 1, 0]))
    _slo_parity(3, {k: v[:0] for k, v in win.items()}, bounds, last, np.array([0, 0, 0]), np.array([1, 2, 1, 0]))    # empty window
    _slo_parity(3, win, bounds, last, np.array([1, 0, 0]), np.array([], np.int32))                                  # no requests
    bad = dict(win); bad["prio"] = np.array([0, 9, 0, -1, 1, 2])
    _slo_parity(3, bad, bounds, last, np.array([0, 0, 1]), np.array([1, 5, 2, -2, 0]))                              # bad priorities


@pytest.mark.parametrize("seed", range(6))
def test_slo_mapping_random(seed):
    rng = np.random.default_rng(seed)
    N = int(rng.integers(1, 65)) if seed else 64
    w = [4096, 1, 37, 1000, 4095, 513][seed]
    ties = seed % 2 == 1
    win = {"prio": rng.integers(0, N, w), "ttft": rng.integers(1, 50 if ties else 10**10, w),
           "tpot": rng.integers(1, 20 if ties else 10**9, w), "queue": rng.integers(0, 10**9, w)}
    lo = rng.integers(0, 10**8, N)
    bounds = {"ttft_min": lo + 10**8, "ttft_max": lo + 5 * 10**9, "ttft_min_relaxed": lo,
              "tpot_min": lo // 10 + 10**7, "tpot_max": lo // 10 + 5 * 10**8, "tpot_min_relaxed": lo // 10}
    last = rng.integers(0, 10**9, N)
    pending = rng.integers(0, 2, N) * rng.integers(0, 2, N)
    new = rng.integers(0, N, 10_000 + seed)
    _slo_parity(N, win, bounds, last, pending, new)


# ---- the two stages of the disaggregated mode coupled by the hand-off --------------------------------------
def _pd_coupled_parity(wl, pair, rounds, x0=2 * MS, x1=500):
    """`rounds` times (committed step, hand-off) on both sides; the table, the clocks and the step's
    outputs must agree after every call."""
    import paper_2508_15919_b200 as hfx
    cpu = wl.copy()
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    now = torch.from_numpy(wl.now.copy()).cuda(); mat = torch.from_numpy(wl.maturity.copy()).cuda()
    prt = torch.from_numpy(pair).cuda()
    out = hfx.StepOut(wl.n_rows, wl.n_replicas, optional=False)
    moved = torch.zeros(4, dtype=torch.int32, device="cuda")
    total_moved = 0
    for k in range(rounds):
        sched.step(tab, now, mat, out, commit=True)
        c = oracle.step(cpu, commit=True)
        g = out.to_numpy()
        for ko, kg in (("order", "order"), ("admit", "admit"), ("budget", "budget"), ("adm_count", "adm_count"), ("slack", "slack_ns")):
            assert np.array_equal(g[kg], c[ko]), (k, kg)
        sched.pd_migrate(tab, now, mat, prt, x0, x1, moved)
        st = sched.status()
        r = oracle.pd_migrate(cpu, pair, x0, x1)
        assert st == (c["status"] | r["status"]), (k, st, c["status"], r["status"])
        assert int(moved[0].item()) == r["moved"], (k, int(moved[0].item()), r["moved"])
        total_moved += r["moved"]
        tg = tab.to_numpy()
        for col in ("replica_id", "state", "gen", "first_token_ns", "last_token_ns", "finish_ns"):
            assert np.array_equal(tg[col], cpu.table[col]), f"round {k}: column {col} differs at {np.nonzero(tg[col] != cpu.table[col])[0][:8]}"
        assert np.array_equal(now.cpu().numpy(), cpu.now), f"round {k}: now"
        assert np.array_equal(mat.cpu().numpy(), cpu.maturity), f"round {k}: maturity"
    sched.close()
    return cpu, total_moved


@pytest.mark.parametrize("seed,pairs,rows_per", [(0, 1, 40), (1, 3, 200), (2, 16, 1500)])
def test_pd_coupled_stages(seed, pairs, rows_per):
    wl = gen.pd_pairs(seed, pairs, rows_per)
    cpu, moved = _pd_coupled_parity(wl, gen.pd_partner_table(pairs), rounds=(60, 40, 25)[seed])
    t = cpu.table
    # requests went through both stages: some finished on a D instance, every first token precedes its last one
    assert moved > 0 and np.count_nonzero((t["state"] == 2) & (t["replica_id"] >= pairs)) > 0
    done = t["state"] == 2
    assert np.all(t["first_token_ns"][done] <= t["finish_ns"][done]) and np.all(t["arrival_ns"][done] <= t["first_token_ns"][done])


def test_pd_handoff_edges_and_errors():
    import paper_2508_15919_b200 as hfx
    # bad partners, rows with bad data, an empty table; argument errors
    wl = gen.pd_pairs(5, 2, 300)
    wl.table["class_id"][::41] = 99
    pair = gen.pd_partner_table(2); pair[1] = 0          # instance 1's partner is a P instance: flagged, its rows stay
    _pd_coupled_parity(wl, pair, rounds=12)
    wl0 = gen.pd_pairs(6, 1, 8)
    sched = make_sched(wl0)
    tab = hfx.DeviceTable.from_numpy(wl0.table)
    now = torch.from_numpy(wl0.now.copy()).cuda(); mat = torch.from_numpy(wl0.maturity.copy()).cuda()
    prt = torch.from_numpy(gen.pd_partner_table(1)).cuda()
    with pytest.raises(hfx.HfxError) as e:
        sched.pd_migrate(tab, now, mat, prt, -1, 0)
    assert e.value.code == -1
    with pytest.raises(hfx.HfxError) as e:
        sched.pd_migrate(tab, now, mat, prt[1:], 0, 0)
    assert e.value.code == -2
    sched.pd_migrate(tab, now, mat, prt, 0, 0)          # nothing is RUNNING on a P instance yet: a no-op
    assert sched.status() == 0 and np.array_equal(tab.to_numpy()["replica_id"], wl0.table["replica_id"])
    sched.close()


# ---- SLO attainment (Eq. 2) ---------------------------------------------------------------------------------
def _attainment_parity(wl):
    import paper_2508_15919_b200 as hfx
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    out = torch.full((len(wl.classes) + 1, 6), -3, dtype=torch.int64, device="cuda")
    for _ in range(2):          # twice: the output must not accumulate
        sched.attainment(tab, out)
    st = sched.status()
    c = oracle.attainment(wl)
    assert st == c["status"] and np.array_equal(out.cpu().numpy(), c["counts"]), (out.cpu().numpy(), c["counts"])
    sched.close()
    return c["counts"]


def test_attainment_parity():
    cls = [(200 * MS, 30 * MS, 0), (1000 * MS, 0, 1)]
    rows = [dict(state=gen.DONE, class_id=0, prompt_len=1000, output_len=101, gen=100, first_token_ns=47 * MS, last_token_ns=859_099_000, finish_ns=859_099_000),
            dict(state=gen.DONE, class_id=0, output_len=11, gen=10, arrival_ns=100 * MS, first_token_ns=350 * MS, last_token_ns=850 * MS, finish_ns=850 * MS),
            dict(state=gen.RUNNING, class_id=0, output_len=50, gen=3, arrival_ns=5 * MS, first_token_ns=15 * MS, last_token_ns=99 * MS),
            dict(state=gen.REJECTED, class_id=1, prompt_len=100000), dict(state=gen.QUEUED, class_id=1, arrival_ns=7 * MS),
            dict(state=gen.DONE, class_id=1, output_len=1, arrival_ns=MS, first_token_ns=1000 * MS, last_token_ns=1000 * MS, finish_ns=1000 * MS)]
    c = _attainment_parity(make_wl(rows, cls))
    assert list(c[2][:4]) == [6, 3, 2, 1]
    _attainment_parity(make_wl([], cls))
    # the table a simulation leaves, and a committed shared-queue table with bad rows
    wl = gen.random_traces(4, 40, 100, 300, 600)
    oracle.sim(wl)
    c = _attainment_parity(wl)
    assert c[-1][1] > 0
    wl = gen.config4(R=32, n=100_003, steps=3)
    for _ in range(3):
        oracle.step(wl, commit=True)
    wl.table["class_id"][::997] = 77
    _attainment_parity(wl)


# ---- first-fit admission variant -----------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(8))
def test_first_fit_random_tables(seed):
    wl = gen.random_table(50 + seed, 1500 + 1333 * seed, 1 + (seed * 3) % 11, modes=MODES3, tie_heavy=seed % 3 == 0,
                          batch_cap=(0, 7)[seed % 2], weight_max=(0, 16)[seed % 4 == 1],
                          budget_mode=(gen.BUDGET_SAFE, gen.BUDGET_CAP_ONLY)[seed % 5 == 2], grouped=seed % 4 == 3)
    wl.meta["first_fit"] = True
    assert_step_parity(wl, steps=3, commit=True)


def test_first_fit_all_segment_sizes_and_simulator():
    for wl in (gen.config4(R=16, n=30_000, steps=3), gen.random_table(7, 9000, 1, tie_heavy=True),
               gen.random_table(9, 40_001, 1), gen.config2(R=8, rows_per=2048, inflight=0.02)):
        wl.meta["first_fit"] = True
        assert_step_parity(wl, steps=2, commit=True)
    wl = gen.random_traces(11, 12, 60, 400, 500)
    wl.meta["first_fit"] = True
    assert_sim_parity(wl)
    wl = gen.config1()
    wl.meta["first_fit"] = True
    assert_sim_parity(wl)


def test_disaggregated_pipeline_dispatch_step_handoff():
    # the whole disaggregated flow on both sides: requests wait unbound in the global queue, the dispatcher hands
    # them to matured P instances, the caller binds them, a committed step prefills and decodes, the hand-off moves
    # prefilled requests to the D instances
    import paper_2508_15919_b200 as hfx
    pairs = 4
    wl = gen.pd_pairs(21, pairs, 400)
    wl.table["replica_id"][:] = -1
    cpu = wl.copy()
    pair = gen.pd_partner_table(pairs)
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    now = torch.from_numpy(wl.now.copy()).cuda(); mat = torch.from_numpy(wl.maturity.copy()).cuda()
    prt = torch.from_numpy(pair).cuda()
    dout = hfx.DispatchOut(wl.n_rows, wl.n_replicas)
    sout = hfx.StepOut(wl.n_rows, wl.n_replicas, optional=False)
    bound = 0
    for k in range(30):
        now_g = (k + 1) * 25 * MS          # the dispatcher's tick; an idle instance's clock catches up at its next step
        sched.dispatch_step(tab, now_g, mat, dout)
        d = oracle.dispatch(cpu, now_g)
        g = dout.to_numpy()
        assert np.array_equal(g["assign"], d["assign"]) and np.array_equal(g["maturity_next"], d["maturity_next"]), k
        # bind: the dispatched requests now belong to their instance, which is busy until its new maturity
        asg = dout.t["assign"][:wl.n_rows]
        tab.cols["replica_id"].copy_(torch.where(asg >= 0, asg, tab.cols["replica_id"]))
        sel = d["assign"] >= 0
        cpu.table["replica_id"][sel] = d["assign"][sel]
        bound += int(sel.sum())
        sched.step(tab, now, mat, sout, commit=True)
        c = oracle.step(cpu, commit=True)
        sched.pd_migrate(tab, now, mat, prt, 2 * MS, 500)
        r = oracle.pd_migrate(cpu, pair, 2 * MS, 500)
        st = sched.status()
        assert st == (d["status"] | c["status"] | r["status"]), (k, st)
        tg = tab.to_numpy()
        for col in ("replica_id", "state", "gen", "first_token_ns", "last_token_ns", "finish_ns"):
            assert np.array_equal(tg[col], cpu.table[col]), f"round {k}: column {col}"
        assert np.array_equal(now.cpu().numpy(), cpu.now) and np.array_equal(mat.cpu().numpy(), cpu.maturity), k
    sched.close()
    assert bound > 50 and np.count_nonzero((cpu.table["state"] == 2) & (cpu.table["replica_id"] >= pairs)) > 0


# ---- rounds on a global clock: commit horizon, binding, the Scaler's decisions carried out -----------------
def test_commit_horizon_all_segment_sizes():
    # replicas whose clock is past the horizon report their decisions and change nothing; small, medium and
    # oversize segments, all three modes, both front ends
    for seed, n, R, kw in ((1, 6000, 37, dict(modes=MODES3)), (2, 30_000, 4, dict(modes=MODES3, grouped=True)),
                           (3, 16384 + 16385 + 3000, 3, dict(grouped=True, modes=MODES3))):
        wl = gen.random_table(seed, n, R, **kw)
        wl.now[::2] += 20 * MS
        wl.meta["horizon"] = int(wl.now.min()) + 10 * MS
        assert np.any(wl.now > wl.meta["horizon"]) and np.any(wl.now <= wl.meta["horizon"])
        assert_step_parity(wl, steps=3, commit=True)
    wl = gen.config2(R=16, rows_per=700)
    wl.now[::3] += 5 * SEC
    wl.meta["horizon"] = int(wl.now.min()) + SEC
    assert_step_parity(wl, steps=2, commit=True)
    wl.meta["horizon"] = -1                       # nobody acts
    assert_step_parity(wl, steps=1, commit=True)


def test_dispatch_bind_parity_and_errors():
    import paper_2508_15919_b200 as hfx
    wl = _colocated(gen.random_table(4, 5000, 9, modes=(gen.COLOCATED,)))
    wl.table["replica_id"][wl.table["state"] == gen.QUEUED] = -1
    now_g = int(wl.now.max())
    wl.now[::2] -= 3 * SEC                         # clocks behind the call are raised, the others stay
    cpu = wl.copy()
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    now = torch.from_numpy(wl.now.copy()).cuda(); mat = torch.from_numpy(wl.maturity.copy()).cuda()
    dout = hfx.DispatchOut(wl.n_rows, wl.n_replicas)
    sched.dispatch_step(tab, now_g, mat, dout)
    d = oracle.dispatch(cpu, now_g)
    assert np.array_equal(dout.to_numpy()["assign"], d["assign"]) and (d["assign"] >= 0).sum() > 5
    sched.dispatch_bind(tab, now_g, dout, now)
    oracle.dispatch_bind(cpu, now_g, d)
    assert np.array_equal(tab.to_numpy()["replica_id"], cpu.table["replica_id"]) and np.array_equal(now.cpu().numpy(), cpu.now)
    assert np.any(cpu.now != wl.now)
    import ctypes as C
    other = hfx.DeviceTable.from_numpy(wl.table)   # replica_id must be the table's own column
    ts, os_ = tab.c_struct(), dout.c_struct()
    assert sched._L.hfx_dispatch_bind(sched._h, C.byref(ts), other.cols["replica_id"].data_ptr(), now_g, C.byref(os_), now.data_ptr()) != 0
    assert sched._L.hfx_dispatch_bind(sched._h, C.byref(ts), tab.cols["replica_id"].data_ptr(), now_g, C.byref(os_), None) != 0
    sched.close()


def _fleet_parity(seed, R, modes, rounds=6):
    import paper_2508_15919_b200 as hfx
    rng = np.random.default_rng(seed)
    wl = gen.random_table(seed, 10, R, modes=modes)
    cpu = wl.copy()
    f = gen.new_fleet(rng.integers(1, 4000, R), rng.choice(R, max(1, R // 3), replace=False))
    f["inst_state"][:] = rng.integers(0, 4, R)                # every state from the start
    f["ready"][:] = rng.integers(0, 3 * SEC, R); f["since"][:] = rng.integers(0, SEC, R); f["billed"][:] = rng.integers(0, SEC, R)
    sched = make_sched(wl)
    fl = hfx.Fleet(f)
    now = torch.from_numpy(wl.now.copy()).cuda(); mat = torch.from_numpy(wl.maturity.copy()).cuda()
    cost = torch.full((3,), -1, dtype=torch.int64, device="cuda")
    cold = [300 * MS, 2 * SEC, 0]
    t = 0
    for k in range(rounds):
        t += int(rng.integers(0, SEC))
        dec = np.stack([rng.integers(-1, 2, 3), rng.integers(-2, R + 2, 3)], axis=1).astype(np.int32)
        used = (rng.integers(0, 50, R) * rng.integers(0, 2, R)).astype(np.int64)
        sched.scale_apply(t, torch.from_numpy(dec).cuda(), torch.from_numpy(used).cuda(), cold, fl, now, mat, cost)
        c = oracle.scale_apply(cpu, t, dec, used, cold, f)
        g = fl.to_numpy()
        for key in f:
            assert np.array_equal(g[key], f[key]), (seed, k, key, np.flatnonzero(g[key] != f[key])[:8])
        assert np.array_equal(cost.cpu().numpy(), c), (k, cost.cpu().numpy(), c)
        assert np.array_equal(now.cpu().numpy(), cpu.now) and np.array_equal(mat.cpu().numpy(), cpu.maturity)
    assert sched.status() == 0
    sched.close()
    return f


def test_scale_apply_parity():
    _fleet_parity(0, 1, (gen.COLOCATED,))
    _fleet_parity(1, 7, (gen.COLOCATED,), rounds=20)
    _fleet_parity(2, 40, MODES3, rounds=20)
    _fleet_parity(3, 1025, MODES3)                # more instances than the block has threads
    _fleet_parity(4, 5000, MODES3)


def test_scale_apply_hand_worked_sequence():
    # the hand-worked sequence of the pin file (costs 29, 56, 83, 104 instance-seconds) through the library
    import paper_2508_15919_b200 as hfx
    S = SEC
    wl = gen.random_table(0, 4, 5, modes=(gen.COLOCATED,))
    wl.replicas[4, 0] = gen.PREFILL
    wl.now[:] = 0; wl.maturity[:] = 0
    sched = make_sched(wl)
    fl = hfx.Fleet(gen.new_fleet([100] * 5, [0, 1, 4]))
    now = torch.zeros(5, dtype=torch.int64, device="cuda"); mat = torch.zeros(5, dtype=torch.int64, device="cuda")
    cost = torch.zeros(3, dtype=torch.int64, device="cuda")
    hold = [0, -1]
    seq = [(10, [1, -1], hold, [50, 20, 0, 0, 10]), (11, [1, -1], hold, [50, 20, 0, 0, 10]), (13, hold, [1, -1], [50, 20, 0, 0, 10]),
           (20, [-1, 1], hold, [50, 20, 5, 0, 10]), (21, hold, hold, [50, 20, 5, 0, 10]), (22, [1, -1], hold, [50, 7, 5, 0, 10]),
           (30, [-1, 0], hold, [9, 7, 5, 0, 10]), (31, hold, hold, [0, 7, 5, 0, 10]), (40, [1, -1], hold, [0, 7, 5, 0, 10]),
           (41, [-1, 0], [-1, 0], [0, 7, 5, 0, 10])]
    costs = {}
    for t, d0, d1, used in seq:
        sched.scale_apply(t * S, torch.tensor([d0, d1, hold], dtype=torch.int32, device="cuda"),
                          torch.tensor(used, dtype=torch.int64, device="cuda"), [2 * S, 5 * S, 7 * S], fl, now, mat, cost)
        costs[t] = cost.cpu().numpy().copy()
    assert [int(costs[t][0]) // S for t in (13, 22, 31, 41)] == [29, 56, 83, 104] and int(costs[41][1]) == 41 * S
    g = fl.to_numpy()
    assert list(g["inst_state"]) == [1, 2, 2, 0, 2] and list(g["billed"]) == [32 * S, 41 * S, 31 * S, 0, 41 * S]
    assert now.cpu().numpy()[2] == 12 * S
    sched.close()


@pytest.mark.parametrize("first_fit,rounds", [(False, 330), (True, 120)])
def test_scaling_loop_round_by_round(first_fit, rounds):
    # the whole loop: instances advance to the tick under the horizon, the Scaler ticks, its decisions are carried
    # out, the dispatcher serves the ACTIVE instances that are due, the requests are bound -- compared after each round
    import paper_2508_15919_b200 as hfx
    from oracle.elastic_loop import COLD, SCALE_KW, SUBSTEPS, oracle_round
    R = 8
    wl = gen.elastic(1, R, 1500)
    wl.meta["first_fit"] = first_fit
    cpu = wl.copy()
    f = gen.new_fleet([2000] * R, [0, 1])
    sched = make_sched(wl)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    fl = hfx.Fleet(f)
    now = torch.from_numpy(wl.now.copy()).cuda(); mat = torch.from_numpy(wl.maturity.copy()).cuda()
    sout = hfx.StepOut(wl.n_rows, R, optional=False)
    dout = hfx.DispatchOut(wl.n_rows, R)
    counts = torch.zeros((3, 4), dtype=torch.int64, device="cuda"); used = torch.zeros(R, dtype=torch.int64, device="cuda")
    dec = torch.zeros((3, 2), dtype=torch.int32, device="cuda"); cost = torch.zeros(3, dtype=torch.int64, device="cuda")
    on_max = 0
    for k in range(rounds):
        o = oracle_round(cpu, f, k)
        sched.set_horizon(o["now"])
        for _ in range(SUBSTEPS):
            sched.step(tab, now, mat, sout, commit=True)
        sched.scale_tick(tab, o["now"], fl.t["total_blocks"], counts, used, dec, window_ns=SCALE_KW["window"],
                         min_samples=SCALE_KW["min_samples"])
        sched.scale_apply(o["now"], dec, used, COLD, fl, now, mat, cost)
        sched.dispatch_step(tab, o["now"], fl.t["due"], dout)
        sched.dispatch_bind(tab, o["now"], dout, now)
        assert sched.status() == o["status"], k
        assert np.array_equal(counts.cpu().numpy(), o["tick"]["counts"]) and np.array_equal(dec.cpu().numpy(), o["tick"]["decision"]), k
        assert np.array_equal(dout.to_numpy()["assign"], o["dispatch"]["assign"]), k
        g = fl.to_numpy()
        for key in f:
            assert np.array_equal(g[key], f[key]), (k, key)
        assert np.array_equal(cost.cpu().numpy(), o["cost"]), k
        tg = tab.to_numpy()
        for col in ("replica_id", "state", "gen", "first_token_ns", "last_token_ns", "finish_ns"):
            assert np.array_equal(tg[col], cpu.table[col]), f"round {k}: column {col}"
        assert np.array_equal(now.cpu().numpy(), cpu.now) and np.array_equal(mat.cpu().numpy(), cpu.maturity), k
        on_max = max(on_max, int(np.count_nonzero(f["inst_state"] != gen.INST_OFF)))
    sched.close()
    if rounds >= 330:
        assert on_max >= 6 and np.count_nonzero(cpu.table["state"] == gen.DONE) > 700
    else:
        assert on_max >= 3 and np.count_nonzero(cpu.table["state"] == gen.DONE) > 50


@pytest.mark.parametrize("R,permute,fused", [(64, False, True), (64, True, True), (4, False, True), (64, False, False), (4, False, False)])
def test_tables_that_are_mostly_global_queue(R, permute, fused):
    # most rows bound to no instance (they wait in the global queue), a few bound ones in between: tiles with one
    # large group of unbound rows; ids rising (the step stays ordered) or permuted; with 4 instances the bound
    # groups of a tile are large too
    rng = np.random.default_rng(R + permute)
    wl = gen.elastic(3, R, 50_000)
    idx = rng.choice(20_000, 3000, replace=False)
    wl.table["replica_id"][idx] = rng.integers(0, R, 3000)
    wl.table["replica_id"][49_990:] = R + 5                      # and a few that are simply out of range
    wl.now[:] = int(np.sort(wl.table["arrival_ns"])[10_000])
    if permute:
        wl.table["req_id"][:] = rng.permutation(wl.n_rows).astype(np.int32)
    sched = make_sched(wl)
    sched.set_fused_front(fused)
    g = assert_step_parity(wl, steps=2, commit=True, sched=sched)
    sched.close()
    assert g["adm_count"].sum() > 0


def test_dispatch_with_instances_that_are_never_due():
    # the maturity array of a fleet: instances that are not ACTIVE are due "never"
    wl = _colocated(gen.random_table(11, 6000, 12, modes=(gen.COLOCATED,)))
    now = int(wl.now.max())
    wl.maturity[:] = gen.T_NEVER
    g = assert_dispatch_parity(wl, now)
    assert g["n_mature"][0] == 0 and (g["assign"] >= 0).sum() == 0
    wl.maturity[::3] = now - 5
    g = assert_dispatch_parity(wl, now)
    assert g["n_mature"][0] == 4 and (g["assign"] >= 0).sum() > 0 and set(np.unique(g["assign"])) <= {-1, 0, 3, 6, 9}


def test_scale_apply_and_horizon_argument_errors():
    import ctypes as C
    import paper_2508_15919_b200 as hfx
    from paper_2508_15919_b200.binding import _Fleet, _ReplicaState
    wl = gen.random_table(0, 10, 4)
    sched = make_sched(wl)
    fl = hfx.Fleet(gen.new_fleet([10] * 4, [0]))
    now = torch.zeros(4, dtype=torch.int64, device="cuda"); mat = torch.zeros(4, dtype=torch.int64, device="cuda")
    dec = torch.zeros((3, 2), dtype=torch.int32, device="cuda"); used = torch.zeros(4, dtype=torch.int64, device="cuda")
    cost = torch.zeros(4, dtype=torch.int64, device="cuda")
    L, h = sched._L, sched._h
    good = (C.c_int64 * 3)(1, 1, 1)
    fs = fl.c_struct(); st = _ReplicaState(now.data_ptr(), mat.data_ptr())

    def call(decision=dec.data_ptr(), usedp=used.data_ptr(), cold=good, fleet=fs, state=st, costp=cost.data_ptr()):
        return L.hfx_scale_apply(h, 5, decision, usedp, cold, C.byref(fleet), C.byref(state), costp)

    assert call() == 0
    assert call(decision=None) != 0 and call(usedp=None) != 0 and call(costp=None) != 0
    assert call(cold=(C.c_int64 * 3)(1, -1, 1)) != 0
    assert call(costp=cost.data_ptr() + 8) != 0                         # misaligned
    holes = fl.c_struct(); holes.due_ns = None
    assert call(fleet=holes) != 0
    assert call(state=_ReplicaState(now.data_ptr(), None)) != 0
    assert L.hfx_scale_apply(None, 5, dec.data_ptr(), used.data_ptr(), good, C.byref(fs), C.byref(st), cost.data_ptr()) != 0
    assert L.hfx_sched_set_horizon(None, 5) != 0
    assert sched.status() == 0
    sched.close()


def test_scale_decide_from_summed_counters():
    # the decision alone: from the tick's own counters it repeats the tick's decision; from counters of two shards
    # of the table, summed, it gives the decision of the whole table; and from arbitrary counters the oracle's
    import paper_2508_15919_b200 as hfx
    rng = np.random.default_rng(12)
    R = 23
    wl = gen.random_table(12, 40_000, R, modes=MODES3, future=0.1, done=0.4)
    wl.table["finish_ns"][:] = wl.now.max() - rng.integers(0, 3 * SEC, wl.n_rows)
    wl.table["replica_id"][::6] = -1
    now = int(wl.now.max())
    tb_np = (rng.integers(1, 900, R) * (rng.random(R) < 0.8)).astype(np.int32)
    kw = dict(window=2 * SEC, min_samples=1, eps_in=(1, 50), eps_wait=(50, 1))
    full = oracle.scale_tick(wl, now, tb_np, **kw)
    sched = make_sched(wl)
    tb = torch.from_numpy(tb_np).cuda()
    tot_c = torch.zeros((3, 4), dtype=torch.int64, device="cuda"); tot_u = torch.zeros(R, dtype=torch.int64, device="cuda")
    for half in range(2):
        part = {k: np.ascontiguousarray(v[half::2]) for k, v in wl.table.items()}
        tab = hfx.DeviceTable.from_numpy(part)
        c = torch.zeros((3, 4), dtype=torch.int64, device="cuda"); u = torch.zeros(R, dtype=torch.int64, device="cuda")
        d = torch.zeros((3, 2), dtype=torch.int32, device="cuda")
        sched.scale_tick(tab, now, tb, c, u, d, window_ns=kw["window"], min_samples=1, eps_in=kw["eps_in"], eps_wait=kw["eps_wait"])
        tot_c += c; tot_u += u
    assert np.array_equal(tot_c.cpu().numpy(), full["counts"]) and np.array_equal(tot_u.cpu().numpy(), full["used_blocks"])
    dec = torch.full((3, 2), 9, dtype=torch.int32, device="cuda")
    sched.scale_decide(tb, tot_c, tot_u, dec, min_samples=1, eps_in=kw["eps_in"], eps_wait=kw["eps_wait"])
    assert np.array_equal(dec.cpu().numpy(), full["decision"])
    seen = set()
    for k in range(40):
        cnt = rng.integers(0, 60, (3, 4)).astype(np.int64); cnt[:, 3] = cnt[:, 2] * rng.integers(0, 1 << 15, 3)
        used = (rng.integers(0, 400, R) * rng.integers(0, 2, R)).astype(np.int64)
        kk = dict(min_samples=int(rng.integers(0, 30)), eps_out=(int(rng.integers(1, 20)), 10), eps_in=(int(rng.integers(1, 20)), 10),
                  eps_wait=(1, int(rng.integers(1, 8))))
        sched.scale_decide(tb, torch.from_numpy(cnt).cuda(), torch.from_numpy(used).cuda(), dec, **kk)
        want = oracle.scale_decide(wl, tb_np, cnt, used, **kk)
        assert np.array_equal(dec.cpu().numpy(), want), (k, dec.cpu().numpy(), want)
        seen |= set(want[:, 0].tolist())
    assert seen == {-1, 0, 1} and sched.status() != 0      # the shards held rows with ids out of range too
    sched.close()


@pytest.mark.parametrize("n", [770, 1024, 1025, 2048, 2049, 4096, 4097, 8192, 8193, 12_345, 16_384])
def test_medium_segment_sizes_around_the_register_sort_shapes(n):
    # one replica whose rows are nearly all active: 1, 2, 4, 8 or 16 items per thread in the sorting network, at
    # and around each boundary; ids in row order (ordered step) and permuted (inactive rows sorted too), ties
    for permute, tie in ((False, False), (True, True)):
        wl = gen.random_table(n, n, 1, modes=(gen.COLOCATED,), permute_ids=permute, tie_heavy=tie, inflight=0.2, done=0.0, future=0.0)
        assert_step_parity(wl, steps=2, commit=True)
    wl = gen.random_table(n + 1, n, 1, modes=(gen.DECODE,), permute_ids=False, inflight=0.6, done=0.01, future=0.01, batch_cap=40)
    assert_step_parity(wl, steps=2, commit=True)
    wl = gen.random_table(n + 2, n, 1, modes=(gen.COLOCATED,), permute_ids=True, inflight=0.05, done=0.45, future=0.45)     # mostly inactive
    assert_step_parity(wl, steps=1, commit=True)


@pytest.mark.parametrize("n", [3000, 16384])
def test_medium_replica_with_crowded_and_outlying_slacks(n):
    # The distribution sort of a larger replica spreads a class over its bins by slack: queued requests that arrived
    # within nanoseconds of each other crowd one bin (the sorting network takes over), a few far outliers stretch the
    # range, and arrivals outside the sampled range go to the end bins.  Ids in row order: an ordered step.
    wl = gen.random_table(900 + n % 7, n, 1, modes=(gen.COLOCATED,), permute_ids=False, inflight=0.3, done=0.0, future=0.0)
    t = wl.table
    q = np.nonzero(t["state"] == gen.QUEUED)[0]
    now = int(wl.now[0])
    t["arrival_ns"][q] = now - 10**9 - (np.arange(len(q)) % 1500)            # crowded: 1500 distinct slacks a nanosecond apart
    t["arrival_ns"][q[::97]] = now - 10**9 * (2 + np.arange(len(q[::97])) % 300)   # outliers up to 300 s back
    t["arrival_ns"][q[5]] = now - 500 * 10**9
    assert_step_parity(wl, steps=2, commit=True)
    wl = gen.random_table(901 + n % 7, n, 1, modes=(gen.DECODE,), permute_ids=False, inflight=0.7, done=0.0, future=0.0)
    t = wl.table
    r = np.nonzero(t["state"] == gen.RUNNING)[0]
    t["last_token_ns"][r] = int(wl.now[0]) - (np.arange(len(r)) % 7)         # requests in flight with seven distinct slacks per class
    assert_step_parity(wl, steps=2, commit=True)


@pytest.mark.parametrize("grouped", [False, True])
def test_idle_replica_with_a_long_list_of_inactive_rows_jumps_to_its_next_arrival(grouped):
    # An ordered step (ids in row order) leaves lists of more than 2048 inactive rows to the end of the kernel; an idle
    # replica that commits must still find the earliest arrival among them for its clock jump.  Replica 0: nothing
    # in flight, nothing arrived, 3000 finished requests and a few that arrive later; replica 1: busy; replica 2:
    # idle with a short list.  Interleaved rows and rows grouped by replica; small and whole-block replicas.
    for n_busy in (300, 2500):
        wl = gen.random_table(70 + n_busy % 7, 3000 + n_busy + 200, 3, modes=(gen.COLOCATED, gen.COLOCATED, gen.DECODE),
                              permute_ids=False, grouped=grouped, inflight=0.4, done=0.0, future=0.0)
        wl.replicas[:, 0] = (gen.COLOCATED, gen.COLOCATED, gen.DECODE)
        t = wl.table
        now = int(wl.now.max())
        wl.now[:] = now
        wl.maturity[:] = now - 1
        rid = np.zeros(wl.n_rows, np.int32)
        rid[3000:3000 + n_busy] = 1
        rid[3000 + n_busy:] = 2
        if not grouped:
            rid = rid[np.random.default_rng(n_busy).permutation(wl.n_rows)]
        t["replica_id"][:] = rid
        r0 = np.nonzero(rid == 0)[0]
        t["state"][r0] = gen.DONE
        late = r0[::211]
        t["state"][late] = gen.QUEUED
        t["arrival_ns"][late] = now + 5 * MS + (np.arange(late.size) * 7919) % (50 * MS)
        r2 = np.nonzero(rid == 2)[0]
        t["state"][r2] = gen.DONE
        t["state"][r2[:3]] = gen.QUEUED
        t["arrival_ns"][r2[:3]] = now + 9 * MS
        assert_step_parity(wl, steps=3, commit=True)


@pytest.mark.parametrize("m", [16, 64, 2048])
def test_simulator_every_row_live_at_once(m):
    # The queue and the running batch share one list array of the trace's length (a multiple of 16 here, so the array
    # has no spare entry): every request arrives at time 0, prompts are short so that several are admitted per
    # iteration, outputs are long so that nothing finishes while the queue drains, then they finish in bunches.
    rng = np.random.default_rng(m)
    rows = [dict(prompt_len=int(rng.integers(1, 40)), output_len=int(rng.integers(150, 170)), arrival_ns=0, req_id=i,
                 class_id=int(rng.integers(0, 2))) for i in range(m)]
    late = np.sort(rng.integers(0, 40 * MS, m))                  # a second trace (rows in arrival order), short outputs: places free up all the time
    rows += [dict(prompt_len=int(rng.integers(1, 40)), output_len=int(rng.integers(2, 5)), arrival_ns=int(late[i]), req_id=m + i)
             for i in range(m)]
    wl = make_wl(rows, [(200 * MS, 30 * MS, 0), (1000 * MS, 50 * MS, 1)], replicas=[(gen.COLOCATED, 8192, 0)] * 2, now=[0, 0],
                 maturity=[0, 0], trace_off=[0, m, 2 * m], sim_iters=600)
    assert_sim_parity(wl)
