#!/usr/bin/env python
"""Benchmark of the scheduler hot path: requests scheduled per second per hfx_sched_step on the
1,048,576-request / 1024-replica shared-queue workload (rows interleaved across replicas, committed
steps with in-flight state carried over), plus simulated scheduler iterations per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-sim] [--no-cpu]

One "step" is one hfx_sched_step(COMMIT) over the whole table: per-replica aggregates, E_d, safe
budget, per-row slack and key, per-replica sort, segmented-scan admission, maturity update, commit.
Steps are timed one by one with CUDA events on the launching stream; between steps L2 is flushed by
writing a 256 MiB buffer (outside the events), and the table is restored to its initial state every
10 steps (outside the events) so that the workload stays the one the configuration names.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import gen  # noqa: E402

METRIC = "requests_scheduled_per_sec_per_hfx_sched_step"
UNIT = "requests/s"
ALGO_BYTES_PER_ROW = 51            # 38 B read (incl. priority weight) + 13 B written (slack 8, order 4, admit 1) per row and step
# what each kernel itself moves of those bytes (they add up to the step's 51): the tile front end reads the
# columns and writes slack and admit, the replica kernel writes the order
KERNEL_BYTES_PER_ROW = {"k_front": 47, "k_replicas": 4, "k_count": 22, "k_offsets": 0, "k_regroup_atomic": 25}
STEPS_PER_EPISODE = 10
KERNEL_SOURCES = ["hfx_front.cu", "hfx_segment.cu", "hfx_step.cu", "hfx_regroup.cu", "hfx_rows.cuh", "hfx_internal.cuh"]
PROFILE = os.path.join(ROOT, "profiles", "step_config4_k_front_k_replicas.md")


def _kernel_source_hash():
    """Identifies the kernels a profile was taken on: a hash of the step's CUDA sources."""
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2508_15919_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def _profile_counters():
    """Per-kernel ncu counters of the committed profile summary (lines `<!-- bench: kernel=.. key=value .. -->`),
    or {} when the summary was taken on other kernel sources than the ones in the tree."""
    import re
    out = {}
    if not os.path.exists(PROFILE):
        return out
    src = _kernel_source_hash()
    with open(PROFILE) as f:
        for m in re.finditer(r"<!-- bench: (.*?) -->", f.read()):
            kv = dict(x.split("=", 1) for x in m.group(1).split())
            if kv.get("src") != src:
                continue
            out[kv["kernel"]] = {"traffic": float(kv["dram_bytes"]), "warp_inst": float(kv["warp_inst"]), "rows": float(kv["rows"])}
    return out


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _workload(rank: int, args):
    if args.workload == "config2":        # (profiling aid: the bench line is config 4)
        return gen.config2(seed=2 + rank, inflight=0.02)
    if args.workload == "config3":
        return gen.config3(seed=3 + rank)
    return gen.config4(seed=4 + rank, R=args.replicas, n=args.rows, steps=STEPS_PER_EPISODE)


def _workload_name(n, R, which="config4"):
    if which != "config4":
        return "%s: %d requests over %d replicas (see gen/workloads.py); not the benchmark configuration" % (which, n, R)
    return ("config4: shared queue, %d requests over %d replicas (rows interleaved), 5 SLO tiers, priority "
            "weights, Pareto prompts, committed steps with in-flight state carried over" % (n, R))


def run_reference(args):
    """The oracle, as it stands, on the host cores: one step = one oracle step (with commit) over
    the same table.  Rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    wl0 = _workload(0, args)
    wl = wl0.copy()
    times = []
    for s in range(args.warmup + args.steps):
        if s % STEPS_PER_EPISODE == 0:
            wl = wl0.copy()
        t0 = time.perf_counter()
        oracle.step(wl, commit=True)
        dt = time.perf_counter() - t0
        if s >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    val = wl0.n_rows / (ms * 1e-3)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int64", "data": "synthetic",
            "config": {"workload": _workload_name(wl0.n_rows, wl0.n_replicas),
                       "note": "CPU oracle (plain single-threaded C), one oracle step per bench step, full table"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": "%d full-table committed steps of the %d-row workload" % (args.steps, wl0.n_rows)},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_gpu(args):
    import torch
    import torch.distributed as dist
    import paper_2508_15919_b200 as hfx

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the scheduler library has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    hfx.load_library()
    wl = _workload(rank, args)
    n, R = wl.n_rows, wl.n_replicas
    sched = hfx.Scheduler(wl.model, wl.classes, wl.replicas, n, budget_mode=wl.budget_mode, weight_max=wl.weight_max)
    if args.front == "fallback":
        sched.set_fused_front(False)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    init = {k: v.clone() for k, v in tab.cols.items()}
    now0 = torch.from_numpy(wl.now).cuda(); mat0 = torch.from_numpy(wl.maturity).cuda()
    now = now0.clone(); mat = mat0.clone()
    out = hfx.StepOut(n, R, optional=False)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def restore():
        for k in ("state", "gen", "first_token_ns", "last_token_ns", "finish_ns"):
            tab.cols[k].copy_(init[k])
        now.copy_(now0); mat.copy_(mat0)

    def timed_pass(steps, warmup, profile=False):
        """Per-step device times (ms) of `steps` steps after `warmup` untimed ones."""
        evs = []
        sched.set_profiling(False)
        for s in range(warmup + steps):
            if s == warmup:
                sched.get_profile()
                sched.set_profiling(profile)
            if s % STEPS_PER_EPISODE == 0:
                restore()
            flush.fill_(s & 0xff)                       # L2 flush, outside the events
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            sched.step(tab, now, mat, out, commit=True)
            b.record(stream)
            if s >= warmup:
                evs.append((a, b))
        torch.cuda.synchronize()
        sched.set_profiling(False)
        return [a.elapsed_time(b) for a, b in evs]

    # ---- device-resident timing: K steps bracketed by barrier + synchronize -----------------------
    timed_pass(0, max(args.warmup, 3))
    clocks = ClockSampler(local)
    barrier()
    if rank == 0:
        clocks.start()
    launches0 = sched.launch_count()
    t_wall0 = time.perf_counter()
    times = timed_pass(args.steps, 0)
    barrier()
    wall = time.perf_counter() - t_wall0
    launches = sched.launch_count() - launches0
    clk = clocks.stop() if rank == 0 else None
    status = sched.status()
    step_ms = float(np.sum(times)) / args.steps
    t = torch.tensor([step_ms], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    step_ms_max = float(t.item())
    value = world * n / (step_ms_max * 1e-3)

    # ---- per-kernel times over the same K steps (events inside the library) ------------------------
    timed_pass(args.steps, 1, profile=True)
    prof = sched.get_profile()

    # ---- end to end: host buffers in, results out, through the C ABI --------------------------------
    in_cols = ["replica_id", "class_id", "state", "prompt_len", "output_len", "gen", "arrival_ns", "first_token_ns",
               "req_id", "weight"]
    pinned = {k: init[k].cpu().pin_memory() for k in in_cols}
    pin_now = now0.cpu().pin_memory(); pin_mat = mat0.cpu().pin_memory()
    res_host = {k: torch.empty_like(out.t[k], device="cpu").pin_memory()
                for k in ("admit", "order", "seg_off", "budget", "adm_cost", "adm_count", "maturity_next")}
    h2d = sum(v.numel() * v.element_size() for v in pinned.values()) + 2 * pin_now.numel() * 8
    d2h = sum(v.numel() * v.element_size() for v in res_host.values())

    def e2e_step():
        for k in in_cols:
            tab.cols[k].copy_(pinned[k], non_blocking=True)
        now.copy_(pin_now, non_blocking=True); mat.copy_(pin_mat, non_blocking=True)
        sched.step(tab, now, mat, out, commit=True)
        for k, v in res_host.items():
            v.copy_(out.t[k], non_blocking=True)

    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(3):
        e2e_step()
    barrier()
    e_evs = []
    for _ in range(e2e_steps):
        flush.fill_(1)
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record(stream); e2e_step(); b.record(stream)
        e_evs.append((a, b))
    barrier()
    e2e_ms = float(np.mean([a.elapsed_time(b) for a, b in e_evs]))
    t = torch.tensor([e2e_ms], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    e2e_ms_max = float(t.item())
    e2e_value = world * n / (e2e_ms_max * 1e-3)

    # ---- simulator: scheduler iterations per second (rank 0, outside the timed steps) --------------
    sim = None
    if rank == 0 and not args.no_sim:
        swl = gen.config5(traces=args.sim_traces, iters=args.sim_iters)
        ssched = hfx.Scheduler(swl.model, swl.classes, swl.replicas, swl.n_rows)
        stab = hfx.DeviceTable.from_numpy(swl.table)
        sout = hfx.SimOut(args.sim_traces)
        ssched.sim_run(stab, swl.trace_off, 50, sout)           # warm-up
        torch.cuda.synchronize()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record(stream); ssched.sim_run(stab, swl.trace_off, swl.sim_iters, sout); b.record(stream)
        torch.cuda.synchronize()
        sim_ms = a.elapsed_time(b)
        so = sout.to_numpy()
        iters_total = int(so["iters_executed"].sum())
        sim = {"workload": "config5: %d traces x 2048 requests, %d iterations" % (args.sim_traces, args.sim_iters),
               "sched_iters_per_sec": iters_total / (sim_ms * 1e-3), "ms": sim_ms, "iterations_executed": iters_total,
               "mean_attainment": float((so["attained"] / 2048.0).mean()), "status": ssched.status()}
        ssched.close()

    # ---- dispatching over the shared global queue of the same table (rank 0, outside the timed steps) --
    disp = None
    if rank == 0 and not args.no_dispatch:
        restore()
        dout = hfx.DispatchOut(n, R)
        now_g = int(wl.now[0])
        for _ in range(3):
            sched.dispatch_step(tab, now_g, mat0, dout)
        torch.cuda.synchronize()
        d_evs = []
        for _ in range(10):
            flush.fill_(3)
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(stream); sched.dispatch_step(tab, now_g, mat0, dout); b.record(stream)
            d_evs.append((a, b))
        torch.cuda.synchronize()
        d_ms = float(np.mean([a.elapsed_time(b) for a, b in d_evs]))
        dn = dout.to_numpy()
        disp = {"workload": "one hfx_dispatch_step over the same table: every matured instance takes its turn",
                "ms": d_ms, "requests_per_sec": n / (d_ms * 1e-3), "queue_length": int(dn["n_queue"][0]),
                "instances_matured": int(dn["n_mature"][0]), "requests_dispatched": int(dn["adm_count"].sum()),
                "status": sched.status()}
        if world == 1 and not args.no_cpu:
            import oracle
            oracle.build()
            t0 = time.perf_counter()
            k_d = 0
            while time.perf_counter() - t0 < 3.0:
                oracle.dispatch(wl, now_g)
                k_d += 1
            disp["cpu_oracle_ms"] = 1e3 * (time.perf_counter() - t0) / k_d
            disp["cpu_oracle_calls"] = k_d

    # ---- the disaggregated mode end to end: committed steps coupled by the hand-off (rank 0) ----------
    pd = None
    if rank == 0 and not args.no_pd:
        pw = gen.pd_pairs(7, 128, 8192, permute_ids=False)      # request ids in arrival order, as a front end assigns them
        psched = hfx.Scheduler(pw.model, pw.classes, pw.replicas, pw.n_rows)
        ptab = hfx.DeviceTable.from_numpy(pw.table)
        pnow = torch.from_numpy(pw.now.copy()).cuda(); pmat = torch.from_numpy(pw.maturity.copy()).cuda()
        ppair = torch.from_numpy(gen.pd_partner_table(128)).cuda()
        pout = hfx.StepOut(pw.n_rows, pw.n_replicas, optional=False)
        pmoved = torch.zeros(4, dtype=torch.int32, device="cuda")
        rounds_w, rounds_t = 10, 40
        moved_total = 0
        evs = []
        for k in range(rounds_w + rounds_t):
            flush.fill_(5)
            a = torch.cuda.Event(enable_timing=True); m = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            psched.step(ptab, pnow, pmat, pout, commit=True)
            m.record(stream)
            psched.pd_migrate(ptab, pnow, pmat, ppair, 2_000_000, 500, pmoved)
            b.record(stream)
            if k >= rounds_w:
                evs.append((a, m, b))
        torch.cuda.synchronize()
        step_ms_pd = float(np.mean([a.elapsed_time(m) for a, m, b in evs]))
        mig_ms = float(np.mean([m.elapsed_time(b) for a, m, b in evs]))
        pt = ptab.to_numpy()
        att = torch.zeros((len(pw.classes) + 1, 6), dtype=torch.int64, device="cuda")
        psched.attainment(ptab, att)
        att_tot = att.cpu().numpy()[-1]
        pd = {"workload": "128 P + 128 D instances, 1,048,576 requests, %d rounds of (committed step, hand-off)" % (rounds_w + rounds_t),
              "step_ms": step_ms_pd, "handoff_ms": mig_ms, "rounds_per_sec": 1e3 / (step_ms_pd + mig_ms),
              "handoff_gbs": 15 * pw.n_rows / (mig_ms * 1e-3) / 1e9,
              "requests_on_d_instances": int(np.count_nonzero(pt["replica_id"] >= 128)),
              "requests_finished": int(att_tot[1]), "requests_attained": int(att_tot[2]), "status": psched.status()}
        psched.close()

    # ---- the scaling loop: global queue, dispatcher, instances under a horizon, Scaler tick and its decisions ----
    elastic = None
    if rank == 0 and not args.no_elastic:
        ER, EN, TICK, SUB = 1024, 1 << 20, 50_000_000, 6
        ew = gen.elastic(11, ER, EN, rates=(800.0, 2400.0))       # about 14 requests/s saturate one instance
        esched = hfx.Scheduler(ew.model, ew.classes, ew.replicas, ew.n_rows)
        etab = hfx.DeviceTable.from_numpy(ew.table)
        efl = hfx.Fleet(gen.new_fleet([4096] * ER, range(64)))
        enow = torch.from_numpy(ew.now.copy()).cuda(); emat = torch.from_numpy(ew.maturity.copy()).cuda()
        eout = hfx.StepOut(EN, ER, optional=False); edout = hfx.DispatchOut(EN, ER)
        ecnt = torch.zeros((3, 4), dtype=torch.int64, device="cuda"); eused = torch.zeros(ER, dtype=torch.int64, device="cuda")
        edec = torch.zeros((3, 2), dtype=torch.int32, device="cuda"); ecost = torch.zeros(3, dtype=torch.int64, device="cuda")
        cold = [300_000_000] * 3
        rounds_all = max(3, args.elastic_rounds)
        rounds_w = min(20, rounds_all // 3); rounds_t = min(60, rounds_all - rounds_w)      # the rounds after the timed ones carry the fleet through two bursts
        evs, on_max = [], 0
        for k in range(rounds_all):
            now_g = (k + 1) * TICK
            flush.fill_(7)
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            esched.set_horizon(now_g)
            e[0].record(stream)
            for _ in range(SUB):
                esched.step(etab, enow, emat, eout, commit=True)
            e[1].record(stream)
            esched.scale_tick(etab, now_g, efl.t["total_blocks"], ecnt, eused, edec, window_ns=2_000_000_000)
            esched.scale_apply(now_g, edec, eused, cold, efl, enow, emat, ecost)
            e[2].record(stream)
            esched.dispatch_step(etab, now_g, efl.t["due"], edout)
            esched.dispatch_bind(etab, now_g, edout, enow)
            e[3].record(stream)
            if rounds_w <= k < rounds_w + rounds_t:
                evs.append(e)
            if k % 10 == 9:
                on_max = max(on_max, int((efl.t["inst_state"] != 0).sum().item()))
        torch.cuda.synchronize()
        seg = [float(np.mean([e[i].elapsed_time(e[i + 1]) for e in evs])) for i in range(3)]
        est = etab.to_numpy()
        eatt = torch.zeros((len(ew.classes) + 1, 6), dtype=torch.int64, device="cuda")
        esched.attainment(etab, eatt)
        eatt_tot = eatt.cpu().numpy()[-1]
        arrived = int(np.count_nonzero(ew.table["arrival_ns"] <= rounds_all * TICK))
        elastic = {"workload": "up to %d colocated instances (64 on at the start), a trace of %d requests in one global queue, its first %d rounds of a %d ms "
                               "tick (%d timed): %d committed steps under the horizon, Scaler tick + its decisions, dispatch + binding"
                               % (ER, EN, rounds_all, TICK // 1_000_000, rounds_t, SUB),
                   "steps_ms": seg[0], "scaler_ms": seg[1], "dispatch_ms": seg[2], "rounds_per_sec": 1e3 / sum(seg),
                   "instances_on_max": on_max, "instances_on_end": int((efl.t["inst_state"] != 0).sum().item()),
                   "cost_instance_seconds": float(ecost.cpu().numpy()[0]) / 1e9,
                   "requests_bound": int(np.count_nonzero(est["replica_id"] >= 0)),
                   "requests_arrived": arrived, "requests_finished": int(eatt_tot[1]), "requests_attained": int(eatt_tot[2]),
                   "status": esched.status()}
        esched.close()
        if world == 1 and not args.no_cpu:
            # the same round on the oracle, one host core (test infrastructure timed as a baseline, two rounds)
            import oracle
            oracle.build()
            from oracle import elastic_loop
            cw_e = ew.copy()
            cf = gen.new_fleet([4096] * ER, range(64))
            t0 = time.perf_counter()
            for k in range(2):
                elastic_loop.oracle_round(cw_e, cf, k)
            elastic["cpu_oracle_round_ms"] = 1e3 * (time.perf_counter() - t0) / 2

    # ---- the other step configurations (parity cases, not the benchmark line): time of one step each ----------
    others = None
    if rank == 0 and not args.no_other_configs:
        others = {}
        peak_o, _ = _peaks()
        perm4 = gen.config4()
        perm4.table["req_id"] = np.random.default_rng(1).permutation(perm4.n_rows).astype(np.int32)      # ids not in row order: the general path
        for name, ow in (("config1", gen.config1()), ("config2", gen.config2()), ("config3", gen.config3()),
                         ("config4_permuted_req_id", perm4)):
            osched = hfx.Scheduler(ow.model, ow.classes, ow.replicas, ow.n_rows, budget_mode=ow.budget_mode, weight_max=ow.weight_max)
            otab = hfx.DeviceTable.from_numpy(ow.table)
            onow = torch.from_numpy(ow.now.copy()).cuda(); omat = torch.from_numpy(ow.maturity.copy()).cuda()
            oout = hfx.StepOut(ow.n_rows, ow.n_replicas, optional=False)
            for _ in range(3):
                osched.step(otab, onow, omat, oout)
            torch.cuda.synchronize()
            oevs = []
            for _ in range(10):
                flush.fill_(9)
                a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
                a.record(stream); osched.step(otab, onow, omat, oout); b.record(stream)
                oevs.append((a, b))
            torch.cuda.synchronize()
            o_ms = float(np.mean([a.elapsed_time(b) for a, b in oevs]))
            osched.get_profile(); osched.set_profiling(True)
            for _ in range(5):
                osched.step(otab, onow, omat, oout)
            oprof = osched.get_profile()
            bpr = 51 if ow.weight_max > 0 else 47
            gbs = bpr * ow.n_rows / (o_ms * 1e-3) / 1e9
            others[name] = {"rows": ow.n_rows, "replicas": ow.n_replicas, "ms_per_step": o_ms,
                            "requests_per_sec": ow.n_rows / (o_ms * 1e-3),
                            "algorithmic_bytes_per_row": bpr, "algorithmic_gbs": gbs, "frac": gbs / peak_o,
                            "kernel_us": {k: 1e3 * v["ms"] / v["launches"] for k, v in oprof.items()},
                            "note": "one step without commit, L2 flushed before it" + ("; launch-latency bound at this size" if ow.n_rows < 100000 else ""),
                            "status": osched.status()}
            osched.close()
            del otab, oout

    # ---- CPU baseline: the oracle on a bounded sample, rank 0 at N = 1 only -----------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        oracle.build()
        cw = wl.copy()
        k_cpu = 0
        t0 = time.perf_counter()
        busy = 0.0
        while busy < 12.0:                       # about 12 s of oracle work: episodes of committed steps
            if k_cpu % STEPS_PER_EPISODE == 0:
                cw = wl.copy()
            t1 = time.perf_counter()
            oracle.step(cw, commit=True)
            busy += time.perf_counter() - t1
            k_cpu += 1
        cpu_s = busy / k_cpu
        cpu = {"value": n / cpu_s, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": "%d committed steps of the full %d-row table" % (k_cpu, n)}

    if rank == 0:
        peak, peak_kind = _peaks()
        counters = _profile_counters()
        roof = None
        if prof:
            step_bytes = ALGO_BYTES_PER_ROW * n
            step_gbs = step_bytes / (step_ms_max * 1e-3) / 1e9
            tot = sum(x["ms"] for x in prof.values())
            kern = {}
            for k, v in prof.items():
                ms_l = v["ms"] / v["launches"]
                bpr = KERNEL_BYTES_PER_ROW.get(k, 0)
                cnt = counters.get(k)
                kern[k] = {"ms_per_launch": ms_l, "launches": v["launches"], "share": v["ms"] / tot,
                           "algorithmic_bytes_per_row": bpr, "algorithmic_bytes_per_launch": bpr * n,
                           "achieved": bpr * n / (ms_l * 1e-3) / 1e9, "frac": bpr * n / (ms_l * 1e-3) / 1e9 / peak,
                           "traffic": cnt["traffic"] * n / cnt["rows"] if cnt else None,
                           "warp_instructions_per_row": cnt["warp_inst"] / cnt["rows"] if cnt else None}
            traffic = sum(kv["traffic"] for kv in kern.values()) if kern and all(kv["traffic"] is not None for kv in kern.values()) else None
            dom = max(prof.items(), key=lambda kv: kv[1]["ms"])[0]
            # the headline is the whole step: every kernel of it runs once per step, and their algorithmic bytes add up to the step's
            roof = {"bound": "hbm", "kernel": "hfx_sched_step = " + " + ".join(sorted(prof)), "dominant_kernel": dom,
                    "achieved": step_gbs, "peak": peak, "unit": "GB/s", "frac": step_gbs / peak, "peak_kind": "of " + peak_kind,
                    "frac_of_nominal_8TBs": step_gbs / 8000.0, "traffic": traffic,
                    "traffic_source": ("profiles/step_config4_k_front_k_replicas.md (ncu dram__bytes_read.sum + dram__bytes_write.sum, "
                                       "taken on these kernel sources: hash %s)" % _kernel_source_hash()) if traffic is not None
                                      else "none: the committed profile was taken on other kernel sources",
                    "algorithmic_bytes_per_launch": step_bytes, "ms_per_launch": step_ms_max,
                    "what_bounds_it": "instruction issue and dependent phases, not bytes: see warp_instructions_per_row and profiles/",
                    "kernels": kern,
                    "kernel_times_note": "per-kernel times come from event brackets inside the library in a second pass over the same steps; "
                                         "the brackets keep the second kernel from being set up while the first drains, so their sum exceeds ms_per_step"}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": step_ms_max, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "int64", "data": "synthetic",
                "config": {"workload": _workload_name(n, R, args.workload), "front_end": args.front,
                           "rows_per_gpu": n, "replicas_per_gpu": R, "parallelism": "replica shards, no collective",
                           "l2": "flushed between steps (256 MiB write, outside the per-step events)",
                           "episode": "table restored every %d steps, outside the events" % STEPS_PER_EPISODE,
                           "wall_s_timed_region": wall},
                "clocks": clk, "gpu_launches": launches, "device_status": status,
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "ms_per_step": e2e_ms_max},
                "roofline": roof, "cpu_baseline": cpu, "sim": sim, "dispatch": disp, "pd": pd, "elastic": elastic, "other_configs": others}
        print(json.dumps(line))
    sched.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="hfx", choices=["hfx", "reference"])
    ap.add_argument("--rows", type=int, default=1 << 20)
    ap.add_argument("--replicas", type=int, default=1024)
    ap.add_argument("--sim-traces", type=int, default=4096)
    ap.add_argument("--sim-iters", type=int, default=10000)
    ap.add_argument("--workload", default="config4", choices=["config4", "config2", "config3"],
                    help="step configuration to time (profiling aid; the benchmark line is config4)")
    ap.add_argument("--front", default="tile", choices=["tile", "fallback"], help="front end of the step (profiling aid)")
    ap.add_argument("--no-sim", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-dispatch", action="store_true")
    ap.add_argument("--no-pd", action="store_true")
    ap.add_argument("--no-elastic", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true")
    ap.add_argument("--elastic-rounds", type=int, default=600, help="rounds of the scaling loop (the first 20 warm up, the next 60 are timed)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
