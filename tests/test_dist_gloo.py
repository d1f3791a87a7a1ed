"""Sharding across ranks on CPU (gloo, world size 2): replica ranges partition the table, every rank's
shard gives the same per-request and per-replica results as the full table (checked with the oracle:
the path needs no collective), and the report reduces time by max and rows by sum."""
import os
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    import gen
    import oracle
    from paper_2508_15919_b200 import shard
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = gen.config4(seed=9, R=13, n=6000, steps=2)
        full = oracle.step(wl.copy())
        lo, hi = shard.replica_range(wl.n_replicas, world, rank)
        cols, rows = shard.shard_columns(wl.table, lo, hi)
        part = wl.copy()
        part.table = cols
        part.replicas = wl.replicas[lo:hi].copy(); part.now = wl.now[lo:hi].copy(); part.maturity = wl.maturity[lo:hi].copy()
        o = oracle.step(part)
        ok = True
        for k in ("slack", "admit", "pred_ttft", "pred_tpot"):
            ok &= np.array_equal(o[k], full[k][rows])
        for k in ("budget", "adm_cost", "adm_count", "maturity_next", "n_run", "sum_kv"):
            ok &= np.array_equal(o[k], full[k][lo:hi])
        # the order of a shard is the full order restricted to its replicas
        seg = full["seg_off"]
        ok &= np.array_equal(rows[o["order"]], full["order"][seg[lo]:seg[hi]])
        t, r = shard.reduce_report(1.0 + rank, int(rows.size))
        q.put((rank, bool(ok), lo, hi, int(rows.size), t, r))
    finally:
        dist.destroy_process_group()


def _scaler_worker(rank, world, port, q):
    # a Scaler over a table whose rows live on two ranks: every rank counts its own rows (instances of its replica
    # range, global ids; the global queue split by row parity), the counters are summed, every rank decides
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch
    import torch.distributed as dist
    import gen
    import oracle
    from paper_2508_15919_b200 import shard
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        SEC = 1_000_000_000
        rng = np.random.default_rng(5)
        wl = gen.random_table(5, 20_000, 11, modes=(gen.COLOCATED, gen.PREFILL, gen.DECODE), future=0.1, done=0.4)
        wl.table["finish_ns"][:] = wl.now.max() - rng.integers(0, 3 * SEC, wl.n_rows)
        wl.table["replica_id"][::5] = -1
        now = int(wl.now.max())
        tb = rng.integers(0, 900, 11) * (rng.random(11) < 0.8)
        kw = dict(window=2 * SEC, min_samples=1, eps_in=(1, 50), eps_wait=(50, 1))
        full = oracle.scale_tick(wl, now, tb, **kw)
        lo, hi = shard.replica_range(wl.n_replicas, world, rank)
        rid = wl.table["replica_id"]
        mine = ((rid >= lo) & (rid < hi)) | ((rid == -1) & (np.arange(wl.n_rows) % world == rank))
        mine |= ((rid < -1) | (rid >= wl.n_replicas)) & (rank == 0)
        part = wl.copy()
        part.table = {k: np.ascontiguousarray(v[mine]) for k, v in wl.table.items()}
        o = oracle.scale_tick(part, now, tb, **kw)
        counts = torch.from_numpy(o["counts"].copy()); used = torch.from_numpy(o["used_blocks"].copy())
        shard.scaler_exchange(counts, used)
        ok = np.array_equal(counts.numpy(), full["counts"]) and np.array_equal(used.numpy(), full["used_blocks"])
        dec = oracle.scale_decide(wl, tb, counts.numpy(), used.numpy(), **kw)
        ok &= np.array_equal(dec, full["decision"])
        partial_differs = not np.array_equal(o["counts"], full["counts"])
        q.put((rank, bool(ok), bool(partial_differs), dec.tolist()))
    finally:
        dist.destroy_process_group()


def test_two_rank_scaler_counters_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_scaler_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert all(r[1] and r[2] for r in res)
    assert res[0][3] == res[1][3]                  # the same decision on every rank


def test_two_rank_sharding_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert all(r[1] for r in res)
    assert res[0][2] == 0 and res[0][3] == res[1][2] and res[1][3] == 13          # ranges tile [0, R)
    assert res[0][4] + res[1][4] == 6000
    assert all(r[5] == 2.0 and r[6] == 6000 for r in res)                          # max time, total rows


def test_replica_range_is_balanced():
    from paper_2508_15919_b200 import shard
    for R in (1, 7, 8, 1024, 4097):
        for world in (1, 2, 3, 8):
            spans = [shard.replica_range(R, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == R
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
