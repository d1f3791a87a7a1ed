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
