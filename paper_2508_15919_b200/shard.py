"""Host-side sharding of a request table across ranks (one process per GPU).

Replicas are independent units of the scheduler step, so a table is split by contiguous replica
ranges and every rank runs the whole path on its own rows; no collective touches the data path.
The only communication is the reduction of timings and counts for reporting -- and, for a Scaler that
watches instances on several GPUs, the sum of the tick's counters (scaler_exchange).
"""
from __future__ import annotations

from typing import Dict, Tuple

import numpy as np


def replica_range(n_replicas: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous, balanced range [lo, hi) of replicas owned by `rank`."""
    base, extra = divmod(n_replicas, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_columns(cols: Dict[str, np.ndarray], lo: int, hi: int) -> Tuple[Dict[str, np.ndarray], np.ndarray]:
    """Rows whose replica_id lies in [lo, hi), in their original order, with replica ids made
    local (id - lo).  Also returns the selected global row indices."""
    rid = cols["replica_id"]
    rows = np.nonzero((rid >= lo) & (rid < hi))[0]
    out = {k: np.ascontiguousarray(v[rows]) for k, v in cols.items()}
    out["replica_id"] = (out["replica_id"] - lo).astype(np.int32)
    return out, rows


def reduce_report(step_ms: float, rows: int, group=None) -> Tuple[float, int]:
    """Max step time and total rows over all ranks (the whole-job throughput is rows / time)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return step_ms, rows
    t = torch.tensor([step_ms], dtype=torch.float64)
    r = torch.tensor([rows], dtype=torch.int64)
    if dist.get_backend(group) == "nccl":
        t, r = t.cuda(), r.cuda()
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    dist.all_reduce(r, op=dist.ReduceOp.SUM, group=group)
    return float(t.item()), int(r.item())


def scaler_exchange(counts, used_blocks, group=None) -> None:
    """Sum, in place and over all ranks, what hfx_scale_tick counted on each rank's shard of the table (counts
    int64 [3, 4]; used_blocks int64 [n_replicas] with global instance ids, zero for instances whose rows live on
    another rank).  Afterwards hfx_scale_decide gives the same decision on every rank.  Integer sums: the order
    of the reduction cannot change the result.  CPU tensors go over gloo, CUDA tensors over NCCL."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return
    dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(used_blocks, op=dist.ReduceOp.SUM, group=group)
