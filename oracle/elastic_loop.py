"""Test infrastructure, like the rest of this package.  The scaling loop both test suites drive: per tick of
the global clock, the instances advance up to the tick (committed steps under a horizon), the Scaler inspects queue and instances, its decisions are carried out, the
dispatcher serves the instances that are due and the dispatched requests are bound.  This module runs it on the
oracle; the GPU parity test runs the same sequence through the library and compares after every call."""
from . import dispatch, dispatch_bind, scale_apply, scale_tick, step

MS = 1_000_000
TICK = 50 * MS
SUBSTEPS = 6
COLD = (300 * MS, 300 * MS, 300 * MS)
SCALE_KW = dict(window=2000 * MS, min_samples=10)


def oracle_round(wl, fleet, k):
    now_g = (k + 1) * TICK
    wl.meta["horizon"] = now_g
    status = 0
    for _ in range(SUBSTEPS):
        status |= step(wl, commit=True)["status"]
    t = scale_tick(wl, now_g, fleet["total_blocks"], **SCALE_KW)
    cost = scale_apply(wl, now_g, t["decision"], t["used_blocks"], COLD, fleet)
    step_mat = wl.maturity
    wl.maturity = fleet["due"]
    d = dispatch(wl, now_g)
    wl.maturity = step_mat
    dispatch_bind(wl, now_g, d)
    return dict(now=now_g, tick=t, cost=cost, dispatch=d, status=status | t["status"] | d["status"])
