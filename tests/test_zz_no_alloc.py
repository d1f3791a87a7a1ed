"""hfx_count_rows_noalloc against hfx_sched_step's seg_off (needs a GPU; collected last).

The entry point serves callers that may not allocate device memory (all of it belongs to a
framework's allocator, or an allocation's hidden synchronisation is unacceptable): its counters
sit in a fixed array inside the library.  Because that array keeps the previous call's contents,
the test makes two calls in a row on different tables and wants both exact."""
import numpy as np
import pytest
import torch

import gen
import paper_2508_15919_b200 as hfx

pytestmark = pytest.mark.gpu


def _seg_off_by_step(wl):
    sched = hfx.Scheduler(wl.model, wl.classes, wl.replicas, max(wl.n_rows, 1), budget_mode=wl.budget_mode,
                          weight_max=wl.weight_max)
    tab = hfx.DeviceTable.from_numpy(wl.table)
    now = torch.from_numpy(wl.now.copy()).cuda(); mat = torch.from_numpy(wl.maturity.copy()).cuda()
    out = hfx.StepOut(wl.n_rows, wl.n_replicas)
    sched.step(tab, now, mat, out)
    torch.cuda.synchronize()
    ref = out.t["seg_off"].cpu().numpy().copy()
    sched.close()
    return ref


def test_two_calls_in_a_row_match_the_step():
    first = gen.random_table(41, 50_003, 1000)
    first.table["replica_id"][::97] = 5000          # some rows bound to no replica
    second = gen.random_table(42, 777, 37)          # smaller: stale counters of the first call would show
    for wl in (first, second):
        ref = _seg_off_by_step(wl)
        rid = torch.from_numpy(wl.table["replica_id"]).cuda()
        seg = torch.full((wl.n_replicas + 1,), -7, dtype=torch.int32, device="cuda")
        bad = torch.zeros(1, dtype=torch.int32, device="cuda")
        hfx.count_rows_noalloc(rid, wl.n_replicas, seg, bad)
        torch.cuda.synchronize()
        assert np.array_equal(seg.cpu().numpy(), ref)
        # and against the definition: rows per replica, as an exclusive prefix
        rid_np = wl.table["replica_id"]
        valid = rid_np[(rid_np >= 0) & (rid_np < wl.n_replicas)]
        want = np.concatenate([[0], np.cumsum(np.bincount(valid, minlength=wl.n_replicas))]).astype(np.int32)
        assert np.array_equal(seg.cpu().numpy(), want)
        assert int(bad.item()) == int(((rid_np < 0) | (rid_np >= wl.n_replicas)).sum())


def test_limits_are_rejected():
    rid = torch.zeros(16, dtype=torch.int32, device="cuda")
    seg = torch.zeros(hfx.NOALLOC_MAX_REPLICAS + 2, dtype=torch.int32, device="cuda")
    hfx.count_rows_noalloc(rid, hfx.NOALLOC_MAX_REPLICAS, seg)
    torch.cuda.synchronize()
    assert seg[1].item() == 16 and seg[hfx.NOALLOC_MAX_REPLICAS].item() == 16
    with pytest.raises(hfx.HfxError) as e:
        hfx.count_rows_noalloc(rid, hfx.NOALLOC_MAX_REPLICAS + 1, torch.zeros(hfx.NOALLOC_MAX_REPLICAS + 2, dtype=torch.int32, device="cuda"))
    assert e.value.code == -3


def test_empty_table_and_misaligned_counter():
    # no rows: every offset is 0 (the kernels still clear what the previous call left)
    seg = torch.full((6,), -7, dtype=torch.int32, device="cuda")
    bad = torch.full((1,), 9, dtype=torch.int32, device="cuda")
    hfx.count_rows_noalloc(torch.zeros(0, dtype=torch.int32, device="cuda"), 5, seg, bad)
    torch.cuda.synchronize()
    assert seg.cpu().tolist() == [0] * 6 and int(bad.item()) == 0
    # a counter address that is not 4-byte aligned is an argument error; nothing is launched
    raw = torch.zeros(8, dtype=torch.uint8, device="cuda")
    rid = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(hfx.HfxError) as e:
        hfx.count_rows_noalloc(rid, 5, seg, raw[1:5])
    assert e.value.code == -2
