"""The C-ABI library loads and exports every symbol include/hfx.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

import paper_2508_15919_b200 as hfx

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    src = open(os.path.join(ROOT, "include", "hfx.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(hfx_[a-z_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    from paper_2508_15919_b200 import build
    build.build()
    lib = ctypes.CDLL(hfx.library_path())
    names = _declared_symbols()
    assert {"hfx_sched_create", "hfx_sched_step", "hfx_sim_run", "hfx_sched_status", "hfx_sched_destroy",
            "hfx_strerror"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(hfx.EXPORTED_SYMBOLS) == set(names)


def test_struct_layouts_match_the_header():
    from paper_2508_15919_b200 import binding as b
    assert ctypes.sizeof(b._Model) == 48 and ctypes.sizeof(b._SloClass) == 24
    assert ctypes.sizeof(b._ReplicaCfg) == 12 and ctypes.sizeof(b._Options) == 16
    assert ctypes.sizeof(b._Table) == 8 + 12 * 8 and ctypes.sizeof(b._ReplicaState) == 16
    assert ctypes.sizeof(b._StepOut) == 15 * 8 and ctypes.sizeof(b._SimOut) == 9 * 8
    assert ctypes.sizeof(b._Profile) == 224 and ctypes.sizeof(b._SloWindow) == 40 and ctypes.sizeof(b._SloBounds) == 48 and ctypes.sizeof(b._DispatchOut) == 13 * 8 and ctypes.sizeof(b._ScaleParams) == 40
    # field order of the header's structs
    src = open(os.path.join(ROOT, "include", "hfx.h")).read()
    for struct, cls in (("hfx_table", b._Table), ("hfx_step_out", b._StepOut), ("hfx_sim_out", b._SimOut),
                        ("hfx_dispatch_out", b._DispatchOut), ("hfx_slo_window", b._SloWindow), ("hfx_slo_bounds", b._SloBounds)):
        body = re.search(r"typedef struct %s \{(.*?)\} %s;" % (struct, struct), src, flags=re.S).group(1)
        body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
        fields = re.findall(r"\*?\s*(\w+)\s*;", body)
        assert fields == [f[0] for f in cls._fields_], struct


def test_strerror_and_argument_checks_without_a_device():
    lib = hfx.load_library()
    assert lib.hfx_strerror(0) == b"ok" and b"aligned" in lib.hfx_strerror(-2)
    assert lib.hfx_strerror(-99) == b"unknown error"
    assert lib.hfx_kernel_name(3) == b"k_regroup_atomic" and lib.hfx_kernel_name(4) == b"k_replicas" and lib.hfx_kernel_name(9) == b"k_front" and lib.hfx_kernel_name(10) == b"k_dispatch" and lib.hfx_kernel_name(11) == b"k_slo_map" and lib.hfx_kernel_name(12) == b"k_pd_migrate" and lib.hfx_kernel_name(13) == b"k_attainment" and lib.hfx_kernel_name(14) is None
    import torch
    if not torch.cuda.is_available():
        # no device: the product path fails loudly, it never falls back to the CPU
        with pytest.raises(hfx.HfxError) as e:
            hfx.Scheduler((1, 1, 0, 1, 1, 0), [(1, 1, 0)], [(0, 16, 0)], 16)
        assert e.value.code == -4
    # out-of-domain configuration is rejected before any CUDA call
    for bad in [dict(model=(-1, 1, 0, 1, 1, 0)), dict(classes=[(1, 1, 63)]), dict(replicas=[(0, 0, 0)]),
                dict(max_rows=0), dict(budget_mode=7)]:
        kw = dict(model=(1, 1, 0, 1, 1, 0), classes=[(1, 1, 0)], replicas=[(0, 16, 0)], max_rows=16)
        kw.update(bad)
        with pytest.raises(hfx.HfxError) as e:
            hfx.Scheduler(**kw)
        assert e.value.code == -1


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2508_15919_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                txt = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in txt.lower(), f
    txt = open(os.path.join(ROOT, "oracle", "hfx_oracle.c")).read() + open(os.path.join(ROOT, "oracle", "__init__.py")).read()
    assert "hfx.h" not in txt and "paper_2508_15919_b200" not in txt
