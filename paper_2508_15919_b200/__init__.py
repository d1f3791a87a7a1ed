"""B200-native hot path of a multi-SLO LLM-serving scheduler (budget estimation, slack,
priority order, budgeted admission, trace-driven simulation) as a C-ABI CUDA library.

This package is a thin binding: it marshals torch device tensors into the C structs of
include/hfx.h and calls the library.  Every step of the path runs in the CUDA kernels;
there is no CPU fallback, and importing the binding fails loudly if the library is missing.
"""
from .binding import (count_rows_noalloc, NOALLOC_MAX_REPLICAS, HfxError, Scheduler, StepOut, SimOut, DispatchOut, Fleet, DeviceTable, load_library, library_path,
                      EXPORTED_SYMBOLS, COMMIT, QUEUED, RUNNING, DONE, REJECTED, COLOCATED, PREFILL, DECODE,
                      BUDGET_SAFE, BUDGET_CAP_ONLY, ST_BAD_REPLICA, ST_BAD_CLASS, ST_BAD_LEN, ST_TIMEOUT)

__all__ = ["HfxError", "Scheduler", "StepOut", "SimOut", "DispatchOut", "Fleet", "DeviceTable", "load_library", "library_path",
           "EXPORTED_SYMBOLS", "COMMIT"]
