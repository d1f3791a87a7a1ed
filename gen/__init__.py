"""Seeded synthetic input generators (no scheduler arithmetic lives here)."""
from .workloads import *  # noqa: F401,F403
from .workloads import Workload, by_name  # noqa: F401
