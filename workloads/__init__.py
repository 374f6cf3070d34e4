"""Seeded synthetic workloads shared by the CPU oracle's tests and the CUDA path's tests/bench."""
from .configs import CONFIGS, Config, Workload, TINY, MID, HEADLINE, RAGGED, PREFILL, PREFILL_SMALL  # noqa: F401
from . import generator  # noqa: F401
