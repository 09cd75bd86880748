"""Seeded synthetic inputs shared by the CUDA library's callers and the CPU oracle's callers."""
from . import rng, workloads  # noqa: F401
