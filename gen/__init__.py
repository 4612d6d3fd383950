"""Seeded synthetic inputs shared by the CUDA library's tests, the benchmark and the CPU oracle."""
from . import rng, workloads  # noqa: F401
