"""Seeded synthetic inputs shared by the CUDA path and the CPU oracle (data only)."""
from . import configs, data, rng  # noqa: F401
