"""B200-native evolution-strategy generation (ask -> rollout -> tell) behind a C-ABI.

``binding`` is the thin ctypes layer over ``libevo.so``; ``workloads`` holds the synthetic
configurations and seeded input generators; ``build`` compiles the CUDA sources.
"""
from .binding import EvoConfig, EvoError, Solver, load_library  # noqa: F401
from . import workloads  # noqa: F401
