"""Bounded-cache MoE decode step for one B200: CUDA kernels behind a C ABI (libremoe.so).

``binding`` marshals arguments to the C entry points (same names); ``loader`` places a
seeded synthetic workload in pinned host memory and registers it with a stack.
"""
from . import binding  # noqa: F401
from .binding import Stack, RemoeError, lib  # noqa: F401
