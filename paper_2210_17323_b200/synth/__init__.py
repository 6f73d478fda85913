"""Seeded synthetic inputs shared by the CUDA path's tests/bench and the CPU oracle's tests.

Nothing here implements any step of the quantization method.
"""
from . import generator, workloads  # noqa: F401
