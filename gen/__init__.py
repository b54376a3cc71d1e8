"""Seeded synthetic inputs (graphs, raw placement states, weights).

Shared by the CPU checker's tests and the CUDA library's tests and benchmark;
contains no part of the policy's arithmetic.
"""
from . import configs, graphs, states  # noqa: F401
