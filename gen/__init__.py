"""Seeded synthetic input generators.

This package is the only code shared by the CPU oracle's tests and the CUDA library's
tests and benchmark.  It produces index arrays, coordinates, features, weights and
cotangents; it contains none of the arithmetic of the message-passing method itself.
"""
from .workloads import *  # noqa: F401,F403
