"""Seeded synthetic inputs (weights, tokens, frozen calibration state) shared by the
oracle-side tests and the CUDA-side tests/benchmark.  Holds no arithmetic of the path."""
from .generate import *  # noqa: F401,F403
from . import generate  # noqa: F401
