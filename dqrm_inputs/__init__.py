"""Seeded synthetic input generators shared by the oracle-side tests and the CUDA-side
harness.  Holds no arithmetic of the quantisation method."""
from . import rng, workloads  # noqa: F401
from .workloads import Workload  # noqa: F401
