"""Seeded synthetic inputs for the MoE layer (shared by the CPU checker's tests and the GPU path)."""
from . import rng, workloads  # noqa: F401
