"""Seeded synthetic input generators shared by the tests, the benchmark and the CPU oracle's callers.

Holds no tensor-algebra arithmetic; see `synth.configs` for the workload recipes.
"""
from .configs import Case, make, random_coo, random_dense, CONFIGS, BASE_SEED  # noqa: F401
