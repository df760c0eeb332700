"""Seeded synthetic input generators shared by the tests and the benchmark (inputs only)."""
from .workloads import *  # noqa: F401,F403
