"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle's callers.
Holds no part of the method's arithmetic."""
from . import configs, graphs, tensors  # noqa: F401
