"""Seeded synthetic inputs shared by the CUDA library's tests, the benchmark and the CPU oracle."""
from .populations import *  # noqa: F401,F403
