"""CPU oracle for the candidate-evaluation step.  Test infrastructure only: the
tests, the smoke check and the benchmark's CPU-baseline leg are its only callers."""
from .oracle import *  # noqa: F401,F403
