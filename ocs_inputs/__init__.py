"""Seeded synthetic inputs shared by the CPU checker and the CUDA library's tests and bench."""
from . import prng, configs  # noqa: F401
