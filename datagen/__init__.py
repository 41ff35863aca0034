"""Seeded synthetic inputs shared by the oracle's tests and the CUDA path's tests/bench."""
from . import rng, stacks  # noqa: F401
from .stacks import CONFIGS, StackConfig  # noqa: F401
