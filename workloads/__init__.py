"""Seeded synthetic inputs shared by the oracle-side and the CUDA-side callers.

Holds shapes and random-number recipes only: none of the method's arithmetic.
"""
from .configs import CONFIGS, Config, get_config  # noqa: F401
