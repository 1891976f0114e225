"""CPU oracle of the cached MoE layer: test infrastructure, never on the product path.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package.
It imports nothing from the CUDA package.
"""
from .ref import *  # noqa: F401,F403
