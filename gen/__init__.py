"""Seeded synthetic inputs for the cached-MoE-layer path.

This package only produces data (weights, hidden states, router biases, workload
shapes).  It holds none of the method's arithmetic: no routing, no cache policy,
no FFN.  Both the CPU oracle's tests and the CUDA path's tests read their inputs
from here, and neither side's code is imported by this package.
"""
from .inputs import *  # noqa: F401,F403
