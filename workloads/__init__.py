"""Seeded synthetic inputs and workload shapes.

This package holds no arithmetic of the compression method itself: it only
draws random inputs (weights by their generating factors, hidden states,
queries, context lengths, page orders) and names the workload shapes.  Both the
CPU oracle's tests and the CUDA path's tests/bench take their inputs from here.
"""
from . import synth  # noqa: F401
from .synth import CONFIGS, Shape  # noqa: F401
