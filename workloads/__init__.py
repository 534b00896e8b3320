"""Seeded synthetic workloads: input recipes for the tests, the smoke check and the benchmark.

Not part of the library.  Nothing here is imported by `paper_2507_19766_b200` or by `oracle`; the
recipes only produce the arrays both sides are then given (hidden states, head weight, targets,
recorded log-probs, policy versions, advantages, sequence offsets).
"""
from . import synth  # noqa: F401
