"""Seeded synthetic workloads (graphs, rollout patterns, inputs, weights).

Shared test data only: no arithmetic of the rollout method lives here.
"""
from . import data, graphs, rng  # noqa: F401
