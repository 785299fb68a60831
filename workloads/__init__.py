"""Seeded synthetic plan spaces (inputs only).

This package builds the problem descriptions that both the CUDA library and the CPU oracle are fed:
model / modeled-cluster / workload numbers, axis value lists and the seeded kernel-efficiency and
realization-overhead tables.  It contains none of the scoring arithmetic and imports neither side.
"""
from .configs import CONFIG_NAMES, make_config, table_draws  # noqa: F401
