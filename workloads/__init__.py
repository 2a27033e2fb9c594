"""Seeded synthetic workloads shared by the CPU oracle tests, the GPU parity tests and the bench.

This package only *describes* and *generates* inputs (shapes, scale schedules, head masks and
Q/K/V tensors).  It holds none of the method's arithmetic: no scoring, selection, compaction,
attention or budget splitting lives here.
"""
from .configs import WorkloadConfig, get_config, SCHEDULES, list_configs  # noqa: F401
from .synthetic import SyntheticQKV, random_observation_rows  # noqa: F401
