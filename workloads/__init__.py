"""Seeded synthetic inputs shared by the tests, the benchmark and the reference checks.

Shapes, value generators and arrival traces only: nothing here computes
timestamps, staleness, learning rates or weight updates.
"""
from . import arrivals, configs, generators, layouts  # noqa: F401
