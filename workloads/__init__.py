"""Seeded synthetic workloads (input generation only; none of the method's arithmetic)."""
from . import configs, generators  # noqa: F401
