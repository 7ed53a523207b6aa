"""Seeded synthetic inputs and declarative chain descriptions (no method arithmetic)."""
from . import rng, workloads  # noqa: F401
from .workloads import Chain, CONFIGS, make_inputs  # noqa: F401
