"""Seeded synthetic inputs shaped like the paper's workloads (no method arithmetic)."""
from .generator import *  # noqa: F401,F403
