"""Seeded synthetic inputs and named workload shapes (no method arithmetic lives here)."""
from . import configs, gen  # noqa: F401
