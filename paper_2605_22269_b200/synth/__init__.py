"""Seeded synthetic K/V/Q streams: ``cpu`` (numpy) and ``gpu`` (CUDA) produce the same bytes."""
from .cpu import StreamSpec, workload  # noqa: F401
