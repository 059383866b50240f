"""Seeded synthetic inputs shared by the oracle's tests and the CUDA path's tests and benchmark."""
from . import gen, workloads  # noqa: F401
