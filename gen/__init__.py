"""Seeded synthetic inputs shared by the CPU checker and the CUDA library."""
from . import configs, graphs  # noqa: F401
