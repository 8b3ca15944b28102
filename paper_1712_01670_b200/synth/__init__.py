"""Seeded synthetic inputs (video streams, layer tables, random weights).

Holds none of the method's arithmetic; it is the only module that the CPU
oracle's tests and the CUDA path's tests both draw from.
"""
from . import configs, nets, streams  # noqa: F401
