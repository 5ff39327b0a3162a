"""Seeded synthetic input generators shared by the oracle-side and CUDA-side tests.

Holds none of the method's arithmetic.  ``gen`` is the numpy generator; ``gpu`` wraps the
CUDA twin (same bits, produced in HBM) and doubles as the stand-in compute kernel that
models the inner training steps between two outer rounds.
"""
from . import gen  # noqa: F401
