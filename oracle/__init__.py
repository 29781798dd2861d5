"""CPU oracle of the embedding-table lookup path (test infrastructure only).

`oracle.cpp` is the arithmetic; this package is a ctypes veneer over it so that
tests, the smoke check and the benchmark's CPU-baseline leg can call it with
numpy arrays. The product package never imports this one.
"""
from .mfet_oracle import *  # noqa: F401,F403
