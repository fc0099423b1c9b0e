"""CPU oracle of the VARCO partitioned layer -- TEST INFRASTRUCTURE ONLY.

Plain fp64 restatement of the paper's method (C++ in ``varco_oracle.cpp`` for
the partitioned algorithm, NumPy/PyTorch dense matrices in ``dense.py`` for
brute force on tiny graphs).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library never
does, and shares no code with it.
"""
from .binding import Oracle, OracleGraph, build_oracle  # noqa: F401
