"""CPU oracle of the per-view training step (test infrastructure, not product code).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
It builds `oracle/liboracle.so` from the C++ sources beside it with g++ (no CUDA) on first use and
wraps its C entry points with NumPy arrays.  It imports nothing from the CUDA package.
"""
from .oracle import (  # noqa: F401
    Oracle,
    Projected,
    build,
    get,
)
