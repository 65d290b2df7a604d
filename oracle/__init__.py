"""TEST INFRASTRUCTURE ONLY: float64 CPU oracle of the sparse-DNN SGD hot path.

Importable from the tests, the smoke check and the benchmark's CPU-baseline leg
only.  The CUDA library and its Python binding never import this package, and
this package never imports them.

Parity status: every function here is pinned by the CPU test-suite (dense brute
force, finite differences, autograd, closed forms, a sparse-library single-layer
product, adjointness); none is "parity unpinned".
"""
from .oracle import OracleNet, build, nonzero_sets  # noqa: F401
