"""fp64 CPU oracle for the gated subspace linear layer (test infrastructure).

Only tests, ``__graft_entry__.smoke()`` and the CPU-baseline leg of ``bench.py``
may import this package.  It shares nothing with the CUDA path.
"""
from . import gsi_oracle, report  # noqa: F401
