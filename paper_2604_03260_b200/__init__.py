"""Focus (learned-grouping sparse attention) inference hot path for B200 / sm_100a.

The work is done by a C-ABI CUDA library (``csrc/``, declared in ``include/focus.h``); this package
is its thin ctypes binding plus the seeded input generators.  Importing the package does not load
the library; ``paper_2604_03260_b200.binding`` does, and fails loudly when it is missing.
"""
__all__ = ["inputs", "binding", "build", "host_pipeline", "multi"]
