"""TEST INFRASTRUCTURE — CPU oracle for the ASD hot path.

A plain, slow, float64 numpy restatement of what the CUDA library computes,
written from the paper.  Only `tests/`, the smoke check and the CPU-baseline /
reference legs of the benchmark import this package; the product path never
does, and the two share no code.
"""
from . import philox, denoisers, asd  # noqa: F401
