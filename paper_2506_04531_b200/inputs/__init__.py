"""Seeded synthetic inputs shared by the CUDA path's tests/benchmark and the oracle's tests:
layouts, value generators (numpy here, a CUDA twin in gen_cuda) and event traces.
None of the method's arithmetic lives in this package."""
from . import gen, layouts, trace, workloads  # noqa: F401
