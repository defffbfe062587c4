"""Tolerances of the GPU parity tests (defined once in workloads/tolerances.py, shared with the benchmark's own
output checks)."""
from workloads.tolerances import BF16_HALF_ULP, BF16_TOL, ELEM_ACC, F32_TOL, assert_close, elem_bound, rel_fro  # noqa: F401
