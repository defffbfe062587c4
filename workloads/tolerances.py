"""Tolerances of the GPU parity tests and of the benchmark's output checks, in one place (no arithmetic of the method).

Two norms are fixed for this library: fp32 results  ||Y - Y*||_F / ||Y*||_F <= 1e-5, and for bf16 operands
max |err| <= 2e-2 * ||W row||_2 * ||X col||_2.  A norm over a whole output hides a single wrong element (one
element that is 1 % off in a 1024 x 1024 output moves the Frobenius ratio by about 1e-8), so every comparison
here is also made element by element against a bound derived from the arithmetic:

  fp32 accumulation of n products has a rounding error of about eps32 * ||w||_2 * ||x||_2 (random signs; the
  worst case is n times that).  ELEM_ACC = 1e-5 times the two norms leaves two orders of magnitude of room for
  any summation order and is still far below one dropped or misplaced term, which changes the result by about
  ||w|| * ||x|| / n.
  A bf16 output adds one rounding of the fp32 result: at most half a bf16 unit in the last place, 2^-9 of the
  power of two below |y|, bounded here by 2^-8 * |y*| (the error of the accumulator may move y across a
  rounding boundary, which the sum of the two terms covers).
"""
import numpy as np

F32_TOL = 1e-5     # relative Frobenius error, fp32 path (fixed requirement)
BF16_TOL = 2e-2    # max |err| / (||W row|| * ||X col||), bf16 path (fixed requirement)
ELEM_ACC = 1e-5    # per element: fp32 accumulator error / (||W row|| * ||X col||)
BF16_HALF_ULP = 2.0 ** -8


def rel_fro(got, want):
    want = np.asarray(want, dtype=np.float64)
    return float(np.linalg.norm(np.asarray(got, dtype=np.float64) - want) / max(np.linalg.norm(want), 1e-300))


def elem_bound(scale, want, out_bf16, bias_abs=None):
    """Per-element bound.  scale = ||W row|| * ||X col|| broadcast to the output's shape; want = oracle output;
    bias_abs (broadcastable) widens the accumulator term by the magnitude of an added bias."""
    s = scale if bias_abs is None else scale + bias_abs
    b = ELEM_ACC * s + 1e-30
    if out_bf16:
        b = b + BF16_HALF_ULP * np.abs(want)
    return b


def assert_close(got, want, scale, *, bf16_in, out_bf16, bias_abs=None, what=""):
    """All checks for one output: the fixed norm for the dtype, then the per-element bound."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = np.abs(got - want)
    if bf16_in:
        loose = BF16_TOL * (scale if bias_abs is None else scale + bias_abs)
        assert np.all(err <= loose + 1e-30), f"{what}: bf16 bound exceeded by {np.max(err - loose)}"
        if not out_bf16:
            assert rel_fro(got, want) < 1e-4, (what, rel_fro(got, want))
    else:
        assert rel_fro(got, want) <= F32_TOL, (what, rel_fro(got, want))
    b = elem_bound(scale, want, out_bf16, bias_abs)
    bad = err > b
    assert not np.any(bad), (f"{what}: {int(bad.sum())} elements outside the per-element bound, worst ratio "
                             f"{float(np.max(err / b))} at {np.unravel_index(int(np.argmax(err / b)), err.shape)}")
