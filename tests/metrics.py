"""Error measures shared by the GPU parity tests.

Two numbers per comparison, both against the oracle's value `ref`:
  rel_err        ||G - O||_F / ||O||_F over the whole tensor (the stated tolerance of every test);
  worst_row_err  max over rows j of ||G_j - O_j|| / max(||O_j||, rms_j ||O_j||): the same ratio for
                 the single worst row (last axis = row), the denominator floored at the typical row
                 norm so that a nearly-zero row cannot inflate it.
The Frobenius ratio alone lets one wrong row among T hide (it contributes ~sqrt(2/T)); the worst-row
ratio does not.  Rounding errors are independent from element to element, so for a correct kernel a
row's ratio scatters around the tensor's by about 1/sqrt(2 n) for rows of n elements: the worst of
many rows stays within 2x the Frobenius tolerance for n >= 64 and within 3x for shorter rows, while a
row of garbage gives a ratio near sqrt(2).
"""
import numpy as np


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def rel_err(got, ref) -> float:
    got, ref = _f64(got), _f64(ref)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


def worst_row_err(got, ref) -> float:
    got, ref = _f64(got), _f64(ref)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if got.ndim == 0 or got.size == 0:
        return 0.0
    g = got.reshape(-1, got.shape[-1])
    r = ref.reshape(-1, ref.shape[-1])
    row_norm = np.linalg.norm(r, axis=1)
    typical = float(np.sqrt(np.mean(row_norm ** 2)))
    den = np.maximum(row_norm, max(typical, 1e-300))
    return float(np.max(np.linalg.norm(g - r, axis=1) / den))


def worst_row_factor(row_len: int) -> float:
    return 2.0 if row_len >= 64 else 3.0


def assert_parity(got, ref, tol: float, what: str = "") -> float:
    """Frobenius ratio <= tol and worst-row ratio <= factor * tol; returns the Frobenius ratio."""
    got, ref = _f64(got), _f64(ref)
    e = rel_err(got, ref)
    assert e <= tol, (what, "frobenius", e, tol)
    if got.ndim >= 1 and got.size:
        wr = worst_row_err(got, ref)
        bound = worst_row_factor(got.shape[-1]) * tol
        assert wr <= bound, (what, "worst row", wr, bound)
    return e
