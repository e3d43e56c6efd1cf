"""Shared test utilities: error metrics and numpy <-> device conversions (no method arithmetic)."""
from __future__ import annotations

import numpy as np

# Tolerances of the workload statement, as numbers (versus the fp64 oracle).
F32_MAX_REL = 1e-5
BF16_MAX_REL = 2e-2
BF16_MEAN_REL = 5e-3


def rel_errors(got: np.ndarray, ref: np.ndarray):
    """Normwise relative errors per problem instance (rows of a 2-D view).

    Returns (max over rows of max|d|/max|ref|, mean over rows of sum|d|/sum|ref|).
    For y and dx a row is a token; for dL and dR a row is one m x m block.
    """
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if got.size == 0:
        return 0.0, 0.0
    g = got.reshape(got.shape[0], -1)
    r = ref.reshape(ref.shape[0], -1)
    d = np.abs(g - r)
    if not np.isfinite(g).all():
        return float("inf"), float("inf")
    den_inf = np.maximum(np.max(np.abs(r), axis=1), 1e-300)
    den_1 = np.maximum(np.sum(np.abs(r), axis=1), 1e-300)
    return float(np.max(np.max(d, axis=1) / den_inf)), float(np.mean(np.sum(d, axis=1) / den_1))


def assert_close(got, ref, dtype: str, what: str = "", scale: float = 1.0):
    emax, emean = rel_errors(got, ref)
    if dtype == "f32":
        assert emax <= F32_MAX_REL * scale, f"{what}: max rel err {emax:.3e} > {F32_MAX_REL * scale:.1e}"
    else:
        assert emax <= BF16_MAX_REL * scale, f"{what}: max rel err {emax:.3e} > {BF16_MAX_REL * scale:.1e}"
        assert emean <= BF16_MEAN_REL * scale, f"{what}: mean rel err {emean:.3e} > {BF16_MEAN_REL * scale:.1e}"
    return emax, emean


from paper_2204_00595_b200.inputs import to_device, to_host64  # noqa: E402,F401  (re-exported for the tests)
