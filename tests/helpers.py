"""Shared test helpers: tolerances and the oracle-vs-library comparison."""
import numpy as np

from workloads import rng

# fp32 results: rel 1e-5 / abs 1e-6.  bf16-stored results computed in fp32: rel 2e-2, plus an
# absolute term of 1e-3 for values near zero.  Integer, mask and index results: bit-exact.
F32_RTOL, F32_ATOL = 1e-5, 1e-6
BF16_RTOL, BF16_ATOL = 2e-2, 1e-3


def as_float(arr: np.ndarray, dtype: str) -> np.ndarray:
    return rng.bf16_bits_to_f32(arr) if dtype == "bf16" else arr


def assert_matches(got: np.ndarray, ref: np.ndarray, dtype: str, what: str = "", exact: bool = False) -> None:
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    if dtype in ("u8", "i32", "u32"):
        np.testing.assert_array_equal(got, ref, err_msg=what)
        return
    g, r = as_float(got, dtype).astype(np.float64), as_float(ref, dtype).astype(np.float64)
    gn, rn = np.isnan(g), np.isnan(r)
    np.testing.assert_array_equal(gn, rn, err_msg=f"{what}: NaN positions differ")
    g, r = np.where(gn, 0.0, g), np.where(rn, 0.0, r)
    inf = np.isinf(r)
    np.testing.assert_array_equal(g[inf], r[inf], err_msg=f"{what}: infinities differ")
    g, r = np.where(inf, 0.0, g), np.where(inf, 0.0, r)
    if exact:
        np.testing.assert_array_equal(g, r, err_msg=what)
        return
    rtol, atol = (BF16_RTOL, BF16_ATOL) if dtype == "bf16" else (F32_RTOL, F32_ATOL)
    err = np.abs(g - r)
    bound = atol + rtol * np.abs(r)
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst at {i}: "
                             f"got {g[i]!r} want {r[i]!r}")
