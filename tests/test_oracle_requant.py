"""Pins of the oracle's int8 re-quantization of a linear's output and of the int8 row sums: brute force
over the 255-point grid, exact grid points, saturation, odd symmetry, monotonicity, numpy sums."""
import numpy as np

import oracle


def test_requantize_is_the_nearest_point_of_the_grid():
    rng = np.random.default_rng(2)
    s = np.float32(0.0371)
    y = (rng.standard_normal(20000) * 2.0).astype(np.float32)
    c = oracle.requantize_i8(y, float(s)).astype(np.int64)
    grid = np.arange(-127, 128, dtype=np.float64) * float(s)
    best = np.abs(y.astype(np.float64)[:, None] - grid[None, :])
    d_c = best[np.arange(y.size), c + 127]
    # nearest up to the rounding of the reciprocal multiply (a few ulp of y / s); ties may go either way
    assert np.all(d_c <= best.min(axis=1) + 4 * np.spacing(np.abs(y)).astype(np.float64) + 1e-12)
    assert c.min() == -127 and c.max() == 127          # both ends reached: values beyond 127 s saturate
    assert np.all(c[np.abs(y) > 127.5 * s] * np.sign(y[np.abs(y) > 127.5 * s]) == 127)


def test_requantize_grid_points_symmetry_monotone():
    for s in (0.5, 0.25, 2.0**-7):                     # powers of two: y = j * s and 1 / s are exact
        j = np.arange(-127, 128)
        assert np.array_equal(oracle.requantize_i8((j * s).astype(np.float32), s), j.astype(np.int8))
        # exact ties go to the even code
        assert list(oracle.requantize_i8(np.array([0.5 * s, 1.5 * s, 2.5 * s, -0.5 * s, -1.5 * s], np.float32), s)) == [0, 2, 2, 0, -2]
    rng = np.random.default_rng(3)
    y = np.sort((rng.standard_normal(5000) * 3).astype(np.float32))
    c = oracle.requantize_i8(y, 0.0213)
    assert np.all(np.diff(c.astype(np.int32)) >= 0)
    assert np.array_equal(oracle.requantize_i8(-y, 0.0213), -c)
    assert np.array_equal(oracle.requantize_i8(np.array([1e30, -1e30, np.float32(3.4e38)], np.float32), 0.01), [127, -127, 127])


def test_rowsum_i8_is_the_plain_sum():
    rng = np.random.default_rng(4)
    xq = rng.integers(-127, 128, (37, 256)).astype(np.int8)
    assert np.array_equal(oracle.rowsum_i8(xq), xq.astype(np.int64).sum(1).astype(np.int32))
    assert np.array_equal(oracle.rowsum_i8(np.full((3, 128), -127, np.int8)), [-127 * 128] * 3)
