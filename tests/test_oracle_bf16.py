"""Pins of the oracle's bfloat16 rounding (narrow-output epilogue) against things that do not call it:
a library conversion (torch CPU), the add-and-shift restatement on bit patterns, closed forms, ties,
the half-ulp error bound, monotonicity and brute force over the neighbouring grid points."""
import numpy as np
import torch

import oracle


def _sample(n=200_000, seed=5):
    rng = np.random.default_rng(seed)
    a = rng.standard_normal(n).astype(np.float32) * np.float32(3.0)
    b = (rng.standard_normal(n) * 10.0 ** rng.uniform(-30, 30, n)).astype(np.float32)
    c = rng.integers(0, 2**32, n, dtype=np.uint64).astype(np.uint32).view(np.float32)
    c = c[np.isfinite(c)]
    return np.concatenate([a, b, c])


def test_matches_torch_cpu_conversion():
    y = _sample()
    ours = oracle.round_bf16(y)
    ref = torch.from_numpy(y).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)


def test_matches_add_and_shift_on_bit_patterns():
    y = _sample(seed=6)
    u = y.view(np.uint32).astype(np.uint64)
    ref = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    assert np.array_equal(oracle.round_bf16(y), ref)


def test_representable_values_are_unchanged_and_ties_go_to_even():
    # every bfloat16 value (finite) is a fixed point
    hi = np.arange(0, 1 << 16, dtype=np.uint32)
    hi = hi[((hi >> 7) & 0xFF) != 0xFF]
    y = (hi << 16).view(np.float32)
    assert np.array_equal(oracle.round_bf16(y), hi.astype(np.uint16))
    # exact ties: the kept field is followed by 0x8000; the result has an even kept field
    ties = ((hi << 16) | 0x8000).view(np.float32)
    ties = ties[np.isfinite(ties)]
    r = oracle.round_bf16(ties).astype(np.uint32)
    k = ties.view(np.uint32) >> 16
    assert np.array_equal(r, k + (k & 1))
    # hand-checked: 1 + 2^-8 -> 1.0, 1 + 3*2^-8 -> 1 + 2^-6, and their negatives
    v = np.array([1 + 2.0**-8, 1 + 3 * 2.0**-8, -(1 + 2.0**-8), -(1 + 3 * 2.0**-8)], dtype=np.float32)
    assert list(oracle.round_bf16(v)) == [0x3F80, 0x3F82, 0xBF80, 0xBF82]


def test_error_bound_monotone_and_nearest_by_brute_force():
    y = np.sort(_sample(50_000, seed=7))
    r = oracle.round_bf16(y)
    back = (r.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    fin = np.isfinite(back)
    # half a unit of the last kept place: 2^-8 relative for normal numbers (2^-9 of the next binade)
    normal = fin & (np.abs(y) >= np.finfo(np.float32).tiny)
    assert np.all(np.abs(back[normal] - y[normal].astype(np.float64)) <= np.abs(y[normal].astype(np.float64)) * 2.0**-8)
    # monotone (y sorted ascending; compare the decoded values)
    assert np.all(np.diff(back[fin]) >= 0)
    # brute force: no representable neighbour (one step either way) is strictly nearer
    for step in (-1, 1):
        nb = ((r.astype(np.int64) + step) & 0xFFFF).astype(np.uint32)
        same_sign = (nb >> 15) == (r.astype(np.uint32) >> 15)
        nbv = (nb << 16).view(np.float32).astype(np.float64)
        ok = fin & same_sign & np.isfinite(nbv)
        assert np.all(np.abs(back[ok] - y[ok]) <= np.abs(nbv[ok] - y[ok]))
