"""Pins for the oracle's weight quantizer Q (Section 3.1, Section 3.3, Appendix A).

None of these tests re-types the oracle's formula: they check its output against
brute-force enumeration in float64, error bounds, invariants and closed forms.
"""
import numpy as np
import pytest

import oracle

BITS = (2, 3, 4, 8)


def _w(N, K, seed, scale=0.05):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((N, K)) * scale).astype(np.float32)


def _grid64(delta, q0, bits):
    """The 2^k quantization points q_j = q0 + j*Delta in double precision (Appendix A)."""
    return np.float64(q0) + np.arange(1 << bits, dtype=np.float64) * np.float64(delta)


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("groups", (1, 4, 12))
def test_codes_are_a_nearest_grid_point_bruteforce(bits, groups):
    # Section 3.1: Q(z) = q_j for z in (t_j, t_{j+1}]: the chosen point is the nearest one.
    N, K = 24, 96
    w = _w(N, K, 100 + bits + groups)
    st, codes, delta, q0 = oracle.quantize_weights(w, bits, groups)
    assert st == oracle.OK
    R = N // groups
    for g in range(groups):
        grid = _grid64(delta[g], q0[g], bits)
        blk = w[g * R:(g + 1) * R].astype(np.float64)
        dist = np.abs(blk[..., None] - grid)          # every element against every grid point
        best = dist.min(axis=-1)
        chosen = np.take_along_axis(dist, codes[g * R:(g + 1) * R][..., None].astype(np.int64), -1)[..., 0]
        # reciprocal-multiply evaluation may differ from the exact quotient by a few ulp, so a
        # value within that distance of a midpoint may land on either neighbour.
        slack = np.float64(delta[g]) * 2.0 ** -18 + np.spacing(np.abs(blk).astype(np.float32))
        assert np.all(chosen <= best + slack)


@pytest.mark.parametrize("bits", BITS)
def test_error_bound_half_step(bits):
    # |W - Q(W)| <= Delta/2 inside the range (uniform grid, Appendix A).
    N, K, G = 36, 128, 6
    w = _w(N, K, 7 + bits)
    st, codes, delta, q0 = oracle.quantize_weights(w, bits, G)
    wq = oracle.dequantize_weights(codes, G, delta, q0).astype(np.float64)
    d = np.repeat(delta.astype(np.float64), N // G)[:, None]
    bound = d / 2 * (1 + 2.0 ** -18) + 2 * np.spacing(np.abs(w))
    assert np.all(np.abs(w.astype(np.float64) - wq) <= bound)


@pytest.mark.parametrize("bits", BITS)
def test_range_and_endpoints(bits):
    # Codes are unsigned integers in {0..2^k-1}; the group's min maps to 0 and its max to 2^k-1.
    N, K, G = 12, 64, 3
    w = _w(N, K, 21 + bits)
    st, codes, delta, q0 = oracle.quantize_weights(w, bits, G)
    L = (1 << bits) - 1
    assert codes.min() >= 0 and codes.max() <= L
    R = N // G
    for g in range(G):
        blk = w[g * R:(g + 1) * R]
        cb = codes[g * R:(g + 1) * R]
        assert cb[blk == blk.min()].tolist() == [0] * int((blk == blk.min()).sum())
        assert np.all(cb[blk == blk.max()] == L)
        # q0 is the group minimum and Delta the range split into 2^k - 1 steps
        assert q0[g] == blk.min()
        assert np.isclose(float(delta[g]), (float(blk.max()) - float(blk.min())) / L, rtol=1e-6)


@pytest.mark.parametrize("bits", BITS)
def test_monotone_within_group(bits):
    # Interval form of Section 3.1: w1 <= w2 implies code(w1) <= code(w2).
    w = _w(8, 256, 33 + bits)
    st, codes, _, _ = oracle.quantize_weights(w, bits, 2)
    R = 4
    for g in range(2):
        v = w[g * R:(g + 1) * R].ravel()
        c = codes[g * R:(g + 1) * R].ravel().astype(np.int64)
        order = np.argsort(v, kind="stable")
        assert np.all(np.diff(c[order]) >= 0)


@pytest.mark.parametrize("bits", BITS)
def test_requantizing_is_idempotent(bits):
    N, K, G = 16, 64, 4
    w = _w(N, K, 55 + bits)
    st, codes, delta, q0 = oracle.quantize_weights(w, bits, G)
    wq = oracle.dequantize_weights(codes, G, delta, q0)
    # (a) same grid supplied by the caller: identical codes
    L = (1 << bits) - 1
    hi = (q0.astype(np.float64) + L * delta.astype(np.float64)).astype(np.float32)
    st2, codes2, delta2, q02 = oracle.quantize_weights(wq, bits, G, range_lo=q0, range_hi=hi)
    assert np.array_equal(codes2, codes)
    # (b) range re-derived from Q(W): the minimum is reproduced exactly, codes unchanged
    st3, codes3, delta3, q03 = oracle.quantize_weights(wq, bits, G)
    assert np.array_equal(q03, q0)
    assert np.allclose(delta3, delta, rtol=1e-5)
    assert np.array_equal(codes3, codes)


@pytest.mark.parametrize("bits", BITS)
def test_integer_grid_closed_form(bits):
    # A group holding exactly the integers 0..2^k-1 has q0 = 0, Delta = 1, code = value, Q(w) = w.
    L = (1 << bits) - 1
    vals = np.arange(L + 1, dtype=np.float32)
    K = 32 * ((L + 1 + 31) // 32)
    w = np.resize(vals, (2, K)).astype(np.float32)
    st, codes, delta, q0 = oracle.quantize_weights(w, bits, 1)
    assert delta[0] == 1.0 and q0[0] == 0.0
    assert np.array_equal(codes.astype(np.float32), w)
    assert np.array_equal(oracle.dequantize_weights(codes, 1, delta, q0), w)


def test_ties_round_half_to_even():
    # range [0, 3] with k = 2 gives Delta = 1: midpoints 0.5, 1.5, 2.5 go to the even neighbour.
    w = np.array([[0.0, 0.5, 1.5, 2.5, 3.0, 1.0, 2.0, 0.25]], np.float32)
    st, codes, delta, q0 = oracle.quantize_weights(w, 2, 1)
    assert delta[0] == 1.0 and q0[0] == 0.0
    assert codes[0].tolist() == [0, 0, 2, 2, 3, 1, 2, 0]


@pytest.mark.parametrize("bits", BITS)
def test_group_partition_equivalences(bits):
    # 1 group == per-tensor; N groups == per-row; G groups == quantizing each row block alone.
    N, K = 12, 64
    w = _w(N, K, 77 + bits)
    for G in (1, 3, 12):
        st, codes, delta, q0 = oracle.quantize_weights(w, bits, G)
        R = N // G
        for g in range(G):
            st1, c1, d1, z1 = oracle.quantize_weights(w[g * R:(g + 1) * R], bits, 1)
            assert np.array_equal(c1, codes[g * R:(g + 1) * R])
            assert d1[0] == delta[g] and z1[0] == q0[g]
    # per-tensor range really is the global min
    st, codes, delta, q0 = oracle.quantize_weights(w, bits, 1)
    assert q0[0] == w.min()
    # per-row range really is each row's min
    st, codes, delta, q0 = oracle.quantize_weights(w, bits, N)
    assert np.array_equal(q0, w.min(axis=1))


def test_groups_change_the_result_when_ranges_differ():
    # rows with very different ranges: per-row quantization is far more accurate than per-tensor
    # (the effect Table 2 measures); guards against a group index that is ignored.
    rng = np.random.default_rng(5)
    w = (rng.standard_normal((8, 128)) * np.logspace(-3, 0, 8)[:, None]).astype(np.float32)
    errs = {}
    for G in (1, 8):
        st, c, d, z = oracle.quantize_weights(w, 4, G)
        errs[G] = np.abs(oracle.dequantize_weights(c, G, d, z) - w)[0].max()
    assert errs[8] < errs[1] / 50


def test_constant_group_and_nonfinite():
    w = np.full((4, 32), 0.125, np.float32)
    w[2:] = np.linspace(-1, 1, 64, dtype=np.float32).reshape(2, 32)
    st, codes, delta, q0 = oracle.quantize_weights(w, 4, 2)
    assert st == oracle.OK
    assert delta[0] == 1.0 and q0[0] == 0.125 and not codes[:2].any()
    assert np.array_equal(oracle.dequantize_weights(codes, 2, delta, q0)[:2], w[:2])
    w[3, 5] = np.inf
    st, *_ = oracle.quantize_weights(w, 4, 2)
    assert st == oracle.ERR_NONFINITE
    w[3, 5] = np.nan
    st, *_ = oracle.quantize_weights(w, 4, 2)
    assert st == oracle.ERR_NONFINITE


def test_caller_range_clamps_outliers():
    # Appendix A: the range may be a sub-interval of [min, max]; values outside are clamped.
    w = np.array([[-10.0, -1.0, -0.5, 0.0, 0.5, 1.0, 10.0, 0.2]], np.float32)
    st, codes, delta, q0 = oracle.quantize_weights(w, 2, 1, range_lo=np.array([-1.0], np.float32),
                                                   range_hi=np.array([1.0], np.float32))
    assert st == oracle.OK and q0[0] == -1.0
    assert np.isclose(delta[0], 2.0 / 3.0)
    assert codes[0, 0] == 0 and codes[0, 1] == 0 and codes[0, 5] == 3 and codes[0, 6] == 3
    assert codes[0, 3] in (1, 2)


def test_invalid_arguments():
    w = np.zeros((6, 32), np.float32)
    assert oracle.quantize_weights(w, 5, 1)[0] == oracle.ERR_INVALID
    assert oracle.quantize_weights(w, 4, 4)[0] == oracle.ERR_INVALID  # 6 % 4 != 0
