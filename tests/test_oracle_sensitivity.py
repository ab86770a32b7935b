"""Pins of the oracle's layer sensitivity and bit assignment (Section 3.2, Eq. 2):
Omega_i = |mean(lambda_i)| + std(lambda_i), layers sorted by Omega in descending order, bit widths dealt
from a caller-supplied budget.  Pinned by a hand-worked example, closed forms (constant samples, sign
flip, power-of-two scaling), invariance under reordering of the samples, equivariance under reordering
of the layers, the standard library's population statistics, tie handling, the reversed assignment of
the appendix's ablation, and the paper's own remark about the 7th layer of SQuAD."""
import statistics
from pathlib import Path

import numpy as np
import pytest

import oracle

GOLDEN = Path(__file__).resolve().parent / "golden"


def test_hand_worked_three_layers():
    # layer 0: constant 1            -> mean 1,  std 0 -> Omega 1
    # layer 1: -2, 2, -2, 2          -> mean 0,  std 2 -> Omega 2
    # layer 2: -3, -3, -1, -1        -> mean -2, std 1 -> Omega |-2| + 1 = 3
    lam = [[1, 1, 1, 1], [-2, 2, -2, 2], [-3, -3, -1, -1]]
    st, omega, order, bits = oracle.sensitivity_bits(lam, [8, 4, 2])
    assert st == oracle.OK
    assert omega.tolist() == [1.0, 2.0, 3.0]
    assert order.tolist() == [2, 1, 0]            # descending Omega
    assert bits.tolist() == [2, 4, 8]             # most sensitive layer (2) gets budget[0] = 8
    st, _, order_r, bits_r = oracle.sensitivity_bits(lam, [8, 4, 2], reverse=True)
    assert order_r.tolist() == [2, 1, 0] and bits_r.tolist() == [8, 4, 2]   # the ablation: most sensitive gets least


def test_population_std_is_the_reading():
    # two samples 0 and 2: mean 1; population std 1 (sample std would be sqrt(2))
    st, omega, _, _ = oracle.sensitivity_bits([[0.0, 2.0]], [2])
    assert omega[0] == 2.0


def test_closed_forms_and_invariances():
    rng = np.random.default_rng(11)
    L, S = 12, 10
    lam = rng.standard_normal((L, S)) * rng.uniform(0.1, 8.0, size=(L, 1)) + rng.uniform(-2, 6, size=(L, 1))
    budget = [3] * 6 + [2] * 6
    st, omega, order, bits = oracle.sensitivity_bits(lam, budget)
    assert st == oracle.OK
    # the standard library's population statistics (another implementation of the same definitions)
    for i in range(L):
        ref = abs(statistics.fmean(lam[i])) + statistics.pstdev(lam[i])
        assert omega[i] == pytest.approx(ref, rel=1e-13)
    # constant samples: Omega = |lambda|
    c = rng.uniform(-5, 5, size=L)
    assert np.allclose(oracle.sensitivity_bits(np.repeat(c[:, None], S, axis=1), budget)[1], np.abs(c), rtol=1e-14, atol=0)
    assert np.array_equal(oracle.sensitivity_bits(np.repeat(c[:, None], 2, axis=1), budget)[1], np.abs(c))  # c + c is exact
    # sign flip and power-of-two scaling are exact in floating point
    assert np.array_equal(oracle.sensitivity_bits(-lam, budget)[1], omega)
    assert np.array_equal(oracle.sensitivity_bits(lam * 4.0, budget)[1], omega * 4.0)
    # a shift moves the mean only: Omega(lambda + t) - |mean + t| = std(lambda)
    t = 1000.0
    shifted = oracle.sensitivity_bits(lam + t, budget)[1] - np.abs(lam.mean(axis=1) + t)
    assert np.allclose(shifted, lam.std(axis=1), rtol=0, atol=1e-9)
    # reordering the samples of a layer changes nothing but the rounding of the sums
    perm = rng.permutation(S)
    assert np.allclose(oracle.sensitivity_bits(lam[:, perm], budget)[1], omega, rtol=1e-13, atol=0)
    # reordering the layers reorders the results with them
    lp = rng.permutation(L)
    st, omega_p, order_p, bits_p = oracle.sensitivity_bits(lam[lp], budget)
    assert np.array_equal(omega_p, omega[lp])
    assert np.array_equal(lp[order_p], order)      # same layers in the same rank order
    assert np.array_equal(bits_p, bits[lp])
    # the order is a permutation, descending in Omega; the bits are the budget dealt along it
    assert sorted(order.tolist()) == list(range(L))
    assert np.all(np.diff(omega[order]) <= 0)
    assert bits[order].tolist() == budget
    assert sorted(bits.tolist()) == sorted(budget)
    # with a non-increasing budget a more sensitive layer never gets fewer bits
    for a in range(L):
        for b in range(L):
            if omega[a] > omega[b]:
                assert bits[a] >= bits[b]
    # reversed: the same order, the budget dealt from the other end
    st, _, order_r, bits_r = oracle.sensitivity_bits(lam, budget, reverse=True)
    assert np.array_equal(order_r, order) and bits_r[order].tolist() == budget[::-1]


def test_ties_keep_the_lower_layer_first():
    lam = [[2.0, 2.0], [1.0, 3.0], [2.0, 2.0], [-2.0, -2.0]]   # Omega = 2, 3, 2, 2
    st, omega, order, bits = oracle.sensitivity_bits(lam, [8, 4, 3, 2])
    assert omega.tolist() == [2.0, 3.0, 2.0, 2.0]
    assert order.tolist() == [1, 0, 2, 3]
    assert bits.tolist() == [4, 8, 3, 2]


def test_variance_outranks_mean_as_in_the_papers_squad_remark():
    mean, var = [float(v) for v in [ln for ln in (GOLDEN / "sensitivity_squad_layer7.txt").read_text().splitlines()
                                    if not ln.startswith("#")][0].split()]
    # two-point distribution with exactly that mean and variance, against a quiet layer with five times the mean
    sd = var ** 0.5
    lam = [[mean - sd, mean + sd] * 5, [5.0 * mean] * 10]
    st, omega, order, bits = oracle.sensitivity_bits(lam, [3, 2])
    assert omega[0] == pytest.approx(abs(mean) + sd, rel=1e-12) and omega[1] == 5.0 * mean
    assert order.tolist() == [0, 1] and bits.tolist() == [3, 2]     # a mean-only rule would give [2, 3]


def test_errors():
    assert oracle.sensitivity_bits([[1.0, np.nan]], [2])[0] == oracle.ERR_NONFINITE
    assert oracle.sensitivity_bits([[1.0, 2.0]], [5])[0] == oracle.ERR_INVALID


def test_printed_bit_table_is_reproduced_by_a_plausible_spectrum():
    # plausibility only: the "2/3-bit MP" row for SST-2 gives 3 bits to layers 4-9; eigenvalue samples whose
    # mean + spread is larger there, with a budget of six 3s and six 2s, reproduce the printed row
    from paper_1909_05840_b200 import synth
    printed = synth.MP_PRESETS["2/3-MP SST-2"]
    rng = np.random.default_rng(5)
    level = np.array([0.4, 0.5, 0.6, 2.0, 2.5, 3.0, 2.8, 2.2, 1.9, 0.7, 0.3, 0.2])
    lam = level[:, None] * (1.0 + 0.1 * rng.standard_normal((12, 10)))
    st, omega, order, bits = oracle.sensitivity_bits(lam, [3] * 6 + [2] * 6)
    assert tuple(int(b) for b in bits) == printed
