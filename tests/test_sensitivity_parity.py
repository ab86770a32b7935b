"""qb_sensitivity_bits (host-only entry point of the library) against the oracle (Section 3.2, Eq. 2).

Both sides compute in fp64 with sums in index order, so Omega is expected bit-equal; the gate is 1e-12
relative.  The order and the bit widths are integers decided by fp64 comparisons on both sides: exact.
No GPU is needed: the call does no device work."""
import numpy as np
import pytest

import oracle
import paper_1909_05840_b200 as qb
from paper_1909_05840_b200 import build as qb_build
from paper_1909_05840_b200 import synth


@pytest.fixture(scope="module", autouse=True)
def _built():
    qb_build.build()


@pytest.mark.parametrize("layers,samples,seed", [(1, 1, 0), (3, 4, 1), (12, 10, 2), (24, 10, 3), (12, 37, 4), (64, 5, 5)])
@pytest.mark.parametrize("reverse", [False, True])
def test_library_matches_oracle(layers, samples, seed, reverse):
    rng = np.random.default_rng(seed)
    lam = rng.standard_normal((layers, samples)) * rng.uniform(0.05, 9.0, size=(layers, 1)) + rng.uniform(-3, 5, size=(layers, 1))
    budget = np.sort(rng.choice(synth.BITS_CHOICES, size=layers))[::-1].copy()
    st, o_omega, o_order, o_bits = oracle.sensitivity_bits(lam, budget, reverse)
    assert st == oracle.OK
    omega, order, bits = qb.sensitivity_bits(lam, budget, reverse)
    assert np.allclose(omega, o_omega, rtol=1e-12, atol=0)
    assert np.array_equal(omega, o_omega)
    assert np.array_equal(order, o_order)
    assert np.array_equal(bits, o_bits)


def test_ties_and_errors_match_oracle():
    lam = np.array([[2.0, 2.0], [1.0, 3.0], [2.0, 2.0], [-2.0, -2.0]])
    budget = [8, 4, 3, 2]
    omega, order, bits = qb.sensitivity_bits(lam, budget)
    st, o_omega, o_order, o_bits = oracle.sensitivity_bits(lam, budget)
    assert np.array_equal(order, o_order) and np.array_equal(bits, o_bits) and order.tolist() == [1, 0, 2, 3]
    with pytest.raises(qb.QbertError) as e:
        qb.sensitivity_bits(lam, [8, 4, 3, 5])
    assert e.value.status == qb.QB_ERR_INVALID and oracle.sensitivity_bits(lam, [8, 4, 3, 5])[0] == oracle.ERR_INVALID
    lam[2, 1] = np.inf
    with pytest.raises(qb.QbertError) as e:
        qb.sensitivity_bits(lam, budget)
    assert e.value.status == qb.QB_ERR_NONFINITE and oracle.sensitivity_bits(lam, budget)[0] == oracle.ERR_NONFINITE


def test_paper_preset_budget_feeds_the_stack_descriptor_width():
    # twelve layers, budget of the 2/3-bit mixed setting: the result is a valid per-layer width list
    rng = np.random.default_rng(9)
    lam = np.abs(rng.standard_normal((12, 10))) * np.linspace(3.0, 0.2, 12)[:, None]
    omega, order, bits = qb.sensitivity_bits(lam, [3] * 6 + [2] * 6)
    assert sorted(bits.tolist()) == [2] * 6 + [3] * 6 and set(bits.tolist()) <= set(synth.BITS_CHOICES)
