"""The dynamic bit-width problem (Eq. 4): the library's exact solver (a host function of the C ABI) against the oracle's
exhaustive enumeration on small instances, plus properties that hold at any size."""
import numpy as np
import pytest

import oracle
import paper_2411_17525_b200 as hb


def instance(L, J, seed):
    rng = np.random.default_rng(seed)
    bits64 = np.array([129, 193, 257, 513][:J], dtype=np.int32)           # 2.02, 3.02, 4.02, 8.02 bits
    t2 = np.sort(rng.uniform(0.5, 1.5, size=(L, 1)) * np.array([0.118, 0.0345, 0.0095, 8.8e-5][:J])[None, :], axis=1)[:, ::-1]
    alpha = rng.lognormal(0.0, 1.0, size=L)
    sizes = rng.choice([2048 * 2048, 512 * 2048, 8192 * 2048], size=L).astype(np.int64)
    return alpha, np.ascontiguousarray(t2), bits64, sizes


@pytest.mark.parametrize("L,J,budget64,seed", [(5, 3, 200, 1), (6, 4, 224, 2), (7, 4, 300, 3), (4, 2, 160, 4), (7, 3, 257, 5)])
def test_solver_matches_exhaustive_enumeration(L, J, budget64, seed):
    alpha, t2, bits64, sizes = instance(L, J, seed)
    choice, obj = hb.higgs_allocate_bits(alpha, t2, bits64, sizes, budget64)
    ref_choice, ref_obj = oracle.allocate_bits_bruteforce(alpha, t2, bits64 / 64.0, sizes, budget64 / 64.0)
    assert ref_choice is not None
    assert abs(obj - ref_obj) <= 1e-12 * max(1.0, abs(ref_obj))
    # the returned assignment is feasible and attains the objective it reports
    assert int(np.dot(bits64[choice].astype(np.int64), sizes)) <= budget64 * int(sizes.sum())
    assert abs(float(np.sum(alpha * t2[np.arange(L), choice])) - obj) <= 1e-12


def test_budget_extremes_and_monotonicity():
    alpha, t2, bits64, sizes = instance(40, 4, 9)
    lo, _ = hb.higgs_allocate_bits(alpha, t2, bits64, sizes, 129)        # only the smallest option fits everywhere
    assert np.all(lo == 0)
    hi, obj_hi = hb.higgs_allocate_bits(alpha, t2, bits64, sizes, 513)   # everything fits: the most accurate option
    assert np.all(hi == 3)
    prev = np.inf
    for b in (129, 160, 193, 224, 257, 320, 513):
        _, obj = hb.higgs_allocate_bits(alpha, t2, bits64, sizes, b)
        assert obj <= prev + 1e-15                                        # a larger budget never hurts
        prev = obj
    assert abs(prev - obj_hi) < 1e-15
    with pytest.raises(RuntimeError):
        hb.higgs_allocate_bits(alpha, t2, bits64, sizes, 100)             # below the smallest option: infeasible


def test_sensitive_layers_get_more_bits():
    """With equal sizes and errors, the budget goes to the layers with the largest alpha (the linear model's weights)."""
    L = 8
    alpha = np.arange(1, L + 1, dtype=np.float64)
    t2 = np.tile(np.array([0.118, 0.0345, 0.0095]), (L, 1))
    bits64 = np.array([129, 193, 257], dtype=np.int32)
    sizes = np.full(L, 4096 * 4096, dtype=np.int64)
    choice, _ = hb.higgs_allocate_bits(alpha, t2, bits64, sizes, 193)
    assert np.all(np.diff(choice) >= 0) and choice[0] < choice[-1]
