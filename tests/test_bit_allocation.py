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


def test_enumeration_and_solver_on_the_hand_solved_instance(golden):
    """Two layers, two options, solved on paper in tests/golden/allocate_2x2.txt: pins the oracle's enumeration (which
    pins the solver everywhere else) and the solver itself."""
    ref = golden("allocate_2x2.txt")
    sizes = np.array(ref["sizes"], dtype=np.int64)
    bits = np.array(ref["bits"])
    alpha = np.array(ref["alpha"])
    t2 = np.array([ref["t2_layer0"], ref["t2_layer1"]])
    for key, budget in (("budget_3", 3.0), ("budget_3p5", 3.5), ("budget_2", 2.0)):
        j0, j1, obj = ref[key]
        choice, got = oracle.allocate_bits_bruteforce(alpha, t2, bits, sizes, budget)
        assert choice.tolist() == [int(j0), int(j1)] and abs(got - obj) < 1e-12
        c2, o2 = hb.higgs_allocate_bits(alpha, t2, (bits * 64).astype(np.int32), sizes, int(budget * 64))
        assert list(c2) == [int(j0), int(j1)] and abs(o2 - obj) < 1e-12
    choice, got = oracle.allocate_bits_bruteforce(alpha, t2, bits, sizes, 1.9)
    assert choice is None and got == np.inf


def test_argument_limits_are_reported_not_wrapped():
    import ctypes
    from paper_2411_17525_b200 import binding
    L, J = 2, 300                                                          # more options than the choice table can index
    alpha = np.ones(L); t2 = np.ones((L, J)); bits = np.arange(1, J + 1, dtype=np.int32); sizes = np.ones(L, dtype=np.int64)
    with pytest.raises(RuntimeError) as e:
        hb.higgs_allocate_bits(alpha, t2, bits, sizes, 64)
    assert e.value.status == hb.HIGGS_ERR_UNSUPPORTED
    alpha, t2, bits64, sizes = instance(4, 3, 1)
    with pytest.raises(RuntimeError) as e:                                 # budget * total would overflow 64 bits
        hb.higgs_allocate_bits(alpha, t2, bits64, sizes, 2 ** 62)
    assert e.value.status == hb.HIGGS_ERR_WORKSPACE
    with pytest.raises(RuntimeError) as e:                                 # a table of more than 2e9 states is refused
        hb.higgs_allocate_bits(np.ones(50), np.ones((50, 3)), bits64, np.arange(1, 51, dtype=np.int64) * 1000003, 10 ** 6)
    assert e.value.status == hb.HIGGS_ERR_WORKSPACE
    with pytest.raises(RuntimeError) as e:
        hb.higgs_allocate_bits(alpha, t2, bits64, sizes, -5)
    assert e.value.status == hb.HIGGS_ERR_INVALID_ARG


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
