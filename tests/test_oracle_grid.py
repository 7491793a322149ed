"""Pins for the oracle's grid fit (Algorithm 2 read as Lloyd's iteration) and MSE evaluation."""
import numpy as np
import pytest

import oracle
from synth import inputs


@pytest.mark.parametrize("n", [4, 8, 16])
def test_1d_lloyd_max_closed_form_matches_published_table(n, golden):
    tab = golden("lloyd_max_gaussian.txt")
    levels, mse = oracle.lloyd_max_1d(n)
    assert abs(mse - tab[f"mse_n{n}"][0]) <= 5e-4 * tab[f"mse_n{n}"][0]
    assert np.allclose(levels, -levels[::-1], atol=1e-9)  # symmetric
    if n in (4, 8):
        assert np.allclose(levels[n // 2:], tab[f"levels_n{n}"], atol=6e-4)
    else:
        assert abs(levels[-1] - tab["levels_n16_outer"][0]) < 1e-3
    # closed-form MSE evaluator agrees with a fine Riemann quadrature of E min_c (x-c)^2
    x = np.linspace(-9, 9, 1_800_001)
    d = np.min((x[:, None] - levels[None, :]) ** 2, axis=1)
    quad = np.trapezoid(d * np.exp(-x * x / 2) / np.sqrt(2 * np.pi), x)
    assert abs(quad - mse) < 1e-8


@pytest.mark.parametrize("n", [2, 4, 8, 16, 32])
def test_uniform_grid_matches_published_table(n, golden):
    """Constrained (uniform) grids: the MSE-optimal step and its error against Max's table of equally spaced levels."""
    tab = golden("uniform_max_gaussian.txt")
    levels, step, mse = oracle.uniform_grid(n)
    assert abs(step - tab[f"step_n{n}"][0]) <= 1e-3 * tab[f"step_n{n}"][0]
    assert abs(mse - tab[f"mse_n{n}"][0]) <= 2e-3 * tab[f"mse_n{n}"][0]
    lv = levels.ravel()
    assert np.allclose(np.diff(lv), step) and np.allclose(lv, -lv[::-1])
    # a uniform grid can never beat the unconstrained Lloyd-Max grid of the same size, and n = 2 coincides with it
    assert mse >= oracle.lloyd_max_1d(n)[1] - 1e-12
    if n == 2:
        assert abs(mse - (1 - 2 / np.pi)) < 1e-9
    # stationarity in the step
    k = np.arange(n) - 0.5 * (n - 1)
    assert oracle.gauss_mse_1d(k * step * 1.01) > mse and oracle.gauss_mse_1d(k * step * 0.99) > mse


def test_gauss_mse_1d_special_cases():
    # one level at 0: MSE = Var = 1; two levels +-sqrt(2/pi): 1 - 2/pi
    assert abs(oracle.gauss_mse_1d([0.0]) - 1.0) < 1e-12
    a = np.sqrt(2 / np.pi)
    assert abs(oracle.gauss_mse_1d([-a, a]) - (1 - 2 / np.pi)) < 1e-12
    assert abs(oracle.lloyd_max_1d(2)[1] - (1 - 2 / np.pi)) < 1e-12


def test_sample_lloyd_1d_close_to_optimum():
    s = inputs.gaussian_samples(1, inputs.grid_sample_seed(1, 16))
    res = oracle.make_grid_lloyd(1, 16, s, max_iters=4000)
    assert res.converged
    opt = oracle.lloyd_max_1d(16)[1]
    mse = oracle.gauss_mse_1d(res.grid[:, 0])
    assert opt <= mse <= opt * 1.004
    assert np.all(np.diff(res.grid[:, 0]) > 0)  # sorted


@pytest.fixture(scope="module")
def fit_p2_n64():
    s = inputs.gaussian_samples(2, inputs.grid_sample_seed(2, 64), log2_count=16)
    return s, oracle.make_grid_lloyd(2, 64, s, max_iters=4000)


def test_lloyd_2d_fixed_point_and_monotone(fit_p2_n64):
    s, res = fit_p2_n64
    assert res.converged and res.iters > 5
    # MSE seen by successive assignment steps never increases
    assert np.all(np.diff(res.mse_hist) <= 1e-15)
    # stationarity: every centre is the mean of the samples nearest to it (numpy brute force)
    d = ((s[:, None, :] - res.grid[None, :, :]) ** 2).sum(-1)
    a = d.argmin(1)
    for c in range(64):
        assert np.allclose(s[a == c].mean(0), res.grid[c], atol=1e-12)
    # lexicographic order
    g = res.grid
    assert all((g[i, 0], g[i, 1]) < (g[i + 1, 0], g[i + 1, 1]) for i in range(63))
    # grid_mse agrees with the numpy brute force
    assert abs(oracle.grid_mse(res.grid, s) - d.min(1).mean() / 2) < 1e-14


def test_lloyd_2d_mse_level(fit_p2_n64, golden):
    _, res = fit_p2_n64
    fresh = inputs.gaussian_samples(2, 991, log2_count=20)
    mse = oracle.grid_mse(res.grid, fresh)
    zador = golden("lloyd_max_gaussian.txt")["zador_p2_n64"][0]
    # the high-resolution estimate ignores the Gaussian tail cells: a fitted grid lands somewhat below it
    assert 0.85 * zador < mse < zador
    # vector quantisation beats the product of two scalar quantisers at equal bits (3 bpw)
    assert mse < oracle.lloyd_max_1d(8)[1]
    assert 0.0290 < mse < 0.0305


def test_stored_grids_are_lloyd_fixed_points():
    """The grids under tests/golden were written by make_grids.py from the oracle alone; check them."""
    from tests.golden import make_grids

    for (p, n) in make_grids.GRIDS:
        g = make_grids.load(p, n)
        assert g.shape == (n, p)
        fresh = inputs.gaussian_samples(p, 4242, log2_count=19)
        mse = oracle.grid_mse(g, fresh)
        lo, hi = {(2, 256): (0.00770, 0.00795), (2, 64): (0.0292, 0.0302), (1, 16): (0.00940, 0.00960), (2, 16): (0.105, 0.1175),
                  (1, 8): (0.0343, 0.0348), (1, 4): (0.1170, 0.1182), (1, 256): (8.0e-5, 9.5e-5)}[(p, n)]     # Lloyd-Max values 0.03454 and 0.1175 for p=1
        assert lo < mse < hi, (p, n, mse)
    # 2-D at 4 bpw beats 1-D at 4 bpw (why the paper prefers p=2)
    f = inputs.gaussian_samples(2, 4243, log2_count=19)
    assert oracle.grid_mse(make_grids.load(2, 256), f) < oracle.lloyd_max_1d(16)[1]
