"""Pins for the oracle's encoder (Algorithm 1) against brute force, hand-worked values and invariants."""
import numpy as np
import pytest
import scipy.linalg
import scipy.stats

import oracle
from synth import inputs
from tests.golden import make_grids


def brute_force_encode(W, g, grid, sgn):
    """Independent numpy restatement: explicit Hadamard matrix from scipy, argmin over all points."""
    N, K = W.shape
    n, p = grid.shape
    H = scipy.linalg.hadamard(g).astype(np.float64) if g > 1 else np.ones((1, 1))
    codes = np.zeros((N, K // p), dtype=np.int64)
    scales = np.zeros((N, K // g))
    for r in range(N):
        for i in range(K // g):
            w = W[r, i * g:(i + 1) * g]
            s = np.sqrt((w * w).sum())
            wd = H @ (sgn[i * g:(i + 1) * g] * w / s)
            t = wd.reshape(-1, p)
            d = ((t[:, None, :] - grid[None, :, :]) ** 2).sum(-1)
            codes[r, i * (g // p):(i + 1) * (g // p)] = d.argmin(1)
            scales[r, i] = s / np.sqrt(g)
    return codes, scales


def test_hand_worked_example(golden):
    ref = golden("worked_g4.txt")
    grid = np.array([[-0.8, -0.8], [-0.8, 0.8], [0.8, -0.8], [0.8, 0.8]])
    W = np.array([ref["w"]])
    # seed whose first four signs are all +1 is not needed: check through rht() with explicit signs,
    # then through quantize() by undoing the seed's signs on the input.
    wd = oracle.rht(W[0] / np.linalg.norm(W[0]), np.ones(4), False)
    assert np.allclose(wd, ref["wdag"], atol=1e-6)
    xi = 12345
    sg = oracle.signs(xi, 4)
    q = oracle.quantize(W * sg[None, :], 4, grid, xi)  # diag(sign) cancels
    assert q.codes.tolist() == [[int(c) for c in ref["codes"]]]
    assert abs(q.scales[0, 0] - ref["scale"][0]) < 1e-6
    assert abs(q.margin[0, 0]) < 1e-12 and q.runner[0, 0] == 3        # exact tie, lowest index wins
    assert abs(q.margin[0, 1] - ref["margin1"][0]) < 1e-6 and q.runner[0, 1] in (1, 2)
    What = oracle.dequantize(q.codes, q.scales, 4, grid, xi) * sg[None, :]
    assert np.allclose(What[0], ref["what"], atol=1e-6)
    rel = ((What - W) ** 2).sum() / (W ** 2).sum()
    assert abs(rel - ref["relerr"][0]) < 1e-6
    # the error-database helper itself on the same instance (its W carries the seed's signs, like quantize's input)
    assert abs(oracle.layer_error(W * sg[None, :], q.codes, q.scales, 4, grid, xi) - ref["relerr"][0]) < 1e-6
    x = np.ones((1, 4)) * sg[None, :]
    assert abs(oracle.linear_dense(x, q.codes, q.scales, 4, grid, xi)[0, 0] - ref["y"][0]) < 1e-6
    assert abs(oracle.linear_rotated(x, q.codes, q.scales, 4, grid, xi)[0, 0] - ref["y"][0]) < 1e-6


def test_layer_error_divides_by_the_norm_of_w_not_of_its_reconstruction():
    """Section 5, 'Measuring Grid Parameters': t^2 = ||W^ - W||^2 / ||W||^2.  One group of g = 2 with a one-point grid
    at the origin makes W^ = 0 whatever W is, so t^2 = 1 exactly (dividing by ||W^||^2 would divide by zero); a
    one-point grid at (1, 1) with w = (3, 4), all by hand: s = 5, stored scale 5 / sqrt 2, rotated reconstruction
    r = (5 / sqrt 2) (1, 1), w^ = diag(sign) (H2 / sqrt 2) r = diag(sign) (5, 0); with signs (+, +):
    ||w^ - w||^2 = 4 + 16 = 20, ||w||^2 = 25, t^2 = 0.8 (and ||w^||^2 = 25 too, so a second case with ||w^|| != ||w||:
    two rows w = (3, 4) and (0, 1) -> w^ rows (5, 0) and (1, 0): errors 20 + 2 = 22 over 25 + 1 = 26)."""
    xi = 4242
    sg = oracle.signs(xi, 2)
    W = np.array([[3.0, 4.0]]) * sg[None, :]
    zero = np.zeros((1, 2))
    q0 = oracle.quantize(W, 2, zero, xi)
    assert abs(oracle.layer_error(W, q0.codes, q0.scales, 2, zero, xi) - 1.0) < 1e-12
    one = np.ones((1, 2))
    q1 = oracle.quantize(W, 2, one, xi)
    assert abs(oracle.layer_error(W, q1.codes, q1.scales, 2, one, xi) - 0.8) < 1e-12
    W2 = np.array([[3.0, 4.0], [0.0, 1.0]]) * sg[None, :]
    q2 = oracle.quantize(W2, 2, one, xi)
    assert abs(oracle.layer_error(W2, q2.codes, q2.scales, 2, one, xi) - 22.0 / 26.0) < 1e-12


@pytest.mark.parametrize("g,p,n", [(2, 1, 2), (4, 1, 4), (4, 2, 4), (8, 2, 16), (64, 2, 64), (64, 1, 16), (1024, 2, 256)])
def test_matches_brute_force(g, p, n):
    rng = np.random.default_rng(100 * g + n)
    grid = make_grids.load(p, n) if (p, n) in make_grids.GRIDS else np.sort(rng.standard_normal((n, p)), axis=0)
    N, K = (6, 3 * g) if g < 1024 else (3, 2048)
    W = rng.standard_normal((N, K)) * 0.02
    xi = 77 + g
    sg = oracle.signs(xi, K)
    q = oracle.quantize(W, g, grid, xi)
    codes, scales = brute_force_encode(W, g, grid, sg)
    clear = q.margin > 1e-9
    assert np.array_equal(q.codes[clear], codes[clear])
    assert clear.mean() > 0.99
    assert np.allclose(q.scales, scales, rtol=1e-13)
    assert q.codes.min() >= 0 and q.codes.max() < n
    # margins really are distances to the bisector: moving the rotated point by less than the margin keeps the code
    assert np.all(q.margin >= 0)
    assert np.all(q.runner != q.codes)


@pytest.mark.parametrize("g,p,n", [(16, 3, 7), (64, 3, 40), (1024, 3, 830), (8, 4, 9), (32, 3, 5)])
def test_ragged_tuples_match_brute_force(g, p, n):
    """p need not divide g (the paper's (p, n) = (3, 830) with g = 1024): the last tuple is completed with zeros and
    matched on all p coordinates; reconstruction drops the completed coordinates.  Independent restatement with an
    explicit Hadamard matrix."""
    rng = np.random.default_rng(7 * g + n)
    grid = rng.standard_normal((n, p))
    grid = grid[np.lexsort(grid.T[::-1])]
    N, K = (4, 2 * g) if g < 1024 else (2, 1024)
    W = rng.standard_normal((N, K)) * 0.02
    xi = 1234 + g
    sg = oracle.signs(xi, K)
    H = scipy.linalg.hadamard(g).astype(np.float64)
    T = -(-g // p)
    assert oracle.tuples_per_group(g, p) == T
    q = oracle.quantize(W, g, grid, xi)
    assert q.codes.shape == (N, (K // g) * T)
    What = np.zeros_like(W)
    for r in range(N):
        for i in range(K // g):
            w = W[r, i * g:(i + 1) * g]
            s = np.sqrt((w * w).sum())
            wd = np.concatenate([H @ (sg[i * g:(i + 1) * g] * w / s), np.zeros(T * p - g)]).reshape(T, p)
            d = ((wd[:, None, :] - grid[None, :, :]) ** 2).sum(-1)
            sl = slice((r * 0) + i * T, i * T + T)
            clear = q.margin[r, sl] > 1e-9
            assert np.array_equal(q.codes[r, sl][clear], d.argmin(1)[clear]) and clear.mean() > 0.98
            rec = (s / np.sqrt(g)) * grid[q.codes[r, sl]].reshape(-1)[:g]
            What[r, i * g:(i + 1) * g] = sg[i * g:(i + 1) * g] * (H @ rec) / np.sqrt(g)
    assert np.allclose(oracle.dequantize(q.codes, q.scales, g, grid, xi), What, atol=1e-13)
    # the paper's bit count for this grid: ceil(1024/3) codes of log2(830) bits plus a 16-bit scale per 1024 weights
    assert round(np.log2(830) / 3 + 16 / 1024, 2) == 3.25 and round(342 * np.log2(830) / 1024 + 16 / 1024, 2) == 3.25


def test_margin_is_distance_to_bisector():
    grid = np.array([[0.0, 0.0], [2.0, 0.0], [0.0, 5.0]])
    # g=2 group whose rotated tuple is (0.6, 0.1)*: choose w so that H2 (w/s) = t
    t = np.array([0.6, 0.8])  # unit norm * sqrt(2)/sqrt(2): w+ has norm sqrt(g)=sqrt(2) -> rescale
    t = t * np.sqrt(2)
    w = 0.5 * np.array([t[0] + t[1], t[0] - t[1]])  # H2^{-1} t = H2 t / 2
    xi = 5
    sg = oracle.signs(xi, 2)
    q = oracle.quantize((w * sg)[None, :], 2, grid, xi)
    # t = (0.8485, 1.1314): nearest is (0,0)? d0=2.0, d1=(1.1515^2+1.28)=2.606, d2=0.72+14.96 -> code 0, runner 1
    assert q.codes[0, 0] == 0 and q.runner[0, 0] == 1
    # bisector of (0,0),(2,0) is the line x=1; distance of t to it = 1 - 0.8485
    assert abs(q.margin[0, 0] - (1 - t[0])) < 1e-12


def test_invariances():
    grid = make_grids.load(2, 64)
    rng = np.random.default_rng(3)
    W = rng.standard_normal((8, 256)) * 0.02
    xi = 99
    q = oracle.quantize(W, 128, grid, xi)
    # power-of-two scaling: same codes, scales scale exactly
    q2 = oracle.quantize(W * 8.0, 128, grid, xi)
    assert np.array_equal(q.codes, q2.codes) and np.array_equal(q.scales * 8.0, q2.scales)
    # row permutation commutes
    perm = rng.permutation(8)
    qp = oracle.quantize(W[perm], 128, grid, xi)
    assert np.array_equal(qp.codes, q.codes[perm]) and np.array_equal(qp.scales, q.scales[perm])
    # stacking rows == separate calls
    qa, qb = oracle.quantize(W[:3], 128, grid, xi), oracle.quantize(W[3:], 128, grid, xi)
    assert np.array_equal(np.vstack([qa.codes, qb.codes]), q.codes)
    # a different seed changes the codes
    assert not np.array_equal(oracle.quantize(W, 128, grid, xi + 1).codes, q.codes)


def test_zero_group_is_finite():
    grid = make_grids.load(2, 64)
    W = np.zeros((2, 256))
    W[1, :128] = 1.0
    q = oracle.quantize(W, 128, grid, 1)
    origin = int(np.argmin((grid ** 2).sum(1)))
    assert np.all(q.codes[0] == origin) and np.all(q.scales[0] == 0)
    assert np.all(q.codes[1, 64:] == origin) and q.scales[1, 1] == 0 and q.scales[1, 0] == 1.0
    assert np.all(np.isfinite(q.margin))
    assert np.all(oracle.dequantize(q.codes, q.scales, 128, grid, 1)[0] == 0)


def test_expected_error_identity_and_gaussianisation():
    """Appendix E: ||W^ - W||_F^2 / ||W||_F^2 ~= per-dimension MSE of the grid, whatever the weights;
    Algorithm 1's comment: rotated entries are approximately N(0,1)."""
    g = 1024
    grid = make_grids.load(2, 256)
    W = inputs.make_weights(96, 2048, seed=11, bf16=False).astype(np.float64)
    assert scipy.stats.kurtosis(W.ravel()) > 20  # heavy-tailed input (outliers)
    xi = inputs.rht_seed(0)
    q = oracle.quantize(W, g, grid, xi)
    What = oracle.dequantize(q.codes, q.scales, g, grid, xi)
    rel = ((What - W) ** 2).sum() / (W ** 2).sum()
    t2 = oracle.grid_mse(grid, inputs.gaussian_samples(2, 555, log2_count=20))
    assert abs(rel - t2) < 0.03 * t2
    # rotated, unit-norm-scaled weights look standard normal
    sg = oracle.signs(xi, 2048)
    wd = np.concatenate([oracle.rht(W[r, :g] / np.linalg.norm(W[r, :g]), sg[:g], False) for r in range(96)])
    assert abs(wd.std() - 1.0) < 1e-3
    assert abs(scipy.stats.kurtosis(wd)) < 0.15
    # bit accounting of the paper's configurations: b = log2(n)/p plus 16-bit scale per 1024 weights
    assert round(np.log2(256) / 2 + 16 / 1024, 2) == 4.02
    assert round(np.log2(88) / 2 + 16 / 1024, 2) == 3.25
    assert round(np.log2(361) / 2 + 16 / 1024, 2) == 4.26
