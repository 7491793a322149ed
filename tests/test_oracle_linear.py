"""Pins for the oracle's decode paths (Appendix F): dense definition == rotated-space product."""
import numpy as np
import pytest

import oracle
from synth import inputs
from tests.golden import make_grids


@pytest.mark.parametrize("p,n,g,N,K,B", [(2, 256, 1024, 24, 2048, 3), (2, 64, 1024, 16, 1024, 1), (1, 16, 256, 8, 512, 5)])
def test_dense_equals_rotated(p, n, g, N, K, B):
    grid = make_grids.load(p, n)
    W = inputs.make_weights(N, K, seed=5, bf16=True).astype(np.float64)
    x = inputs.make_activations(B, K, seed=6).astype(np.float64)
    xi = 4711
    q = oracle.quantize(W, g, grid, xi)
    sc = oracle.round_scales_fp16(q.scales).astype(np.float64)
    yd = oracle.linear_dense(x, q.codes, sc, g, grid, xi)
    yr = oracle.linear_rotated(x, q.codes, sc, g, grid, xi)
    assert np.max(np.abs(yd - yr)) <= 1e-12 * np.max(np.abs(yd))
    # and it approximates the unquantised layer to about sqrt(t^2) relative
    y0 = x @ W.T
    rel = np.linalg.norm(yd - y0) / np.linalg.norm(y0)
    assert rel < 2.0 * np.sqrt({256: 0.0078, 64: 0.0296, 16: 0.0095}[n])


def test_matmul_against_numpy():
    rng = np.random.default_rng(1)
    x, w = rng.standard_normal((3, 40)), rng.standard_normal((7, 40))
    assert np.allclose(oracle.matmul_nt(x, w), x @ w.T, atol=1e-12)


def test_rotation_invariance_of_the_product():
    """With exact (unquantised) rotated weights the rotated-space product is x W^T: a one-point-per-weight
    'grid' cannot express that, so check the identity <Hn D x, Hn D w> = <x, w> through rht() itself."""
    g = 256
    rng = np.random.default_rng(2)
    sg = oracle.signs(9, g)
    x, w = rng.standard_normal(g), rng.standard_normal(g)
    assert abs(oracle.rht(x, sg, True) @ oracle.rht(w, sg, True) - x @ w) < 1e-11


def test_single_output_by_hand():
    # g=2, p=1, grid {-1, +1}; K=2, N=1, B=1.  Choose signs away by multiplying inputs with them.
    grid = np.array([[-1.0], [1.0]])
    xi = 31
    sg = oracle.signs(xi, 2)
    w = np.array([3.0, 1.0])
    # w/s = (3,1)/sqrt(10); H2 -> (4,2)/sqrt(10) -> codes (1,1); scale = sqrt(10)/sqrt(2) = sqrt(5)
    q = oracle.quantize((w * sg)[None, :], 2, grid, xi)
    assert q.codes.tolist() == [[1, 1]] and abs(q.scales[0, 0] - np.sqrt(5)) < 1e-14
    # w^ = D Hn (sqrt5, sqrt5) = D (sqrt10, 0);  x = D (2, 7) -> y = 2 sqrt(10)
    x = (np.array([2.0, 7.0]) * sg)[None, :]
    assert abs(oracle.linear_dense(x, q.codes, q.scales, 2, grid, xi)[0, 0] - 2 * np.sqrt(10)) < 1e-13
    assert abs(oracle.linear_rotated(x, q.codes, q.scales, 2, grid, xi)[0, 0] - 2 * np.sqrt(10)) < 1e-13
