"""Pins for the oracle's randomised Hadamard transform and sign function (Algorithm 1, Appendix F)."""
import numpy as np
import pytest
import scipy.linalg

import oracle


def explicit_hadamard(g):
    i = np.arange(g)
    pc = np.array([[bin(a & b).count("1") for b in i] for a in i]) if g <= 64 else None
    if pc is None:
        x = i[:, None] & i[None, :]
        pc = np.zeros_like(x)
        while x.any():
            pc += x & 1
            x >>= 1
    return np.where(pc % 2 == 0, 1.0, -1.0)


@pytest.mark.parametrize("g", [1, 2, 4, 8, 64, 1024])
def test_matches_explicit_sylvester_matrix(g):
    rng = np.random.default_rng(g)
    H = explicit_hadamard(g)
    if g > 1:
        assert np.array_equal(H, scipy.linalg.hadamard(g))  # library construction agrees with the popcount form
    v = rng.standard_normal(g)
    s = rng.choice([-1.0, 1.0], size=g)
    got = oracle.rht(v, s, normalised=False)
    assert np.allclose(got, H @ (s * v), rtol=0, atol=1e-10)
    gotn = oracle.rht(v, s, normalised=True)
    assert np.allclose(gotn, H @ (s * v) / np.sqrt(g), rtol=0, atol=1e-11)


def test_by_hand_small_groups():
    assert oracle.rht([5.0], [1.0], False).tolist() == [5.0]
    assert oracle.rht([5.0], [-1.0], True).tolist() == [-5.0]
    assert oracle.rht([1.0, 2.0], [1.0, 1.0], False).tolist() == [3.0, -1.0]
    assert oracle.rht([1.0, 2.0], [1.0, -1.0], False).tolist() == [-1.0, 3.0]
    # H4 rows: ++++ / +-+- / ++-- / +--+
    assert oracle.rht([1.0, 2.0, 3.0, 4.0], [1.0] * 4, False).tolist() == [10.0, -2.0, -4.0, 0.0]


@pytest.mark.parametrize("g", [2, 16, 256, 1024])
def test_orthogonality_norm_involution(g):
    ones = np.ones(g)
    # columns of H from unit vectors: H H^T = g I
    if g <= 256:
        H = np.stack([oracle.rht(np.eye(g)[j], ones, False) for j in range(g)], axis=1)
        assert np.array_equal(H @ H.T, g * np.eye(g))
        assert np.array_equal(H, H.T)
    rng = np.random.default_rng(7 + g)
    u = rng.standard_normal(g)
    v = rng.standard_normal(g)
    s = rng.choice([-1.0, 1.0], size=g)
    ru, rv = oracle.rht(u, s, True), oracle.rht(v, s, True)
    assert abs(np.linalg.norm(ru) - np.linalg.norm(u)) < 1e-12 * np.linalg.norm(u)
    assert abs(ru @ rv - u @ v) < 1e-11
    # involution of the normalised transform without signs; with signs the inverse is D Hn
    assert np.allclose(oracle.rht(oracle.rht(u, ones, True), ones, True), u, atol=1e-12)
    assert np.allclose(s * oracle.rht(ru, ones, True), u, atol=1e-12)


def test_sign_stream_matches_published_splitmix64_vectors(golden):
    g = golden("splitmix64.txt")
    words = [(int(h) << 32) | int(l) for h, l in zip(g["hi32"], g["lo32"])]
    assert words[0] == 0xE220A8397B1DCDAF and words[4] == 0x1B39896A51A8749B
    for m, w in enumerate(words):
        for b in range(64):
            want = -1.0 if (w >> b) & 1 else 1.0
            assert oracle.sign(0, 64 * m + b) == want, (m, b)


def test_sign_properties():
    s = oracle.signs(0x48494747, 8192)
    assert set(np.unique(s)) == {-1.0, 1.0}
    assert abs(s.mean()) < 4 / np.sqrt(len(s))  # balanced Rademacher
    # lag-1 autocorrelation small, different seeds decorrelated
    assert abs(np.mean(s[1:] * s[:-1])) < 4 / np.sqrt(len(s))
    t = oracle.signs(0x48494748, 8192)
    assert abs(np.mean(s * t)) < 4 / np.sqrt(len(s))
    assert np.array_equal(s, oracle.signs(0x48494747, 8192))
