"""fp64 CPU oracle for the HIGGS quantized linear layer (test infrastructure only).

This package is NOT part of the product.  Only ``tests/``, the smoke check and
the benchmark's CPU-baseline / reference leg may import it.  It shares no code
with the CUDA library and never imports it.

The arithmetic lives in ``higgs_oracle.c`` (plain C, double precision, the
paper's steps in the paper's order); this module only compiles it with gcc,
loads it with ctypes and marshals numpy arrays.

Functions follow Algorithm 1 (RHT-VQ), Algorithm 2 (grid fit, read as Lloyd's
iteration on a Gaussian sample) and Appendix F (dequantisation and the product
in the rotated space) of the paper.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import NamedTuple, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "higgs_oracle.c")
_LIB = os.path.join(_HERE, "libhiggs_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP over rows). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c_d = ctypes.POINTER(ctypes.c_double)
    c_i = ctypes.POINTER(ctypes.c_int32)
    i64, i32, u64 = ctypes.c_int64, ctypes.c_int, ctypes.c_uint64
    lib.higgs_oracle_threads.restype = i32
    lib.higgs_oracle_set_threads.argtypes = [i32]
    lib.higgs_oracle_sign.restype = ctypes.c_double
    lib.higgs_oracle_sign.argtypes = [u64, i64]
    lib.higgs_oracle_rht.argtypes = [c_d, i64, c_d, i32]
    lib.higgs_oracle_lloyd.restype = i32
    lib.higgs_oracle_lloyd.argtypes = [i32, i32, c_d, i64, i32, c_d, c_d, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.higgs_oracle_gauss_mse_1d.restype = ctypes.c_double
    lib.higgs_oracle_gauss_mse_1d.argtypes = [c_d, i32]
    lib.higgs_oracle_lloyd_max_1d.restype = ctypes.c_double
    lib.higgs_oracle_lloyd_max_1d.argtypes = [i32, i32, c_d]
    lib.higgs_oracle_grid_mse.restype = ctypes.c_double
    lib.higgs_oracle_grid_mse.argtypes = [i32, i32, c_d, c_d, i64]
    lib.higgs_oracle_quantize.restype = i32
    lib.higgs_oracle_quantize.argtypes = [c_d, i64, i64, i32, i32, i32, c_d, u64, c_i, c_i, c_d, c_d]
    lib.higgs_oracle_dequantize.restype = i32
    lib.higgs_oracle_dequantize.argtypes = [c_i, c_d, i64, i64, i32, i32, i32, c_d, u64, c_d]
    lib.higgs_oracle_matmul_nt.argtypes = [c_d, c_d, i64, i64, i64, c_d]
    lib.higgs_oracle_linear_rotated.restype = i32
    lib.higgs_oracle_linear_rotated.argtypes = [c_d, i64, c_i, c_d, i64, i64, i32, i32, i32, c_d, u64, c_d]
    _lib = lib
    return lib


def _d(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _pd(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _pi(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def threads() -> int:
    return int(_load().higgs_oracle_threads())


def set_threads(t: int) -> None:
    _load().higgs_oracle_set_threads(int(t))


def sign(xi: int, j: int) -> float:
    """Rademacher sign of input index j under RHT seed xi (Algorithm 1's seed)."""
    return float(_load().higgs_oracle_sign(ctypes.c_uint64(xi & (2**64 - 1)), int(j)))


def signs(xi: int, K: int) -> np.ndarray:
    return np.array([sign(xi, j) for j in range(K)], dtype=np.float64)


def rht(v, sgn, normalised: bool) -> np.ndarray:
    """H diag(sgn) v for one group (Algorithm 1 / Appendix F); /sqrt(g) if normalised."""
    v = _d(v).copy()
    sgn = _d(sgn)
    assert v.ndim == 1 and sgn.shape == v.shape
    _load().higgs_oracle_rht(_pd(v), v.shape[0], _pd(sgn), int(bool(normalised)))
    return v


class LloydResult(NamedTuple):
    grid: np.ndarray  # [n][p], lexicographically sorted
    iters: int
    converged: bool
    mse_hist: np.ndarray  # per-dimension training MSE seen by each assignment step


def make_grid_lloyd(p: int, n: int, samples, max_iters: int = 4000) -> LloydResult:
    """Algorithm 2's grid, fitted by Lloyd's iteration on the given N(0,I_p) samples."""
    s = _d(samples).reshape(-1, p)
    grid = np.zeros((n, p), dtype=np.float64)
    hist = np.full(max_iters, np.nan, dtype=np.float64)
    it, conv = ctypes.c_int(0), ctypes.c_int(0)
    rc = _load().higgs_oracle_lloyd(p, n, _pd(s), s.shape[0], max_iters, _pd(grid), _pd(hist), ctypes.byref(it), ctypes.byref(conv))
    if rc != 0:
        raise ValueError("higgs_oracle_lloyd: bad arguments")
    return LloydResult(grid, it.value, bool(conv.value), hist[: it.value].copy())


def lloyd_max_1d(n: int, iters: int = 20000):
    """Continuous Lloyd-Max fixed point for N(0,1): (levels[n], per-dimension MSE)."""
    lv = np.zeros(n, dtype=np.float64)
    mse = _load().higgs_oracle_lloyd_max_1d(n, iters, _pd(lv))
    return lv, float(mse)


def gauss_mse_1d(levels) -> float:
    """Closed-form MSE of rounding N(0,1) to the sorted 1-D levels."""
    lv = _d(np.sort(np.asarray(levels, dtype=np.float64).ravel()))
    return float(_load().higgs_oracle_gauss_mse_1d(_pd(lv), lv.shape[0]))


def uniform_grid(n: int, iters: int = 200):
    """Constrained HIGGS ("CH", Section 4.3): the uniform n-level grid, symmetric about 0, whose step minimises the
    expected squared error of rounding N(0,1).  Golden-section search on the step over the closed-form MSE.
    Returns (levels[n][1], step, mse)."""
    k = np.arange(n, dtype=np.float64) - 0.5 * (n - 1)
    f = lambda step: gauss_mse_1d(k * step)
    lo, hi = 1e-4, 8.0 / n + 2.0
    r = 0.5 * (np.sqrt(5.0) - 1.0)
    a, b = hi - r * (hi - lo), lo + r * (hi - lo)
    fa, fb = f(a), f(b)
    for _ in range(iters):
        if fa < fb:
            hi, b, fb = b, a, fa
            a = hi - r * (hi - lo)
            fa = f(a)
        else:
            lo, a, fa = a, b, fb
            b = lo + r * (hi - lo)
            fb = f(b)
    step = 0.5 * (lo + hi)
    return (k * step).reshape(n, 1), float(step), float(f(step))


def grid_mse(grid, pts) -> float:
    """Per-dimension MSE of rounding pts[m][p] to grid[n][p] (the t^2 of Appendix E)."""
    g = _d(grid)
    n, p = g.shape
    x = _d(pts).reshape(-1, p)
    return float(_load().higgs_oracle_grid_mse(p, n, _pd(g), _pd(x), x.shape[0]))


def tuples_per_group(g: int, p: int) -> int:
    """Number of p-tuples a group of g rotated values is cut into.  When p does not divide g (the paper's p = 3 grids
    with g = 1024; it does not say how) the last tuple is completed with zeros, matched on all p coordinates, and its
    completed coordinates are dropped on reconstruction."""
    return (g + p - 1) // p


class Quantized(NamedTuple):
    codes: np.ndarray  # int32 [N][(K/g) * tuples_per_group] (= [N][K/p] when p divides g), 0-based
    runner: np.ndarray  # int32, same shape, second-nearest point
    margin: np.ndarray  # float64, same shape, distance to the winner/runner-up bisector
    scales: np.ndarray  # float64 [N][K/g] = ||w||/sqrt(g), unrounded


def quantize(W, g: int, grid, xi: int) -> Quantized:
    """Algorithm 1 on every row of W[N][K], groups of g along K."""
    W = _d(W)
    N, K = W.shape
    gr = _d(grid)
    n, p = gr.shape
    cols = (K // g) * tuples_per_group(g, p)
    codes = np.zeros((N, cols), dtype=np.int32)
    runner = np.zeros((N, cols), dtype=np.int32)
    margin = np.zeros((N, cols), dtype=np.float64)
    scales = np.zeros((N, K // g), dtype=np.float64)
    rc = _load().higgs_oracle_quantize(_pd(W), N, K, g, p, n, _pd(gr), ctypes.c_uint64(xi & (2**64 - 1)), _pi(codes), _pi(runner), _pd(margin), _pd(scales))
    if rc != 0:
        raise ValueError("higgs_oracle_quantize: bad arguments")
    return Quantized(codes, runner, margin, scales)


def round_scales_fp16(scales) -> np.ndarray:
    """Stored scale: rounded once to fp16 (16-bit storage implied by the paper's bit counts)."""
    return np.asarray(scales, dtype=np.float64).astype(np.float16)


def dequantize(codes, scales, g: int, grid, xi: int) -> np.ndarray:
    """Appendix F 'Dequantization': LUT restore, inverse rotation per group, unscale."""
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    gr = _d(grid)
    n, p = gr.shape
    N = codes.shape[0]
    K = codes.shape[1] // tuples_per_group(g, p) * g
    sc = _d(scales)
    assert sc.shape == (N, K // g) and codes.shape[1] == (K // g) * tuples_per_group(g, p)
    out = np.zeros((N, K), dtype=np.float64)
    rc = _load().higgs_oracle_dequantize(_pi(codes), _pd(sc), N, K, g, p, n, _pd(gr), ctypes.c_uint64(xi & (2**64 - 1)), _pd(out))
    if rc != 0:
        raise ValueError("higgs_oracle_dequantize: bad arguments")
    return out


def layer_error(W, codes, scales, g: int, grid, xi: int) -> float:
    """Section 5, 'Measuring Grid Parameters': t^2 = ||W^ - W||_F^2 / ||W||_F^2 with W^ the dequantised layer."""
    Wd = _d(W)
    What = dequantize(codes, scales, g, grid, xi)
    return float(np.sum((What - Wd) ** 2) / np.sum(Wd ** 2))


def allocate_bits_bruteforce(alpha, t2, bits, sizes, budget):
    """Eq. 4 by exhaustive enumeration (tiny instances only): argmin over all J^L assignments of sum_l alpha_l t2[l][j_l]
    subject to sum_l bits[j_l] sizes[l] <= budget * sum_l sizes[l].  Returns (choice, objective) or (None, inf)."""
    import itertools
    a = np.asarray(alpha, dtype=np.float64)
    t = np.asarray(t2, dtype=np.float64)
    b = np.asarray(bits, dtype=np.float64)
    d = np.asarray(sizes, dtype=np.float64)
    L, J = t.shape
    best, arg = np.inf, None
    for js in itertools.product(range(J), repeat=L):
        idx = np.array(js)
        if float(np.dot(b[idx], d)) > budget * float(d.sum()) * (1 + 1e-12):
            continue
        v = float(np.sum(a * t[np.arange(L), idx]))
        if v < best - 1e-15:
            best, arg = v, idx
    return arg, best


def matmul_nt(x, What) -> np.ndarray:
    x = _d(x)
    What = _d(What)
    B, K = x.shape
    N = What.shape[0]
    assert What.shape[1] == K
    y = np.zeros((B, N), dtype=np.float64)
    _load().higgs_oracle_matmul_nt(_pd(x), _pd(What), B, N, K, _pd(y))
    return y


def linear_dense(x, codes, scales, g: int, grid, xi: int) -> np.ndarray:
    """y = x What^T with What from dequantize(): the definition of the layer."""
    return matmul_nt(x, dequantize(codes, scales, g, grid, xi))


def linear_rotated(x, codes, scales, g: int, grid, xi: int) -> np.ndarray:
    """Appendix F 'Rotating Activations': the same product without leaving the rotated space."""
    x = _d(x)
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    gr = _d(grid)
    n, p = gr.shape
    B, K = x.shape
    N = codes.shape[0]
    sc = _d(scales)
    y = np.zeros((B, N), dtype=np.float64)
    rc = _load().higgs_oracle_linear_rotated(_pd(x), B, _pi(codes), _pd(sc), N, K, g, p, n, _pd(gr), ctypes.c_uint64(xi & (2**64 - 1)), _pd(y))
    if rc != 0:
        raise ValueError("higgs_oracle_linear_rotated: bad arguments")
    return y
