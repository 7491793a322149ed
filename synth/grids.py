"""Stored grid tables: Lloyd fits (Algorithm 2) and the constrained uniform grid, written once by the fp64 oracle
(``python -m tests.golden.make_grids``) and read by tests, the smoke check and the benchmark's CPU arm.

This module only reads text files; it holds none of the method's arithmetic.
"""
import os

import numpy as np

HERE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "grids")
GRIDS = [(2, 256), (2, 64), (1, 16), (2, 16), (1, 8), (1, 4), (1, 256)]


def path(p: int, n: int) -> str:
    return os.path.join(HERE, f"grid_p{p}_n{n}.txt")


def load(p: int, n: int) -> np.ndarray:
    """The stored table as float64 holding exactly the fp32 values (9 printed digits identify an fp32)."""
    g = np.loadtxt(path(p, n), dtype=np.float64, comments="#", ndmin=2)
    return g.astype(np.float32).astype(np.float64).reshape(n, p)
