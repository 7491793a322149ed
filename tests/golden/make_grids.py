"""Writes the stored grids tests use: Lloyd fits (Algorithm 2) computed by the fp64 oracle ONLY.

Run from the repository root:  python -m tests.golden.make_grids
Each grid is fitted on 2^18 seeded N(0, I_p) samples (seed = synth.inputs.grid_sample_seed(p, n)),
started from the first n samples, run until no assignment changes, and stored as fp32-exact
decimal text (the values are rounded to fp32 first, because the library's grid table is fp32 and
both sides of a parity test must see the same table).
"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))

from synth.grids import GRIDS, load, path  # noqa: F401  (tests import the loader from here or from synth.grids)

UNIFORM = {(1, 256)}      # constrained (equally spaced) grids: closed-form optimum of the step, no samples


def main():
    import oracle
    from synth import inputs

    for p, n in GRIDS:
        if os.path.exists(path(p, n)) and "--all" not in sys.argv:
            continue        # stored tables are never rewritten silently
        if (p, n) in UNIFORM:
            levels, step, mse = oracle.uniform_grid(n)
            hdr = (f"MSE-optimal uniform grid (Section 4.3, constrained HIGGS), p={p} n={n}, step {step:.9g}, expected "
                   f"squared error {mse:.6g}; written by tests/golden/make_grids.py from the fp64 oracle; values are fp32-exact")
            np.savetxt(path(p, n), levels.astype(np.float32).astype(np.float64), fmt="%.9g", header=hdr)
            print(p, n, "uniform", step, mse)
            continue
        s = inputs.gaussian_samples(p, inputs.grid_sample_seed(p, n))
        res = oracle.make_grid_lloyd(p, n, s, max_iters=6000)
        g32 = res.grid.astype(np.float32)
        hdr = (f"Lloyd fit of the Gaussian-MSE-optimal grid (Algorithm 2), p={p} n={n}, 2^18 samples, seed "
               f"{inputs.grid_sample_seed(p, n)}, iterations {res.iters}, converged {res.converged}; "
               f"written by tests/golden/make_grids.py from the fp64 oracle; values are fp32-exact")
        np.savetxt(path(p, n), g32.astype(np.float64), fmt="%.9g", header=hdr)
        print(p, n, res.iters, res.converged, res.mse_hist[-1])


if __name__ == "__main__":
    main()
