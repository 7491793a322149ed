"""GPU checks outside the element-wise parity files: the bounded-wait failure path, the library's own sample
generator and seeded grid fit, and producer -> consumer ordering on one stream."""
import numpy as np
import pytest
import torch

import oracle
import paper_2411_17525_b200 as hb
from synth import inputs
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("which", [0, 1])
def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable(which):
    """A barrier nothing arrives at, no copy in flight, a limit of a few hundred polls: the kernel returns, the status
    word reads HIGGS_ERR_TIMEOUT once, clears, and the next product is correct.  Nothing traps or hangs."""
    assert hb.higgs_device_status() == hb.HIGGS_OK
    res = hb.higgs_selftest_wait(which, 300)
    assert hb.higgs_device_status(clear=False) == hb.HIGGS_ERR_TIMEOUT
    got = res.cpu().numpy()
    assert got[0] == 0 and (which == 1 or got[1] == 0)            # every wait of the self-check gave up
    assert hb.higgs_device_status(clear=True) == hb.HIGGS_ERR_TIMEOUT
    assert hb.higgs_device_status() == hb.HIGGS_OK                # cleared
    # the context is intact: a product right after it matches the oracle
    p, n, N, K, B, xi = 2, 256, 128, 2048, (1 if which == 0 else 32), 5
    g64, gt = U.grid32(p, n)
    W = inputs.make_weights(N, K, seed=31, bf16=True)
    q, sc16 = U.oracle_encode(W, 1024, g64, xi)
    d = hb.make_desc(p, n, N, K, xi)
    packed = hb.higgs_pack_codes(d, torch.from_numpy(q.codes.astype(np.uint8)).to(U.dev()))
    sc = hb.scales_to_tile_major(torch.from_numpy(sc16).to(U.dev()))
    x = inputs.make_activations(B, K, seed=32)
    y = hb.higgs_linear(d, U.bf16_tensor(x), packed, sc, gt).cpu().numpy()
    assert hb.higgs_device_status() == hb.HIGGS_OK
    y_ref = oracle.linear_dense(x.astype(np.float64), q.codes, sc16.astype(np.float64), 1024, g64, xi)
    assert U.linear_error(y, y_ref) <= 2e-3


def test_library_samples_are_standard_normal():
    """higgs_gaussian_samples: mean, variance, fourth moment and coordinate independence of 2^20 draws (a Gaussian's
    kurtosis is 3; the tolerances are about five standard errors)."""
    s = hb.higgs_gaussian_samples(2, 12345, 1 << 20).cpu().numpy().astype(np.float64)
    assert s.shape == (1 << 20, 2) and np.all(np.isfinite(s))
    assert np.all(np.abs(s.mean(0)) < 5e-3)
    assert np.all(np.abs(s.var(0) - 1.0) < 8e-3)
    assert np.all(np.abs((s ** 4).mean(0) - 3.0) < 5e-2)
    assert abs(np.mean(s[:, 0] * s[:, 1])) < 5e-3
    assert np.abs(s).max() < 6.0
    t = hb.higgs_gaussian_samples(2, 12346, 1 << 12).cpu().numpy()
    assert not np.array_equal(t, s[: 1 << 12].astype(np.float32))   # another seed, another sample


@pytest.mark.parametrize("p,n", [(2, 64), (1, 16)])
def test_seeded_grid_fit_reaches_the_oracle_grid_quality(p, n):
    """Algorithm 2 with library-drawn samples: the fitted grid is a different, equally valid fixed point, so it is
    judged by its mean-squared error on fresh samples against the stored oracle-fitted grid's (within 1.5 %)."""
    grid, mse, iters = hb.higgs_make_grid_seeded(p, n, 777, log2_samples=18, max_iters=3000)
    assert int(iters) > 0, "the iteration did not terminate"
    g = grid.cpu().numpy().astype(np.float64)
    fresh = np.random.default_rng(99).standard_normal((1 << 20, p))
    mine = oracle.grid_mse(g, fresh)
    ref = oracle.grid_mse(U.grid32(p, n)[0], fresh)
    assert abs(mine - ref) <= 0.015 * ref
    assert abs(float(mse) - mine) <= 0.03 * mine                       # the in-sample figure the call reports


def test_quantize_then_linear_back_to_back_on_one_stream():
    """The product kernel starts its weight copies before the previous kernel of the stream has finished; the encoder
    ends with an ordinary kernel so that those early reads still see its output.  A large layer makes the encoder's
    last kernels long enough for a violation to show."""
    p, n, N, K, B, xi = 2, 256, 4096, 4096, 1, 9
    g64, gt = U.grid32(p, n)
    W = U.bf16_tensor(inputs.make_weights(N, K, seed=77, bf16=True))
    x = inputs.make_activations(B, K, seed=78)
    xt = U.bf16_tensor(x)
    d = hb.make_desc(p, n, N, K, xi)
    packed0, scales0, _ = hb.higgs_quantize(d, W, gt)
    y0 = hb.higgs_linear(d, xt, packed0, scales0, gt)
    torch.cuda.synchronize()
    for _ in range(3):
        packed = torch.zeros_like(packed0)
        scales = torch.zeros_like(scales0)
        ws = torch.empty(hb.higgs_workspace_bytes(d, hb.HIGGS_OP_QUANTIZE), dtype=torch.uint8, device=U.dev())
        torch.cuda.synchronize()
        # no synchronisation between the two calls
        from paper_2411_17525_b200 import binding
        import ctypes
        rc = binding.lib.higgs_quantize(ctypes.byref(d), W.data_ptr(), hb.HIGGS_BF16, gt.data_ptr(), packed.data_ptr(),
                                        scales.data_ptr(), None, ws.data_ptr(), ws.numel(), binding._stream())
        assert rc == hb.HIGGS_OK
        y = hb.higgs_linear(d, xt, packed, scales, gt)
        torch.cuda.synchronize()
        assert torch.equal(packed, packed0)
        assert torch.equal(y, y0)


@pytest.mark.parametrize("mode", ["rows", "k"])
def test_sharded_benchmark_mode_on_one_rank(mode):
    """bench.py --shard runs the sharded-layer entry points on peer-mapped symmetric memory; with one rank the peer list
    is this device alone, which still takes the whole path: symmetric allocation, rendezvous, the epilogue's stores into
    the mapped buffer, the barrier, (k) the slot sum, all inside CUDA graphs.  Its own-shard check must agree with the
    plain product."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29541", NCCL_NVLS_ENABLE="0")
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        env.pop(k, None)
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--shard", mode, "--workload", "llama-3.2-1b",
                          "--grid", "2,256", "--steps", "8", "--warmup", "3"], cwd=root, env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert line["scaling"] == "strong" and line["n_gpus"] == 1 and line["device_status"] == 0
    assert line["config"]["parallelism"] == f"{mode}-sharded x1"
    assert line["own_shard_max_rel_dev"] <= 1e-5
    assert line["value"] > 0
