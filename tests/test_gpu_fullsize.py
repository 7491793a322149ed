"""Parity at the benchmark's full layer sizes, through the same entry points and launch configuration bench.py
times.  The oracle cannot afford whole layers, so it computes SAMPLED rows (rows are independent in Algorithm 1
and Appendix F): the GPU encodes the whole matrix, the sampled rows are compared code by code with the oracle, then
those rows' codes and scales are replaced by the oracle's ("given identical codes") and the layer output is compared
on the sampled rows."""
import numpy as np
import pytest
import torch

import oracle
import paper_2411_17525_b200 as hb
from synth import inputs
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
G = 1024


def sampled_rows(N, count, seed):
    rng = np.random.default_rng(seed)
    rows = set(range(16)) | set(range(N - 16, N)) | set(rng.choice(N, size=count, replace=False).tolist())
    return np.array(sorted(rows))


@pytest.mark.parametrize("name,N,K,p,n,batches", [
    ("1b-gate", 8192, 2048, 2, 256, (1, 16)),
    ("1b-down", 2048, 8192, 2, 256, (1, 16)),       # K split over thread blocks
    ("1b-kv", 512, 2048, 2, 256, (1,)),
    ("8b-gate-3bit", 14336, 4096, 2, 64, (1, 4)),
    ("8b-q-p1", 4096, 4096, 1, 16, (16,)),
    ("8b-gate-tensor", 14336, 4096, 2, 256, (64, 256)),   # tensor-core regime, outlier channels (log-normal scales)
    ("8b-down-tensor", 4096, 14336, 2, 256, (64,)),       # K split over a thread-block cluster
    ("8b-gate-2bit", 14336, 4096, 2, 16, (1,)),
    ("70b-gate-3bit", 28672, 8192, 2, 64, (1, 32)),       # K in two chunks: cluster pairs
    ("70b-gate-4bit", 28672, 8192, 2, 256, (1, 32)),      # the largest code stream of the benchmark's configurations (117.9 MB)
    ("70b-down-4bit", 8192, 28672, 2, 256, (1, 32)),      # 28 groups: K split over seven thread blocks (atomics) / a cluster
    ("70b-q-3bit", 8192, 8192, 2, 64, (1, 32)),
    ("70b-k-4bit", 1024, 8192, 2, 256, (1, 32)),
    ("8b-gate-p1", 14336, 4096, 1, 16, (4,)),
])
def test_full_size_layer_on_sampled_rows(name, N, K, p, n, batches):
    cfg = 1
    xi = inputs.rht_seed(cfg)
    W = inputs.make_weights(N, K, inputs.weight_seed(cfg, N % 97), bf16=True)
    g64, gt = U.grid32(p, n)
    d = hb.make_desc(p, n, N, K, xi)
    packed, scales, canon = hb.higgs_quantize(d, U.bf16_tensor(W), gt, want_canonical=True)
    rows = sampled_rows(N, 48, seed=N + K)
    q, sc16 = U.oracle_encode(W[rows], G, g64, xi)
    # encoder parity on the sampled rows
    gpu_codes = canon[torch.from_numpy(rows).to(U.dev())].cpu().numpy()
    U.compare_codes(gpu_codes, q, max_frac=2e-4)     # a sample of ~1e5..1e6 codes: allow a couple of near-ties
    s_gpu = hb.scales_from_tile_major(scales, N)[torch.from_numpy(rows).to(U.dev())].cpu().numpy()
    ulp = np.abs(s_gpu.view(np.int16).astype(np.int64) - sc16.view(np.int16).astype(np.int64))
    assert ulp.max() <= 1
    # identical codes and scales on the sampled rows, then the layer as bench.py runs it
    ridx = torch.from_numpy(rows).to(U.dev())
    canon[ridx] = torch.from_numpy(q.codes.astype(np.uint8)).to(U.dev())
    sc_rows = hb.scales_from_tile_major(scales, N)
    sc_rows[ridx] = torch.from_numpy(sc16).to(U.dev())
    packed2 = hb.higgs_pack_codes(d, canon)
    scales2 = hb.scales_to_tile_major(sc_rows)
    for B in batches:
        x = inputs.make_activations(B, K, inputs.activation_seed(cfg, B), lognormal_channels=B >= 64)
        y = hb.higgs_linear(d, U.bf16_tensor(x), packed2, scales2, gt)
        assert hb.higgs_device_status() == hb.HIGGS_OK
        y_ref = oracle.linear_dense(x.astype(np.float64), q.codes, sc16.astype(np.float64), G, g64, xi)
        got = y.cpu().numpy()[:, rows]
        err = float(np.max(np.abs(got - y_ref)) / np.max(np.abs(y_ref)))
        assert err <= 2e-3, (name, B, err)
        # the same deviation against the typical output size (rms) instead of the largest output
        assert U.linear_error_rms(got, y_ref) <= 6e-3, (name, B, U.linear_error_rms(got, y_ref))
        # every output (not only the sampled rows) is finite and of the magnitude the weights imply
        assert bool(torch.isfinite(y).all())
        # the split rotation + product entry points give the same result as the one-call form
        xd = hb.higgs_rotate_activations(d, U.bf16_tensor(x))
        y2 = hb.higgs_linear_prerotated(d, xd, packed2, scales2, gt, B=B)
        assert float((y2 - y).abs().max()) <= 1e-5 * float(y.abs().max())


@pytest.mark.parametrize("p,n,N,K", [(2, 256, 8192, 2048), (2, 64, 4096, 4096), (1, 256, 8192, 1024)])
def test_pruned_search_equals_exhaustive_scan(p, n, N, K):
    """Large layers are encoded with the exact pruned nearest-point search, small ones with the exhaustive scan: rows are
    independent, so re-encoding a slice of the rows as a small matrix must give the very same codes and scales."""
    cfg = 2
    xi = inputs.rht_seed(cfg)
    W = inputs.make_weights(N, K, inputs.weight_seed(cfg, 5), bf16=True)
    W[7, :] *= 40.0                                     # a row of large values changes nothing (groups are normalised)
    W[9, 100:110] = 3.0                                 # a few huge entries: rotated values beyond the cell table's range
    W = inputs.bf16_round(W)
    _, gt = U.grid32(p, n)
    d = hb.make_desc(p, n, N, K, xi)
    packed, scales, canon = hb.higgs_quantize(d, U.bf16_tensor(W), gt, want_canonical=True)
    rows = 64
    ds = hb.make_desc(p, n, rows, K, xi)
    packed_s, scales_s, canon_s = hb.higgs_quantize(ds, U.bf16_tensor(W[:rows]), gt, want_canonical=True)
    assert torch.equal(canon[:rows], canon_s)
    assert torch.equal(hb.scales_from_tile_major(scales, N)[:rows], hb.scales_from_tile_major(scales_s, rows))


def test_general_grid_encoder_full_size_on_sampled_rows():
    """The 3.25-bit grid (p, n) = (3, 830) of the paper's experiment configurations on the 8B q/o matrix: the whole
    matrix is encoded on the device, sampled rows are compared with the oracle code by code, and the device's t^2 for
    the whole layer is bracketed by the oracle's t^2 on the sample."""
    p, n, N, K = 3, 830, 4096, 4096
    xi = inputs.rht_seed(1)
    W = inputs.make_weights(N, K, inputs.weight_seed(1, 5), bf16=True)
    s = inputs.gaussian_samples(p, inputs.grid_sample_seed(p, n), log2_count=16)
    grid, _, _ = hb.higgs_make_grid(p, n, U.f32_tensor(s), max_iters=500)
    g64 = grid.cpu().numpy().astype(np.float64)
    codes, scales, t2 = hb.higgs_quantize_general(p, n, U.bf16_tensor(W), grid, xi)
    rows = sampled_rows(N, 16, seed=9)
    q, sc16 = U.oracle_encode(W[rows], G, g64, xi)
    gc = codes.cpu().numpy().astype(np.int64)[rows].reshape(len(rows), -1)
    U.compare_codes(gc, q, max_frac=2e-4)
    sg = scales.cpu().numpy()[rows]
    ulp = np.abs(sg.view(np.int16).astype(np.int64) - sc16.view(np.int16).astype(np.int64))
    assert ulp.max() <= 1
    t2_rows = oracle.layer_error(W[rows], q.codes, sc16.astype(np.float64), G, g64, xi)
    assert abs(t2 - t2_rows) <= 0.03 * t2_rows, (t2, t2_rows)
