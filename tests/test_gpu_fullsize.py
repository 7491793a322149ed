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


@pytest.mark.parametrize("p,n,N,K", [(2, 256, 8192, 2048), (2, 64, 4096, 4096), (1, 256, 8192, 1024), (2, 16, 4096, 2048),
                                     (1, 16, 2048, 4096), (1, 8, 4096, 2048), (1, 4, 8192, 1024)])
def test_pruned_search_equals_exhaustive_scan(p, n, N, K):
    """Large layers are encoded with the exact pruned nearest-point search (which also emits the packed stream), small
    ones with the exhaustive scan and the pack kernel: rows are independent, so re-encoding a slice of the rows as a
    small matrix must give the very same codes, scales and packed bytes.  The same holds for the call with a search
    table prepared beforehand and for the call that lends no workspace (pruned search, then the pack kernel)."""
    cfg = 2
    xi = inputs.rht_seed(cfg)
    W = inputs.make_weights(N, K, inputs.weight_seed(cfg, 5), bf16=True)
    W[7, :] *= 40.0                                     # a row of large values changes nothing (groups are normalised)
    W[9, 100:110] = 3.0                                 # a few huge entries: rotated values beyond the cell table's range
    W = inputs.bf16_round(W)
    _, gt = U.grid32(p, n)
    d = hb.make_desc(p, n, N, K, xi)
    Wt = U.bf16_tensor(W)
    packed, scales, canon = hb.higgs_quantize(d, Wt, gt, want_canonical=True)
    rows = 64
    ds = hb.make_desc(p, n, rows, K, xi)
    packed_s, scales_s, canon_s = hb.higgs_quantize(ds, U.bf16_tensor(W[:rows]), gt, want_canonical=True)
    assert torch.equal(canon[:rows], canon_s)
    assert torch.equal(hb.scales_from_tile_major(scales, N)[:rows], hb.scales_from_tile_major(scales_s, rows))
    nb = hb.higgs_packed_bytes(ds)
    assert torch.equal(packed[:nb], packed_s[:nb])
    # the whole packed stream against the pack kernel on the canonical codes
    assert torch.equal(packed[:hb.higgs_packed_bytes(d)], hb.higgs_pack_codes(d, canon)[:hb.higgs_packed_bytes(d)])
    table = hb.higgs_make_encoder_table(p, n, gt)
    for kwargs in ({"table": table}, {"table": table, "want_canonical": True}, {"want_canonical": True, "workspace": False}, {}):
        packed2, scales2, canon2 = hb.higgs_quantize(d, Wt, gt, **kwargs)
        assert torch.equal(packed2, packed) and torch.equal(scales2, scales), kwargs
        assert canon2 is None or torch.equal(canon2, canon), kwargs
    assert hb.higgs_device_status() == hb.HIGGS_OK


@pytest.mark.parametrize("p,n", [(2, 256), (2, 64), (1, 256), (1, 16)])
def test_pruned_search_on_a_crowded_grid_falls_back_to_the_scan(p, n):
    """A grid that is nothing like the optimal one: its points crowd on a small circle (p = 2) or in a short interval
    (p = 1), with exact duplicates, so cells near the middle have more candidates than a list holds and the encoder
    must take the exhaustive scan for the points that land there - with the lowest index among equal distances."""
    rng = np.random.default_rng(77)
    if p == 2:
        ang = np.sort(rng.uniform(0, 2 * np.pi, n))
        g = np.stack([0.4 * np.cos(ang), 0.4 * np.sin(ang)], axis=1)
    else:
        g = np.sort(rng.uniform(-0.02, 0.02, n))[:, None]
    g[n // 2] = g[n // 2 - 1]                           # a duplicate: equal distances, the lower index must win
    gt = torch.from_numpy(g.astype(np.float32)).to(U.dev())
    N, K, xi = 4096, 1024, inputs.rht_seed(3)
    W = inputs.make_weights(N, K, inputs.weight_seed(3, 1), bf16=True)
    d = hb.make_desc(p, n, N, K, xi)
    packed, scales, canon = hb.higgs_quantize(d, U.bf16_tensor(W), gt, want_canonical=True)
    rows = 32
    ds = hb.make_desc(p, n, rows, K, xi)
    _, _, canon_s = hb.higgs_quantize(ds, U.bf16_tensor(W[:rows]), gt, want_canonical=True)
    assert torch.equal(canon[:rows], canon_s)
    assert int((canon == n // 2).sum()) == 0            # the duplicate with the higher index never wins
    # and the oracle agrees on a few rows (exact ties between duplicates aside, which the rule above settles)
    q, _ = U.oracle_encode(W[:4], G, g.astype(np.float32).astype(np.float64), xi)
    U.compare_codes(canon[:4].cpu().numpy(), q, max_frac=5e-3)
    assert hb.higgs_device_status() == hb.HIGGS_OK


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


@pytest.mark.parametrize("p,n,N,K", [(2, 256, 14336, 4096), (2, 64, 8192, 8192), (1, 16, 4096, 14336)])
def test_encoder_is_reproducible_run_to_run(p, n, N, K):
    """The warps of an encoder block run up to one turn apart and hand their rows over through a shared-memory tile: a
    race there would show as packed bytes that differ between runs, or from the pack kernel on the canonical codes."""
    _, gt = U.grid32(p, n)
    W = U.bf16_tensor(inputs.make_weights(N, K, inputs.weight_seed(2, 9), bf16=True))
    d = hb.make_desc(p, n, N, K, inputs.rht_seed(2))
    table = hb.higgs_make_encoder_table(p, n, gt)
    ref_p, ref_s, ref_c = hb.higgs_quantize(d, W, gt, want_canonical=True, workspace=False)      # search, then the pack kernel
    assert torch.equal(hb.higgs_pack_codes(d, ref_c), ref_p)
    for it in range(12):
        pk, sc, _ = hb.higgs_quantize(d, W, gt, table=table if it % 2 else None)
        assert torch.equal(pk, ref_p) and torch.equal(sc, ref_s), it
    assert hb.higgs_device_status() == hb.HIGGS_OK


@pytest.mark.parametrize("p,n,N,K", [(2, 256, 16, 131072), (2, 64, 48, 65536), (1, 16, 32768, 1024), (2, 256, 32784, 1024)])
def test_encoder_on_extreme_aspect_ratios(p, n, N, K):
    """One row tile with 128 groups, many row tiles with one group, a row count that is not a multiple of the grid of
    blocks: the persistent encoder's (row tile, group) bookkeeping against the pack kernel and the exhaustive scan."""
    _, gt = U.grid32(p, n)
    W = U.bf16_tensor(inputs.make_weights(N, K, inputs.weight_seed(4, 2), bf16=True))
    xi = inputs.rht_seed(4)
    d = hb.make_desc(p, n, N, K, xi)
    packed, scales, canon = hb.higgs_quantize(d, W, gt, want_canonical=True)
    assert torch.equal(hb.higgs_pack_codes(d, canon), packed)
    rows, Ks = 16, min(K, 65536)                        # 16 rows x at most 64 groups: a small layer, exhaustive scan
    ds = hb.make_desc(p, n, rows, Ks, xi)
    _, scales_s, canon_s = hb.higgs_quantize(ds, W[:rows, :Ks].contiguous(), gt, want_canonical=True)
    assert torch.equal(canon[:rows, :Ks // p], canon_s)
    assert torch.equal(hb.scales_from_tile_major(scales, N)[:rows, :Ks // G], hb.scales_from_tile_major(scales_s, rows))
    assert hb.higgs_device_status() == hb.HIGGS_OK
