"""GPU parity tests: the CUDA path (through the C ABI) against the fp64 oracle on the same seeded inputs.

Bars: codes bit-exact except near-ties (oracle margin < 1e-5, GPU code = oracle runner-up, fewer than 1e-4 of
all codes); layer outputs, given identical codes, within max|dy|/max|y| <= 2e-3.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2411_17525_b200 as hb
from synth import inputs
from tests import gpu_util as U

pytestmark = pytest.mark.gpu

G = 1024
Y_TOL = 2e-3


# ----------------------------------------------------------------------------- RHT
@pytest.mark.parametrize("rows,K,dtype", [(1, 1024, "f32"), (3, 2048, "f32"), (5, 4096, "bf16"), (17, 1024, "bf16")])
def test_rht_matches_oracle(rows, K, dtype):
    rng = np.random.default_rng(rows * K)
    x = rng.standard_normal((rows, K)).astype(np.float32)
    xi = inputs.rht_seed(0)
    d = hb.make_desc(2, 256, 16, K, xi)
    if dtype == "bf16":
        x = inputs.bf16_round(x)
        xt = U.bf16_tensor(x)
    else:
        xt = U.f32_tensor(x)
    sg = oracle.signs(xi, K)
    for normalised in (False, True):
        got = hb.higgs_rht(d, xt, normalised).cpu().numpy().astype(np.float64)
        want = np.stack([np.concatenate([oracle.rht(x[r, i * G:(i + 1) * G].astype(np.float64), sg[i * G:(i + 1) * G], normalised)
                                         for i in range(K // G)]) for r in range(rows)])
        scale = np.abs(want).max()
        assert np.max(np.abs(got - want)) <= 2e-6 * scale


# ----------------------------------------------------------------------------- encoder
def run_quantize(W32, p, n, xi, bf16):
    N, K = W32.shape
    d = hb.make_desc(p, n, N, K, xi)
    g64, gt = U.grid32(p, n)
    Wt = U.bf16_tensor(W32) if bf16 else U.f32_tensor(W32)
    packed, scales, canon = hb.higgs_quantize(d, Wt, gt, want_canonical=True)
    torch.cuda.synchronize()
    return d, g64, gt, packed, scales, canon


@pytest.mark.parametrize("p,n,N,K,bf16", [
    (2, 256, 512, 1024, False),     # the single-layer reference configuration (fp32 weights, one group per row)
    (2, 256, 48, 3072, True),       # several groups per row, ragged against any block size
    (2, 64, 80, 2048, True),
    (1, 16, 64, 2048, True),
    (2, 16, 80, 2048, True),        # 2 bits per weight: two codes per byte
    (1, 256, 32, 2048, True),       # constrained 8-bit grid: one byte per input
    (1, 8, 48, 2048, True),         # scalar grids: two codes per table index
    (1, 4, 48, 2048, True),
    (2, 256, 16, 1024, False),      # smallest supported matrix
])
def test_quantize_codes_and_scales(p, n, N, K, bf16):
    W = inputs.make_weights(N, K, seed=inputs.weight_seed(0, n + N), bf16=bf16)
    xi = inputs.rht_seed(0)
    d, g64, gt, packed, scales, canon = run_quantize(W, p, n, xi, bf16)
    q, sc16 = U.oracle_encode(W, G, g64, xi)
    gpu_codes = canon.cpu().numpy()
    assert gpu_codes.shape == q.codes.shape and gpu_codes.max() < n
    U.compare_codes(gpu_codes, q)
    # scales: fp32 norm then fp16 rounding; at most one fp16 ulp from the oracle's, almost all identical
    s_gpu = hb.scales_from_tile_major(scales, N).cpu().numpy()
    assert s_gpu.shape == sc16.shape
    ulp = np.abs(s_gpu.view(np.int16).astype(np.int64) - sc16.view(np.int16).astype(np.int64))
    assert ulp.max() <= 1 and (ulp == 0).mean() > 0.98
    # the packed stream holds exactly the canonical codes
    back = hb.higgs_unpack_codes(d, packed).cpu().numpy()
    assert np.array_equal(back, gpu_codes)
    repacked = hb.higgs_pack_codes(d, canon)
    assert torch.equal(repacked[: hb.higgs_packed_bytes(d)], packed[: hb.higgs_packed_bytes(d)])
    # without the optional canonical output (codes staged in the workspace) the stream is the same
    Wt = U.bf16_tensor(W) if bf16 else U.f32_tensor(W)
    packed2, scales2, none = hb.higgs_quantize(d, Wt, gt, want_canonical=False)
    assert none is None and torch.equal(packed2, packed) and torch.equal(scales2, scales)


def test_quantize_invariants_on_gpu():
    """Power-of-two scaling leaves codes unchanged and scales exact; zero groups stay finite."""
    p, n, N, K = 2, 256, 32, 2048
    xi = 99
    W = inputs.make_weights(N, K, seed=5, bf16=False)
    d, g64, gt, packed, scales, canon = run_quantize(W, p, n, xi, False)
    d2, _, _, packed2, scales2, canon2 = run_quantize(W * 4.0, p, n, xi, False)
    assert torch.equal(canon, canon2) and torch.equal(scales * 4.0, scales2)
    Wz = W.copy()
    Wz[3, :1024] = 0.0
    dz, _, _, _, scz, cz = run_quantize(Wz, p, n, xi, False)
    origin = int(np.argmin((g64 ** 2).sum(1)))
    scz = hb.scales_from_tile_major(scz, N)
    assert float(scz[3, 0]) == 0.0 and bool((cz[3, :512] == origin).all())
    assert torch.equal(cz[4:], canon[4:]) and bool(torch.isfinite(scz.float()).all())


# ----------------------------------------------------------------------------- decode
def run_linear_case(p, n, N, K, B, xi, wseed, xseed, out_dtype=torch.float32, lognormal=False):
    W = inputs.make_weights(N, K, seed=wseed, bf16=True)
    x = inputs.make_activations(B, K, seed=xseed, lognormal_channels=lognormal)
    g64, gt = U.grid32(p, n)
    q, sc16 = U.oracle_encode(W, G, g64, xi)
    d = hb.make_desc(p, n, N, K, xi)
    canon = torch.from_numpy(q.codes.astype(np.uint8)).to(U.dev())
    packed = hb.higgs_pack_codes(d, canon)                       # identical codes on both sides
    scales = hb.scales_to_tile_major(torch.from_numpy(sc16).to(U.dev()))   # storage order only
    y = hb.higgs_linear(d, U.bf16_tensor(x), packed, scales, gt, out_dtype=out_dtype)
    assert hb.higgs_device_status() == hb.HIGGS_OK
    y_ref = oracle.linear_dense(x.astype(np.float64), q.codes, sc16.astype(np.float64), G, g64, xi)
    return y, y_ref


@pytest.mark.parametrize("p,n,N,K,B", [
    (2, 256, 512, 1024, 1),      # reference configuration
    (2, 256, 48, 2048, 1),
    (2, 256, 48, 2048, 3),
    (2, 256, 272, 4096, 8),
    (2, 256, 272, 4096, 9),
    (2, 256, 64, 8192, 16),      # K split over several blocks (atomic accumulation)
    (2, 256, 32, 14336, 1),
    (2, 256, 32, 14336, 16),
    (2, 64, 48, 2048, 1),
    (2, 64, 272, 4096, 4),
    (2, 64, 64, 8192, 16),
    (2, 64, 32, 1024, 12),
    (1, 16, 48, 2048, 1),
    (1, 16, 64, 4096, 16),
    (2, 16, 48, 2048, 1),        # nibble format: one byte looks up the fp16 pairs of two codes
    (2, 16, 272, 4096, 5),
    (2, 16, 272, 4096, 8),
    (2, 16, 64, 8192, 16),
    (2, 16, 32, 14336, 2),
    (2, 16, 144, 1024, 40),      # more tokens than one launch takes (the row count keeps it off the tensor-core path)
    (1, 8, 272, 4096, 4),        # scalar 3-bit grid: six-bit format, two codes per index
    (1, 8, 64, 8192, 16),
    (1, 4, 272, 4096, 8),        # scalar 2-bit grid: nibble format, four codes per byte
    (1, 4, 48, 2048, 1),
    (1, 256, 48, 2048, 1),       # 8-bit scalar codes: a register is put together from two lookups
    (1, 256, 272, 4096, 7),
    (1, 256, 64, 8192, 16),
    (1, 256, 144, 1024, 33),
    (2, 256, 16, 1024, 17),      # more tokens than one launch takes
    (2, 256, 32, 2048, 40),
])
def test_linear_matches_oracle_given_identical_codes(p, n, N, K, B):
    y, y_ref = run_linear_case(p, n, N, K, B, xi=inputs.rht_seed(2), wseed=100 + N, xseed=200 + B)
    assert y.shape == (B, N) and y.dtype == torch.float32
    err = U.linear_error(y.cpu().numpy(), y_ref)
    assert err <= Y_TOL, err
    assert err <= 6e-4, err   # expected level for fp16 operands with fp32 accumulation


def test_linear_bf16_output_and_outlier_channels():
    y, y_ref = run_linear_case(2, 256, 64, 8192, 8, xi=3, wseed=7, xseed=8, out_dtype=torch.bfloat16, lognormal=True)
    assert y.dtype == torch.bfloat16
    # bf16 output rounding (2^-9 relative per element) sits on top of the fp32 result
    err = U.linear_error(y.float().cpu().numpy(), y_ref)
    assert err <= Y_TOL + 2.0 ** -9
    y32, _ = run_linear_case(2, 256, 64, 8192, 8, xi=3, wseed=7, xseed=8, lognormal=True)
    assert U.linear_error(y32.cpu().numpy(), y_ref) <= Y_TOL
    y1, y1_ref = run_linear_case(2, 256, 64, 2048, 2, xi=3, wseed=7, xseed=8, out_dtype=torch.bfloat16)
    assert U.linear_error(y1.float().cpu().numpy(), y1_ref) <= Y_TOL + 2.0 ** -9


def test_end_to_end_quantize_then_linear():
    """GPU encoder feeding GPU decode approximates the unquantised layer at the level the grid's MSE predicts
    (Appendix E: relative error^2 ~= t^2(grid)), and equals the oracle's layer on the oracle's own codes except
    for the few near-tie codes."""
    p, n, N, K, B = 2, 256, 256, 4096, 4
    xi = inputs.rht_seed(2)
    W = inputs.make_weights(N, K, seed=31, bf16=True)
    x = inputs.make_activations(B, K, seed=32)
    d, g64, gt, packed, scales, canon = run_quantize(W, p, n, xi, True)
    y = hb.higgs_linear(d, U.bf16_tensor(x), packed, scales, gt).cpu().numpy().astype(np.float64)
    y0 = x.astype(np.float64) @ W.astype(np.float64).T
    rel = np.linalg.norm(y - y0) / np.linalg.norm(y0)
    assert 0.06 < rel < 0.12          # sqrt(0.0078) = 0.088
    q, sc16 = U.oracle_encode(W, G, g64, xi)
    y_ref = oracle.linear_dense(x.astype(np.float64), q.codes, sc16.astype(np.float64), G, g64, xi)
    assert U.linear_error(y, y_ref) <= Y_TOL


def test_empty_inputs():
    d = hb.make_desc(2, 256, 0, 1024, 1)
    _, gt = U.grid32(2, 256)
    W = torch.empty((0, 1024), dtype=torch.float32, device=U.dev())
    packed, scales, canon = hb.higgs_quantize(d, W, gt, want_canonical=True)
    assert scales.numel() == 0 and canon.shape == (0, 512)
    d = hb.make_desc(2, 256, 16, 1024, 1)
    x = torch.empty((0, 1024), dtype=torch.bfloat16, device=U.dev())
    y = hb.higgs_linear(d, x, torch.zeros(16 * 512, dtype=torch.uint8, device=U.dev()),
                        torch.zeros((1, 1, 16), dtype=torch.float16, device=U.dev()), gt)
    assert y.shape == (0, 16)


# ----------------------------------------------------------------------------- grid fit
@pytest.mark.parametrize("p,n", [(2, 64), (1, 16), (2, 16)])
def test_make_grid_is_a_lloyd_fixed_point_at_the_oracle_mse(p, n):
    s = inputs.gaussian_samples(p, inputs.grid_sample_seed(p, n), log2_count=16)
    st = U.f32_tensor(s)
    grid, mse, iters = hb.higgs_make_grid(p, n, st, max_iters=3000)
    torch.cuda.synchronize()
    g = grid.cpu().numpy().astype(np.float64)
    assert int(iters) > 5, int(iters)                 # converged (negative = ran out of iterations)
    # sorted lexicographically
    keys = [tuple(r) for r in g]
    assert keys == sorted(keys)
    s32 = s.astype(np.float32).astype(np.float64)
    # reported MSE equals the oracle's evaluation of the device grid on the same samples
    assert abs(float(mse) - oracle.grid_mse(g, s32)) <= 1e-5 * float(mse)
    # fixed point: one more oracle Lloyd step from the device grid leaves it in place
    d2 = ((s32[:, None, :] - g[None, :, :]) ** 2).sum(-1)
    a = d2.argmin(1)
    means = np.stack([s32[a == c].mean(0) for c in range(n)])
    assert np.max(np.abs(means - g)) < 5e-6
    # quality: held-out MSE within 1% of the oracle's own fit on the same samples
    ref = oracle.make_grid_lloyd(p, n, s32, max_iters=4000)
    fresh = inputs.gaussian_samples(p, 777, log2_count=20)
    m_dev, m_ref = oracle.grid_mse(g, fresh), oracle.grid_mse(ref.grid, fresh)
    assert abs(m_dev - m_ref) <= 0.01 * m_ref


def test_uniform_grid_fit_matches_oracle():
    """Constrained HIGGS: the device's golden-section search lands on the oracle's step and MSE."""
    for n in (16, 256):
        grid, step, mse = hb.higgs_make_uniform_grid(n)
        levels, step_ref, mse_ref = oracle.uniform_grid(n)
        assert abs(float(step) - step_ref) <= 1e-5 * step_ref
        assert abs(float(mse) - mse_ref) <= 1e-5 * mse_ref
        assert np.allclose(grid.cpu().numpy().astype(np.float64), levels, rtol=1e-5, atol=1e-7)


# ----------------------------------------------------------------------------- dequantisation to the original space
@pytest.mark.parametrize("p,n,N,K", [(2, 256, 48, 2048), (2, 64, 32, 3072), (1, 16, 16, 1024), (2, 16, 32, 2048),
                                     (1, 8, 16, 2048), (1, 4, 16, 1024), (1, 256, 16, 2048)])
def test_dequantize_matches_oracle(p, n, N, K):
    """Appendix F 'Dequantization': LUT restore, inverse rotation, unscale; element by element against the oracle."""
    xi = inputs.rht_seed(2)
    W = inputs.make_weights(N, K, seed=900 + n, bf16=True)
    g64, gt = U.grid32(p, n)
    q, sc16 = U.oracle_encode(W, G, g64, xi)
    d = hb.make_desc(p, n, N, K, xi)
    packed = hb.higgs_pack_codes(d, torch.from_numpy(q.codes.astype(np.uint8)).to(U.dev()))
    scales = hb.scales_to_tile_major(torch.from_numpy(sc16).to(U.dev()))
    W_ref = oracle.dequantize(q.codes, sc16.astype(np.float64), G, g64, xi)
    W_gpu = hb.higgs_dequantize(d, packed, scales, gt).cpu().numpy().astype(np.float64)
    assert W_gpu.shape == (N, K)
    assert np.max(np.abs(W_gpu - W_ref)) <= 2e-6 * np.max(np.abs(W_ref))      # fp32 butterflies over 10 stages
    # and it is the matrix the layer stands for: relative error against W equals the grid's MSE level (Appendix E)
    rel = np.sum((W_gpu - W) ** 2) / np.sum(W.astype(np.float64) ** 2)
    assert rel < 0.25 if n <= 16 else rel < 0.05
    W_bf = hb.higgs_dequantize(d, packed, scales, gt, out_dtype=torch.bfloat16).float().cpu().numpy()
    assert np.max(np.abs(W_bf - W_ref)) <= 2.0 ** -8 * np.max(np.abs(W_ref))


@pytest.mark.parametrize("p,n,N,K", [(2, 256, 64, 2048), (2, 16, 32, 2048), (1, 256, 32, 1024)])
def test_layer_error_matches_oracle(p, n, N, K):
    """Section 5, 'Measuring Grid Parameters': the relative layer error t^2 against the oracle's, and against the
    grid's own expected squared error (Appendix E: they agree for Gaussian-like rotated weights)."""
    xi = inputs.rht_seed(3)
    W = inputs.make_weights(N, K, seed=1200 + n, bf16=True)
    g64, gt = U.grid32(p, n)
    q, sc16 = U.oracle_encode(W, G, g64, xi)
    d = hb.make_desc(p, n, N, K, xi)
    packed = hb.higgs_pack_codes(d, torch.from_numpy(q.codes.astype(np.uint8)).to(U.dev()))
    scales = hb.scales_to_tile_major(torch.from_numpy(sc16).to(U.dev()))
    t2 = hb.higgs_layer_error(d, U.bf16_tensor(W), packed, scales, gt)
    t2_ref = oracle.layer_error(W, q.codes, sc16.astype(np.float64), G, g64, xi)
    assert abs(t2 - t2_ref) <= 2e-4 * t2_ref, (t2, t2_ref)
    mse = oracle.grid_mse(g64, inputs.gaussian_samples(p, 99, log2_count=18))
    assert abs(t2 - mse) <= (0.08 if n < 256 or p == 2 else 0.25) * mse, (t2, mse)


# ----------------------------------------------------------------------------- shared rotation from the first layer
@pytest.mark.parametrize("N,K,B", [(512, 2048, 1), (256, 4096, 2), (128, 1024, 1), (256, 8192, 1), (256, 2048, 8), (256, 2048, 40)])
def test_linear_share_leaves_the_rotated_activations(N, K, B):
    """higgs_linear_share: y equals higgs_linear's, and the rotated activations it leaves behind equal what
    higgs_rotate_activations writes, bit for bit - whether the product kernel emitted them (1-2 tokens, K not split) or a
    rotation kernel did."""
    xi = inputs.rht_seed(8)
    p, n = 2, 256
    d = hb.make_desc(p, n, N, K, xi)
    _, gt = U.grid32(p, n)
    W = inputs.make_weights(N, K, seed=81, bf16=True)
    packed, scales, _ = hb.higgs_quantize(d, U.bf16_tensor(W), gt)
    x = U.bf16_tensor(inputs.make_activations(B, K, seed=82))
    y_ref = hb.higgs_linear(d, x, packed, scales, gt)
    xd_ref = hb.higgs_rotate_activations(d, x)
    xd = torch.full_like(xd_ref, float("nan"))
    y, xd = hb.higgs_linear_share(d, x, packed, scales, gt, xdag_out=xd)
    torch.cuda.synchronize()
    assert hb.higgs_device_status() == hb.HIGGS_OK
    if hb.higgs_rotated_layout(d, B) == 0:            # (the blocked tensor-core layout has padding tokens nobody writes)
        assert torch.equal(xd.view(torch.int16), xd_ref.view(torch.int16))
    if not hb.higgs_linear_uses_atomics(d, B):
        assert torch.equal(y, y_ref)
    else:
        assert U.linear_error(y.cpu().numpy(), y_ref.cpu().numpy().astype(np.float64)) <= 1e-5
    # and a second layer on the shared activations
    d2 = hb.make_desc(p, n, 128, K, xi)
    W2 = inputs.make_weights(128, K, seed=83, bf16=True)
    pk2, sc2, _ = hb.higgs_quantize(d2, U.bf16_tensor(W2), gt)
    if hb.higgs_rotated_layout(d2, B) == hb.higgs_rotated_layout(d, B):
        y2 = hb.higgs_linear_prerotated(d2, xd, pk2, sc2, gt, B=B)
        y2_ref = hb.higgs_linear(d2, x, pk2, sc2, gt)
        assert U.linear_error(y2.cpu().numpy(), y2_ref.cpu().numpy().astype(np.float64)) <= 1e-5


# ----------------------------------------------------------------------------- row-sharded layer, gathered output
@pytest.mark.parametrize("p,n,N,K,B,world,dtype", [
    (2, 256, 512, 2048, 1, 2, torch.float32),       # fused rotation, stores from the flusher warp
    (2, 256, 384, 2048, 8, 3, torch.float32),       # three uneven shards (128-row units)
    (2, 256, 256, 8192, 4, 2, torch.float32),       # K split in the small-batch kernel: workspace sum + copy kernel
    (2, 64, 512, 2048, 16, 2, torch.bfloat16),      # six-bit grid, bf16 output
    (2, 256, 512, 2048, 40, 2, torch.float32),      # tensor-core kernel, cluster K split
    (2, 256, 16896, 1024, 24, 2, torch.bfloat16),   # tensor-core kernel without a K split (66 row tiles per shard)
])
def test_linear_gather_writes_every_destination(p, n, N, K, B, world, dtype):
    """A layer split by rows over `world` shards; each shard's product writes its columns into every destination
    buffer.  One GPU stands in for all devices: the shards' launches run one after the other (they never wait on one
    another) and the destination buffers are separate allocations of this GPU.  Every destination must hold the whole
    [B][N] output, equal to the oracle's."""
    xi = inputs.rht_seed(7)
    W = inputs.make_weights(N, K, seed=70 + n, bf16=True)
    x = inputs.make_activations(B, K, seed=71)
    g64, gt = U.grid32(p, n)
    q, sc16 = U.oracle_encode(W, G, g64, xi)
    y_ref = oracle.linear_dense(x.astype(np.float64), q.codes, sc16.astype(np.float64), G, g64, xi)
    dsts = [torch.full((B, N), float("nan"), dtype=dtype, device=U.dev()) for _ in range(world)]
    xt = U.bf16_tensor(x)
    covered = 0
    for rank in range(world):
        r0, r1 = hb.shard_rows(N, world, rank)
        assert r0 == covered and r1 > r0
        covered = r1
        d = hb.make_desc(p, n, r1 - r0, K, xi)
        codes = torch.from_numpy(q.codes[r0:r1].astype(np.uint8)).to(U.dev())
        packed = hb.higgs_pack_codes(d, codes)
        scales = hb.scales_to_tile_major(torch.from_numpy(sc16[r0:r1]).to(U.dev()))
        # "own buffer first, then the peers'": rank r's own buffer is dsts[r]
        order = [dsts[rank]] + [dsts[o] for o in range(world) if o != rank]
        hb.higgs_linear_gather(d, xt, packed, scales, gt, order, r0)
    torch.cuda.synchronize()
    assert covered == N and hb.higgs_device_status() == hb.HIGGS_OK
    tol = Y_TOL + (2.0 ** -8 if dtype == torch.bfloat16 else 0.0)
    for t in dsts:
        y = t.float().cpu().numpy()
        assert np.isfinite(y).all()
        assert U.linear_error(y, y_ref) <= tol
    for t in dsts[1:]:
        assert torch.equal(t, dsts[0]) or hb.higgs_linear_uses_atomics(hb.make_desc(p, n, hb.shard_rows(N, world, 0)[1], K, xi), B)


def test_linear_gather_argument_checks():
    d = hb.make_desc(2, 256, 128, 1024, 1)
    _, gt = U.grid32(2, 256)
    x = torch.zeros((1, 1024), dtype=torch.bfloat16, device=U.dev())
    packed = torch.zeros(hb.higgs_packed_bytes(d), dtype=torch.uint8, device=U.dev())
    scales = torch.zeros((8, 1, 16), dtype=torch.float16, device=U.dev())
    y = torch.zeros((1, 256), dtype=torch.float32, device=U.dev())
    for off in (8, 144, -16):                       # not a row-tile multiple / beyond the row count / negative
        with pytest.raises(hb.HiggsError) as e:
            hb.higgs_linear_gather(d, x, packed, scales, gt, [y], off)
        assert e.value.status == hb.HIGGS_ERR_INVALID_ARG
    with pytest.raises(hb.HiggsError):
        hb.higgs_linear_gather(d, x, packed, scales, gt, [y] * 9, 0)


# ----------------------------------------------------------------------------- host-buffer entry points
@pytest.mark.parametrize("B", [1, 4, 40])
def test_linear_host_and_host_batch_match_device_path(B):
    """higgs_linear_host / higgs_linear_host_batch (host activations in, host outputs out) give exactly what
    higgs_linear gives on device buffers; layers naming the same host tensor share one copy."""
    xi = inputs.rht_seed(6)
    shapes = [(2, 256, 256, 2048), (2, 256, 128, 2048), (2, 64, 128, 1024)]
    descs, packed, scales, grids, xs, ys_dev = [], [], [], [], [], []
    x_shared = torch.from_numpy(inputs.make_activations(B, 2048, seed=31)).to(torch.bfloat16).pin_memory()
    x_other = torch.from_numpy(inputs.make_activations(B, 1024, seed=32)).to(torch.bfloat16).pin_memory()
    for li, (p, n, N, K) in enumerate(shapes):
        d = hb.make_desc(p, n, N, K, xi)
        # bit-for-bit comparison: the small-batch path must not split K (atomics); the cluster split of the tensor-core
        # path sums in a fixed order
        assert not hb.higgs_linear_uses_atomics(d, B)
        _, gt = U.grid32(p, n)
        W = inputs.make_weights(N, K, seed=40 + li, bf16=True)
        pk, sc, _ = hb.higgs_quantize(d, U.bf16_tensor(W), gt)
        xh = x_shared if K == 2048 else x_other
        descs.append(d); packed.append(pk); scales.append(sc); grids.append(gt); xs.append(xh)
        ys_dev.append(hb.higgs_linear(d, xh.to(U.dev()), pk, sc, gt).cpu())
    ws = [torch.empty(hb.higgs_linear_host_workspace_bytes(d, B), dtype=torch.uint8, device=U.dev()) for d in descs]
    # one call per layer
    for li, d in enumerate(descs):
        yh = torch.empty((B, d.N), dtype=torch.float32).pin_memory()
        hb.higgs_linear_host(d, xs[li], packed[li], scales[li], grids[li], yh, ws[li])
        torch.cuda.synchronize()
        assert torch.equal(yh, ys_dev[li])
    # one call for all
    ys_host = [torch.zeros((B, d.N), dtype=torch.float32).pin_memory() for d in descs]
    batch = hb.HostBatch(descs, xs, packed, scales, grids, ys_host, ws)
    hb.higgs_linear_host_batch(batch)
    torch.cuda.synchronize()
    assert hb.higgs_device_status() == hb.HIGGS_OK
    for li in range(len(descs)):
        assert torch.equal(ys_host[li], ys_dev[li])
    # one pinned block in, one pinned block out (two copies per step); the first two layers share input and grid and run
    # as one product over their concatenated rows
    blk = hb.HostBlock(descs, ["a", "a", "b"], [("a", x_shared), ("b", x_other)], packed, scales, grids, B)
    for _ in range(2):
        for y in blk.y:
            y.fill_(float("nan"))
        hb.higgs_linear_host_block(blk)
        torch.cuda.synchronize()
        assert hb.higgs_device_status() == hb.HIGGS_OK
        for li in range(len(descs)):
            if B <= 2:      # one or two tokens: the merged product rotates in its own kernel; equal to fp16 rounding of x+
                assert U.linear_error(blk.y[li].numpy(), ys_dev[li].numpy().astype(np.float64)) <= 2e-3
            else:
                assert torch.equal(blk.y[li], ys_dev[li])


# ----------------------------------------------------------------------------- general grids (evaluation encoder)
def _random_grid(p, n, seed):
    """n points of N(0, I_p), fp32-exact, sorted lexicographically: a valid grid for encoder parity (the encoder
    does not care whether the grid is optimal)."""
    g = np.random.default_rng(seed).standard_normal((n, p)).astype(np.float32).astype(np.float64)
    return g[np.lexsort(g.T[::-1])]


@pytest.mark.parametrize("p,n,N,K,bf16", [
    (3, 830, 12, 2048, True),     # the paper's 3.25-bit grid: 342 tuples per group, the last one completed with zeros
    (2, 88, 16, 1024, True),      # 3.25 bits, p = 2
    (2, 361, 9, 3072, False),     # 4.25 bits
    (1, 19, 16, 2048, True),      # 4.25 bits, scalar
    (4, 256, 8, 2048, True),      # 2 bits, p = 4
    (4, 4096, 5, 1024, False),    # the largest supported grid (64 KB of fp32)
    (3, 9, 300, 1024, True),      # smallest n of the paper's sweep; more items than one wave of warps
    (2, 256, 16, 2048, True),     # a kernel-supported grid through the general encoder
])
def test_quantize_general_matches_oracle(p, n, N, K, bf16):
    """Algorithm 1 with any grid: codes against the oracle (near-ties counted), scales, and the layer error t^2 the
    same pass accumulates against the oracle's dequantise-and-subtract in the original space."""
    xi = inputs.rht_seed(4)
    W = inputs.make_weights(N, K, seed=3000 + n, bf16=bf16)
    g64 = _random_grid(p, n, 50 + n)
    gt = U.f32_tensor(g64)
    Wt = U.bf16_tensor(W) if bf16 else U.f32_tensor(W)
    codes, scales, t2 = hb.higgs_quantize_general(p, n, Wt, gt, xi)
    torch.cuda.synchronize()
    q, sc16 = U.oracle_encode(W, G, g64, xi)
    T = oracle.tuples_per_group(G, p)
    gc = codes.cpu().numpy().astype(np.int64).reshape(N, (K // G) * T)
    assert gc.min() >= 0 and gc.max() < n
    U.compare_codes(gc, q, max_frac=max(1e-4, 1.5 / gc.size))
    # stored scale: the oracle's value rounded once to fp16, up to one unit in the last place (fp32 norm on the device)
    sg = scales.cpu().numpy()
    assert sg.shape == sc16.shape
    assert np.max(np.abs(sg.astype(np.float64) - sc16.astype(np.float64)) / sc16.astype(np.float64)) <= 2.0 ** -10
    # t^2 from the device's own codes and scales, evaluated by the oracle in the original space
    t2_ref = oracle.layer_error(W, gc.astype(np.int32), sg.astype(np.float64), G, g64, xi)
    assert abs(t2 - t2_ref) <= 2e-4 * t2_ref, (t2, t2_ref)
    if (p, n) == (2, 256):
        d = hb.make_desc(p, n, N, K, xi)
        _, _, canon = hb.higgs_quantize(d, Wt, gt, want_canonical=True)
        assert np.array_equal(canon.cpu().numpy().astype(np.int64), gc)


def test_quantize_general_edge_cases():
    xi = inputs.rht_seed(4)
    g64 = _random_grid(3, 17, 1)
    gt = U.f32_tensor(g64)
    # a zero group: scale 0, finite codes (the point nearest the origin), error 0
    W = np.zeros((2, 1024), dtype=np.float32)
    codes, scales, t2 = hb.higgs_quantize_general(3, 17, U.f32_tensor(W), gt, xi)
    q, _ = U.oracle_encode(W, G, g64, xi)
    assert np.array_equal(codes.cpu().numpy().astype(np.int64).reshape(2, -1), q.codes)
    assert float(scales.abs().max()) == 0.0 and t2 == 0.0
    # empty matrix
    codes, scales, t2 = hb.higgs_quantize_general(3, 17, torch.empty((0, 1024), dtype=torch.float32, device=U.dev()), gt, xi)
    assert codes.numel() == 0 and t2 == 0.0
    # unsupported shapes are refused
    for (pp, nn) in [(5, 16), (2, 4097)]:
        with pytest.raises(hb.HiggsError) as e:
            hb.higgs_quantize_general(pp, nn, U.f32_tensor(np.zeros((1, 1024))), torch.zeros((nn, pp), device=U.dev()), xi)
        assert e.value.status == hb.HIGGS_ERR_UNSUPPORTED
    with pytest.raises(hb.HiggsError) as e:                       # K must be a multiple of the group size
        hb.higgs_quantize_general(3, 17, U.f32_tensor(np.zeros((1, 512))), gt, xi)
    assert e.value.status == hb.HIGGS_ERR_UNSUPPORTED


@pytest.mark.parametrize("p,n,log2m", [(3, 830, 15), (2, 88, 15), (1, 19, 16), (4, 300, 14), (2, 361, 15)])
def test_make_grid_general_is_a_lloyd_fixed_point(p, n, log2m):
    """Algorithm 2 for the grids outside the kernel family: the device's fit is a fixed point of the oracle's Lloyd
    step on the same samples, sorted, with the MSE the oracle computes for it; t^2 of a layer encoded with it agrees
    with that MSE on fresh Gaussian samples (Appendix 'Proof of Expected Error')."""
    s = inputs.gaussian_samples(p, 4000 + n, log2_count=log2m)
    grid, mse, iters = hb.higgs_make_grid(p, n, U.f32_tensor(s), max_iters=3000)
    torch.cuda.synchronize()
    g = grid.cpu().numpy().astype(np.float64)
    assert int(iters) > 3, int(iters)
    keys = [tuple(r) for r in g]
    assert keys == sorted(keys)
    s32 = s.astype(np.float32).astype(np.float64)
    assert abs(float(mse) - oracle.grid_mse(g, s32)) <= 1e-5 * float(mse)
    a = np.concatenate([((c[:, None, :] - g[None, :, :]) ** 2).sum(-1).argmin(1) for c in np.array_split(s32, 64)])
    sums = np.zeros((n, p))
    np.add.at(sums, a, s32)
    cnt = np.bincount(a, minlength=n)
    occupied = cnt > 0
    assert np.max(np.abs(sums[occupied] / cnt[occupied, None] - g[occupied])) < 5e-6
    # rate-distortion sanity: below the scalar Lloyd-Max error at the next lower integer rate, above Shannon's bound
    rate = np.log2(n) / p
    assert 2.0 ** (-2 * rate) < float(mse)
    # the layer error of weights encoded with this grid is the grid's error on fresh samples
    xi = inputs.rht_seed(5)
    W = inputs.make_weights(48, 2048, seed=77 + n, bf16=True)
    _, _, t2 = hb.higgs_quantize_general(p, n, U.bf16_tensor(W), grid, xi)
    fresh = oracle.grid_mse(g, inputs.gaussian_samples(p, 778, log2_count=18))
    assert abs(t2 - fresh) <= 0.06 * fresh, (t2, fresh)


# ----------------------------------------------------------------------------- tensor-core path (B > 16, N % 128 == 0)
@pytest.mark.parametrize("p,n,N,K,B", [
    (2, 256, 128, 1024, 17),     # smallest tile: one block, 16 stages, token tile of 32
    (2, 256, 256, 2048, 64),
    (2, 256, 384, 4096, 100),    # ragged batch (token tile 112)
    (1, 16, 128, 2048, 48),
    (2, 256, 128, 8192, 256),    # full 256-token tile, long K
    (2, 256, 256, 1024, 300),    # two token tiles
    (2, 256, 8448, 1024, 40),    # 66 row tiles: K is not split
    (2, 256, 4096, 3072, 24),    # two K slices of 1536 inputs: the boundary falls inside a scale group
    (2, 64, 128, 2048, 20),      # six-bit format: bit planes rebuilt into index words by the dequant warps
    (2, 64, 384, 4096, 100),
    (2, 64, 8448, 1024, 40),     # six-bit, K not split
    (2, 64, 256, 1024, 300),
    (1, 8, 256, 2048, 64),       # scalar 3-bit grid on the six-bit path
    (2, 16, 128, 1024, 17),      # nibble format: the row's nibbles become the bytes of its index words
    (2, 16, 256, 2048, 64),
    (2, 16, 384, 4096, 100),
    (2, 16, 8448, 1024, 40),     # K not split
    (2, 16, 128, 8192, 256),
    (1, 4, 256, 2048, 64),       # scalar 2-bit grid on the nibble path
    (1, 256, 128, 1024, 17),     # 8-bit scalar codes: two lookups per operand register, 8 KB code stages
    (1, 256, 256, 2048, 64),
    (1, 256, 384, 4096, 100),
    (1, 256, 8448, 1024, 40),
    (1, 256, 128, 8192, 256),
    (1, 256, 256, 1024, 300),
])
def test_linear_tensor_core_path_matches_oracle(p, n, N, K, B):
    y, y_ref = run_linear_case(p, n, N, K, B, xi=inputs.rht_seed(3), wseed=300 + N, xseed=400 + B, lognormal=(B == 64))
    assert y.shape == (B, N)
    err = U.linear_error(y.cpu().numpy(), y_ref)
    assert err <= Y_TOL, err


def test_tensor_core_rotate_then_product_equals_one_call():
    p, n, N, K, B = 2, 256, 256, 2048, 80
    W = inputs.make_weights(N, K, seed=77, bf16=True)
    d = hb.make_desc(p, n, N, K, 11)
    _, gt = U.grid32(p, n)
    packed, scales, _ = hb.higgs_quantize(d, U.bf16_tensor(W), gt)
    x = U.bf16_tensor(inputs.make_activations(B, K, seed=78))
    assert hb.higgs_rotated_layout(d, B) == 80 and hb.higgs_rotated_layout(d, 16) == 0
    y1 = hb.higgs_linear(d, x, packed, scales, gt)
    xd = hb.higgs_rotate_activations(d, x)
    assert xd.numel() * 2 == hb.higgs_rotated_bytes(d, B)
    y2 = hb.higgs_linear_prerotated(d, xd, packed, scales, gt, B=B)
    assert hb.higgs_device_status() == hb.HIGGS_OK
    assert torch.equal(y1, y2)


def test_tensor_core_k_split_is_deterministic():
    """The K slices of a tile are summed in a fixed order inside a cluster: two runs agree bit for bit."""
    p, n, N, K, B = 2, 256, 256, 4096, 96
    d = hb.make_desc(p, n, N, K, 3)
    assert hb.higgs_linear_k_splits(d, B) == 8 and hb.higgs_linear_k_splits(hb.make_desc(p, n, 16384, K, 3), B) == 1
    W = inputs.make_weights(N, K, seed=5, bf16=True)
    _, gt = U.grid32(p, n)
    packed, scales, _ = hb.higgs_quantize(d, U.bf16_tensor(W), gt)
    x = U.bf16_tensor(inputs.make_activations(B, K, seed=6))
    ys = [hb.higgs_linear(d, x, packed, scales, gt).clone() for _ in range(3)]
    assert hb.higgs_device_status() == hb.HIGGS_OK
    assert torch.equal(ys[0], ys[1]) and torch.equal(ys[0], ys[2])


@pytest.mark.parametrize("N,K,B", [(128, 2048, 32),      # K split over a cluster: the reduction writes bf16
                                   (8448, 1024, 40),     # no K split: the parked tile is written out as bf16
                                   (8448, 1024, 300)])   # two token tiles, the second one ragged
def test_linear_tensor_core_path_bf16_output(N, K, B):
    y, y_ref = run_linear_case(2, 256, N, K, B, xi=5, wseed=9, xseed=10, out_dtype=torch.bfloat16)
    assert y.dtype == torch.bfloat16
    assert U.linear_error(y.float().cpu().numpy(), y_ref) <= Y_TOL + 2.0 ** -8


@pytest.mark.parametrize("p,n,N,K,B,dtype", [
    (2, 256, 512, 8192, 1, torch.float32),      # fused rotation, both halves of K in one cluster pair
    (2, 256, 4096, 8192, 2, torch.float32),
    (2, 64, 1040, 8192, 1, torch.bfloat16),     # six-bit planes, ragged row-tile split over the pairs
    (2, 16, 2048, 8192, 2, torch.float32),      # nibble format: partial tiles behind the table
    (1, 256, 2368, 8192, 3, torch.float32),     # 8-bit scalar codes
    (2, 256, 2048, 8192, 5, torch.float32),     # rotation kernel + product, generic flusher
    (1, 16, 1184, 8192, 8, torch.bfloat16),
])
def test_two_k_chunks_meet_in_a_cluster_pair_in_a_fixed_order(p, n, N, K, B, dtype):
    """K ranges of 2 x 4096 inputs at up to eight tokens: the two blocks of a thread-block
    cluster take them, item j is summed by block j % 2 in a fixed order.  Checked against the oracle, bit for bit
    between two runs, and the call must report that it uses no atomics."""
    xi = 2024
    g64, gt = U.grid32(p, n)
    W = inputs.make_weights(N, K, seed=600 + N + B, bf16=True)
    q, sc16 = U.oracle_encode(W, 1024, g64, xi)
    d = hb.make_desc(p, n, N, K, xi)
    assert hb.higgs_linear_k_splits(d, B) == 2 and not hb.higgs_linear_uses_atomics(d, B)
    packed = hb.higgs_pack_codes(d, torch.from_numpy(q.codes.astype(np.uint8)).to(U.dev()))
    sc = hb.scales_to_tile_major(torch.from_numpy(sc16).to(U.dev()))
    x = inputs.make_activations(B, K, seed=601 + B)
    xt = U.bf16_tensor(x)
    y1 = hb.higgs_linear(d, xt, packed, sc, gt, out_dtype=dtype)
    y2 = hb.higgs_linear(d, xt, packed, sc, gt, out_dtype=dtype)
    y3 = hb.higgs_linear_prerotated(d, hb.higgs_rotate_activations(d, xt), packed, sc, gt, out_dtype=dtype)
    torch.cuda.synchronize()
    assert hb.higgs_device_status() == hb.HIGGS_OK
    assert torch.equal(y1, y2)
    y_ref = oracle.linear_dense(x.astype(np.float64), q.codes, sc16.astype(np.float64), 1024, g64, xi)
    tol = Y_TOL + (2.0 ** -8 if dtype == torch.bfloat16 else 0.0)
    assert U.linear_error(y1.float().cpu().numpy(), y_ref) <= tol
    assert U.linear_error(y3.float().cpu().numpy(), y_ref) <= tol


@pytest.mark.parametrize("p,n,N,K,B,world,dtype", [
    (2, 256, 256, 8192, 1, 2, torch.float32),      # shards of 4096 inputs: fused rotation
    (2, 256, 2048, 16384, 2, 2, torch.float32),    # shards of 8192 inputs: cluster pairs
    (2, 64, 128, 4096, 5, 4, torch.bfloat16),      # shards of one group
    (2, 256, 256, 8192, 40, 4, torch.float32),     # tensor-core path, K split inside a cluster
    (2, 256, 64, 28672, 3, 2, torch.float32),      # shards of 14336 inputs: atomics inside a shard, copy kernel spreads
])
def test_k_sharded_layer_sums_to_the_unsharded_output(p, n, N, K, B, world, dtype):
    """higgs_linear_kshard + higgs_reduce_slots with the `world` devices emulated on one GPU (the shards are launched
    one after the other and never wait on one another; every "device" has its own slot buffer): each shard is the
    layer's columns [k0, k0 + K / world) with the shifted seed, and every device's reduced output is the oracle's
    output of the whole layer."""
    xi = 4711
    g64, gt = U.grid32(p, n)
    W = inputs.make_weights(N, K, seed=700 + N, bf16=True)
    q, sc16 = U.oracle_encode(W, 1024, g64, xi)
    x = inputs.make_activations(B, K, seed=701 + B)
    Kr = K // world
    slot_bufs = [torch.full((world, B, N), float("nan"), dtype=torch.float32, device=U.dev()) for _ in range(world)]
    for r in range(world):
        k0 = r * Kr
        d = hb.make_desc(p, n, N, Kr, hb.higgs_shard_seed(xi, k0))
        codes = np.ascontiguousarray(q.codes[:, k0 // p:(k0 + Kr) // p]).astype(np.uint8)
        packed = hb.higgs_pack_codes(d, torch.from_numpy(codes).to(U.dev()))
        sc = hb.scales_to_tile_major(torch.from_numpy(np.ascontiguousarray(sc16[:, k0 // 1024:(k0 + Kr) // 1024])).to(U.dev()))
        xs = U.bf16_tensor(np.ascontiguousarray(x[:, k0:k0 + Kr]))
        # "device" r: its own buffer first in its call, the others as peers
        hb.higgs_linear_kshard(d, xs, packed, sc, gt, slot_bufs, r)
    torch.cuda.synchronize()
    assert hb.higgs_device_status() == hb.HIGGS_OK
    y_ref = oracle.linear_dense(x.astype(np.float64), q.codes, sc16.astype(np.float64), 1024, g64, xi)
    tol = Y_TOL + (2.0 ** -8 if dtype == torch.bfloat16 else 0.0)
    ys = [hb.higgs_reduce_slots(sb, out_dtype=dtype) for sb in slot_bufs]
    for y in ys:
        got = y.float().cpu().numpy()
        assert np.isfinite(got).all()
        assert U.linear_error(got, y_ref) <= tol
    for y in ys[1:]:
        assert torch.equal(y, ys[0])


@pytest.mark.parametrize("p,n,Ns,K,B,dtype", [
    (2, 256, (256, 64, 64), 4096, 1, torch.float32),        # q|k|v: one launch that also rotates
    (2, 256, (1024, 1024), 8192, 2, torch.float32),         # gate|up over cluster pairs
    (2, 64, (272, 48, 16, 528), 2048, 1, torch.bfloat16),   # four matrices, ragged sizes, six-bit planes
    (2, 256, (512, 128, 128), 4096, 5, torch.float32),      # rotation kernel + one product launch
    (1, 16, (320, 320), 4096, 16, torch.float32),           # two token blocks per MMA step
    (2, 16, (256, 256), 2048, 40, torch.float32),           # more than 16 tokens: the tensor-core path per matrix
    (2, 256, (32, 32), 14336, 3, torch.float32),            # few rows, long K: the K ranges meet in atomics, per matrix
])
def test_linear_multi_equals_the_separate_products(p, n, Ns, K, B, dtype):
    """Matrices that read the same activations as one product over their concatenated rows (rows are independent):
    every output equals what higgs_linear gives for that matrix alone - bit for bit where no atomics are involved - and
    the oracle's."""
    xi = 31337
    g64, gt = U.grid32(p, n)
    x = inputs.make_activations(B, K, seed=800 + B)
    xt = U.bf16_tensor(x)
    descs, packed, scales, refs, oracles = [], [], [], [], []
    for i, N in enumerate(Ns):
        W = inputs.make_weights(N, K, seed=810 + 7 * i + N, bf16=True)
        q, sc16 = U.oracle_encode(W, 1024, g64, xi)
        d = hb.make_desc(p, n, N, K, xi)
        pk = hb.higgs_pack_codes(d, torch.from_numpy(q.codes.astype(np.uint8)).to(U.dev()))
        sc = hb.scales_to_tile_major(torch.from_numpy(sc16).to(U.dev()))
        descs.append(d); packed.append(pk); scales.append(sc)
        refs.append(hb.higgs_linear(d, xt, pk, sc, gt, out_dtype=dtype))
        oracles.append(oracle.linear_dense(x.astype(np.float64), q.codes, sc16.astype(np.float64), 1024, g64, xi))
    ys = [torch.full((B, N), float("nan"), dtype=dtype, device=U.dev()) for N in Ns]
    m = hb.MultiLinear(descs, packed, scales, gt, ys, B)
    hb.higgs_linear_multi(m, xt)
    hb.higgs_linear_multi(m, xt)                  # a second call into the same buffers
    torch.cuda.synchronize()
    assert hb.higgs_device_status() == hb.HIGGS_OK
    total = hb.make_desc(p, n, sum(Ns), K, xi)
    one_product = B <= 16 and hb.higgs_rotated_layout(total, B) == 0 and not hb.higgs_linear_uses_atomics(total, B)
    assert m.launches == ((1 if B <= 2 else 1 + (B + 15) // 16) if one_product else sum(hb.higgs_linear_launch_count(d, B) for d in descs))
    tol = Y_TOL + (2.0 ** -8 if dtype == torch.bfloat16 else 0.0)
    for d, y, ref, y_or in zip(descs, ys, refs, oracles):
        got = y.float().cpu().numpy()
        assert np.isfinite(got).all()
        assert U.linear_error(got, y_or) <= tol
        if not hb.higgs_linear_uses_atomics(d, B) and one_product and B > 2:
            assert torch.equal(y, ref)            # same rotation kernel, same fixed-order sums
        else:
            assert U.linear_error(got, ref.float().cpu().numpy().astype(np.float64)) <= 2e-3
