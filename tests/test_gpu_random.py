"""Seeded random shapes, grids, batches and output types through the whole path (encode, pack/unpack, linear) against the
oracle: the cases the hand-written parametrisations do not list."""
import numpy as np
import pytest
import torch

import oracle
import paper_2411_17525_b200 as hb
from synth import inputs
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
G = 1024
GRIDS = [(2, 256), (2, 64), (2, 16), (1, 16), (1, 8), (1, 4), (1, 256)]


@pytest.mark.parametrize("seed", range(24))
def test_random_case_matches_oracle(seed):
    rng = np.random.default_rng(1000 + seed)
    p, n = GRIDS[seed % len(GRIDS)]
    N = int(rng.choice([16, 48, 128, 144, 256, 272, 384, 1040]))
    K = int(rng.choice([1024, 2048, 3072, 4096, 7168]))
    if N * K > 2_500_000:
        K = 1024 * max(1, 2_500_000 // (N * 1024))
    B = int(rng.choice([1, 3, 8, 9, 16, 17, 33, 100, 257]))
    xi = int(rng.integers(1, 2 ** 62))
    W = inputs.make_weights(N, K, seed=int(rng.integers(1e9)), bf16=True)
    x = inputs.make_activations(B, K, seed=int(rng.integers(1e9)), lognormal_channels=bool(rng.integers(2)))
    g64, gt = U.grid32(p, n)
    d = hb.make_desc(p, n, N, K, xi)
    _, _, canon = hb.higgs_quantize(d, U.bf16_tensor(W), gt, want_canonical=True)
    q, sc16 = U.oracle_encode(W, G, g64, xi)
    U.compare_codes(canon.cpu().numpy(), q, max_frac=1e-4 + 3.0 / q.codes.size)
    codes = torch.from_numpy(q.codes.astype(np.uint8)).to(U.dev())
    packed = hb.higgs_pack_codes(d, codes)
    assert torch.equal(hb.higgs_unpack_codes(d, packed), codes)
    scales = hb.scales_to_tile_major(torch.from_numpy(sc16).to(U.dev()))
    out_dtype = torch.bfloat16 if seed % 3 == 2 else torch.float32
    y = hb.higgs_linear(d, U.bf16_tensor(x), packed, scales, gt, out_dtype=out_dtype)
    assert hb.higgs_device_status() == hb.HIGGS_OK
    y_ref = oracle.linear_dense(x.astype(np.float64), q.codes, sc16.astype(np.float64), G, g64, xi)
    err = U.linear_error(y.float().cpu().numpy(), y_ref)
    assert err <= 2e-3 + (2.0 ** -8 if out_dtype == torch.bfloat16 else 0.0), (p, n, N, K, B, err)
