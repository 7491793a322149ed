"""higgs_linear_static: the workspace-free variant for callers that cannot allocate device memory
(no cudaMalloc allowed where they run, or they only own their input/output buffers).  It must give what
higgs_linear gives, on repeated calls that reuse the library's built-in scratch array, and must refuse
shapes that do not fit that array.  Collected last so a failure here cannot hide the other tests."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2411_17525_b200 as hb
from paper_2411_17525_b200 import binding
from synth import inputs
from tests import gpu_util as U

pytestmark = pytest.mark.gpu

Y_TOL = 2e-3


def make_layer(p, n, N, K, xi, seed):
    W = inputs.make_weights(N, K, seed=seed, bf16=True)
    d = hb.make_desc(p, n, N, K, xi)
    g64, gt = U.grid32(p, n)
    packed, scales, canon = hb.higgs_quantize(d, U.bf16_tensor(W), gt, want_canonical=True)
    return d, g64, gt, packed, scales, canon


# Every case below really goes through the built-in array: with three or sixteen tokens the rotation kernel writes the
# rotated activations there, and the two-token case has its K range split over thread blocks, so the rotated
# activations AND the fp32 staging copy of the bf16 output live there.  (One or two tokens with K in one piece would take
# the kernel that rotates in its own prologue and never touch the array; such a case would prove nothing here.)
@pytest.mark.parametrize("p,n,N,K,B,dtype", [
    (2, 256, 64, 2048, 3, torch.float32),
    (2, 256, 48, 8192, 2, torch.bfloat16),    # K split over blocks: fp32 staging in the scratch array as well
    (2, 64, 32, 4096, 16, torch.float32),
])
def test_matches_higgs_linear_on_two_calls_in_a_row(p, n, N, K, B, dtype):
    d, g64, gt, packed, scales, canon = make_layer(p, n, N, K, xi=77, seed=900 + N)
    assert hb.higgs_linear_launch_count(d, B, hb.HIGGS_BF16 if dtype == torch.bfloat16 else hb.HIGGS_F32) > 1
    x1 = U.bf16_tensor(inputs.make_activations(B, K, seed=1))
    x2 = U.bf16_tensor(inputs.make_activations(B, K, seed=2))
    ref1 = hb.higgs_linear(d, x1, packed, scales, gt, out_dtype=dtype).float().cpu().numpy()
    ref2 = hb.higgs_linear(d, x2, packed, scales, gt, out_dtype=dtype).float().cpu().numpy()
    y1 = torch.full((B, N), float("nan"), dtype=dtype, device=U.dev())
    y2 = torch.full((B, N), float("nan"), dtype=dtype, device=U.dev())
    hb.higgs_linear_static(d, x1, packed, scales, gt, y1)     # first call on this device also looks the array up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    hb.higgs_linear_static(d, x1, packed, scales, gt, y1)
    hb.higgs_linear_static(d, x2, packed, scales, gt, y2)     # reuses the array with the previous call's contents
    assert hb.higgs_device_status() == hb.HIGGS_OK
    assert torch.cuda.mem_get_info()[0] == free_before, "the workspace-free call changed the device's free memory"
    tol = Y_TOL + (2.0 ** -8 if dtype == torch.bfloat16 else 0.0)
    # the oracle on the device's own codes and stored scales ("given identical codes")
    codes = canon.cpu().numpy().astype(np.int64)
    sc = hb.scales_from_tile_major(scales, N).float().cpu().numpy().astype(np.float64)
    for y, ref, x in ((y1, ref1, x1), (y2, ref2, x2)):
        got = y.float().cpu().numpy()
        assert np.all(np.isfinite(got))
        assert np.max(np.abs(got - ref)) <= tol * np.max(np.abs(ref))
        y_or = oracle.linear_dense(x.float().cpu().numpy().astype(np.float64), codes, sc, 1024, g64, 77)
        assert U.linear_error(got, y_or) <= tol


def test_refuses_what_does_not_fit_and_reports_capacity():
    cap = hb.higgs_linear_static_capacity()
    assert cap == 4 << 20
    big = hb.make_desc(2, 256, 28672, 8192, 1)
    assert hb.higgs_workspace_bytes(big, hb.HIGGS_OP_LINEAR, 16) <= cap          # the largest configured layer fits
    assert hb.higgs_workspace_bytes(big, hb.HIGGS_OP_LINEAR, 64) > cap
    a = ctypes.c_void_p(0x1000)                                                  # never dereferenced: refused first
    rc = binding.lib.higgs_linear_static(ctypes.byref(big), a, 64, a, a, a, a, hb.HIGGS_F32, None)
    assert rc == hb.HIGGS_ERR_STATIC_SCRATCH
    assert "scratch" in hb.status_string(rc)
    bad = hb.make_desc(2, 100, 64, 1024, 1)
    assert binding.lib.higgs_linear_static(ctypes.byref(bad), a, 1, a, a, a, a, hb.HIGGS_F32, None) == hb.HIGGS_ERR_UNSUPPORTED
