"""Helpers for the GPU parity tests: moving seeded host arrays to the device and calling the C ABI binding."""
import numpy as np
import torch

import oracle
import paper_2411_17525_b200 as hb
from synth import grids as make_grids


def dev():
    return torch.device("cuda:0")


def bf16_tensor(a32: np.ndarray) -> torch.Tensor:
    """fp32 array of bf16-representable values -> cuda bf16 tensor with identical values."""
    t = torch.from_numpy(np.ascontiguousarray(a32, dtype=np.float32)).to(dev())
    b = t.to(torch.bfloat16)
    assert torch.equal(b.float(), t)
    return b.contiguous()


def f32_tensor(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dev())


def grid32(p, n):
    """Stored oracle-fitted grid: (float64 array with fp32-exact values, cuda fp32 tensor)."""
    g = make_grids.load(p, n)
    t = f32_tensor(g)
    assert np.array_equal(t.cpu().numpy().astype(np.float64), g)
    return g, t


def oracle_encode(W, g, grid, xi):
    """Oracle codes plus the stored (fp16-rounded) scales widened to float64."""
    q = oracle.quantize(np.asarray(W, dtype=np.float64), g, grid, xi)
    sc16 = oracle.round_scales_fp16(q.scales)
    return q, sc16


def compare_codes(gpu_codes: np.ndarray, q, max_margin=1e-5, max_frac=1e-4):
    """Bit-exact except near-ties: every mismatch must be the oracle's runner-up at margin < max_margin."""
    mism = gpu_codes.astype(np.int64) != q.codes
    cnt = int(mism.sum())
    if cnt:
        assert np.all(gpu_codes[mism] == q.runner[mism]), "a mismatching GPU code is not the oracle's runner-up"
        assert float(q.margin[mism].max()) < max_margin, f"mismatch at margin {q.margin[mism].max()}"
    assert cnt <= max_frac * gpu_codes.size, f"{cnt} mismatches of {gpu_codes.size}"
    return cnt


def linear_error(y_gpu: np.ndarray, y_ref: np.ndarray) -> float:
    """max |y - y_ref| / max |y_ref| over the whole call (the layer-level relative error)."""
    return float(np.max(np.abs(y_gpu.astype(np.float64) - y_ref)) / np.max(np.abs(y_ref)))


def linear_error_rms(y_gpu: np.ndarray, y_ref: np.ndarray) -> float:
    """max |y - y_ref| / rms(y_ref): the same deviation against the typical output size instead of the largest."""
    return float(np.max(np.abs(y_gpu.astype(np.float64) - y_ref)) / np.sqrt(np.mean(np.square(y_ref))))
