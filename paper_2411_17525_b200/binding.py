"""Thin ctypes binding of the C ABI declared in include/higgs.h.

Argument marshalling only: every step of the path runs in the CUDA library.
torch is used for device memory and streams.  There is no CPU fallback: if the
shared library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libhiggs_b200.so")

HIGGS_OK, HIGGS_ERR_INVALID_ARG, HIGGS_ERR_UNSUPPORTED, HIGGS_ERR_WORKSPACE, HIGGS_ERR_CUDA, HIGGS_ERR_TIMEOUT, HIGGS_ERR_STATIC_SCRATCH = range(7)
HIGGS_F32, HIGGS_F16, HIGGS_BF16 = 0, 1, 2
HIGGS_OP_QUANTIZE, HIGGS_OP_LINEAR, HIGGS_OP_MAKE_GRID, HIGGS_OP_MAKE_GRID_SEEDED = 0, 1, 2, 3
HIGGS_LAYOUT_VERSION = 1

EXPORTS = [
    "higgs_status_string", "higgs_sign", "higgs_packed_bytes", "higgs_scales_bytes", "higgs_canonical_bytes",
    "higgs_workspace_bytes", "higgs_make_grid", "higgs_quantize", "higgs_linear", "higgs_rht",
    "higgs_encoder_table_bytes", "higgs_make_encoder_table", "higgs_quantize_prepared",
    "higgs_pack_codes", "higgs_unpack_codes", "higgs_rotate_activations", "higgs_linear_prerotated",
    "higgs_linear_host", "higgs_linear_host_workspace_bytes", "higgs_linear_launch_count", "higgs_device_status",
    "higgs_linear_static", "higgs_linear_static_capacity", "higgs_linear_k_splits", "higgs_rotated_bytes",
    "higgs_rotated_layout", "higgs_dequantize", "higgs_make_uniform_grid", "higgs_layer_error",
    "higgs_allocate_bits", "higgs_general_tuples", "higgs_quantize_general", "higgs_linear_host_batch",
    "higgs_linear_gather", "higgs_linear_share", "higgs_make_grid_seeded", "higgs_gaussian_samples", "higgs_shard_rows",
    "higgs_launch_floor", "higgs_selftest_wait", "higgs_linear_uses_atomics", "higgs_shard_seed", "higgs_linear_kshard", "higgs_reduce_slots", "higgs_linear_multi", "higgs_linear_multi_workspace_bytes",
    "higgs_linear_multi_launch_count", "higgs_linear_host_block", "higgs_linear_host_block_workspace_bytes",
]


class higgs_desc(ctypes.Structure):
    _fields_ = [
        ("p", ctypes.c_int32), ("n", ctypes.c_int32), ("g", ctypes.c_int32), ("scale_dtype", ctypes.c_int32),
        ("rht_seed", ctypes.c_uint64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
        ("layout_version", ctypes.c_int32), ("reserved", ctypes.c_int32),
    ]


class HiggsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2411_17525_b200.build` "
            "(there is no CPU or PyTorch fallback for the HIGGS kernels)")
    lib = ctypes.CDLL(LIB_PATH)
    P, vp, sz, i64, i32, u64 = ctypes.POINTER(higgs_desc), ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int64, ctypes.c_int, ctypes.c_uint64
    lib.higgs_status_string.restype = ctypes.c_char_p
    lib.higgs_status_string.argtypes = [i32]
    lib.higgs_sign.restype = i32
    lib.higgs_sign.argtypes = [u64, i64]
    for f in ("higgs_packed_bytes", "higgs_scales_bytes", "higgs_canonical_bytes"):
        getattr(lib, f).restype = sz
        getattr(lib, f).argtypes = [P]
    lib.higgs_workspace_bytes.restype = sz
    lib.higgs_workspace_bytes.argtypes = [P, i32, i64]
    lib.higgs_make_grid.restype = i32
    lib.higgs_make_grid.argtypes = [i32, i32, vp, i64, i32, vp, vp, vp, vp, sz, vp]
    lib.higgs_quantize.restype = i32
    lib.higgs_quantize.argtypes = [P, vp, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.higgs_encoder_table_bytes.restype = sz
    lib.higgs_encoder_table_bytes.argtypes = [i32, i32]
    lib.higgs_make_encoder_table.restype = i32
    lib.higgs_make_encoder_table.argtypes = [i32, i32, vp, vp, vp]
    lib.higgs_quantize_prepared.restype = i32
    lib.higgs_quantize_prepared.argtypes = [P, vp, i32, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.higgs_linear.restype = i32
    lib.higgs_linear.argtypes = [P, vp, i64, vp, vp, vp, vp, i32, vp, sz, vp]
    lib.higgs_rotate_activations.restype = i32
    lib.higgs_rotate_activations.argtypes = [P, vp, i64, vp, vp]
    lib.higgs_linear_prerotated.restype = i32
    lib.higgs_linear_prerotated.argtypes = [P, vp, i64, vp, vp, vp, vp, i32, vp, sz, vp]
    lib.higgs_linear_host.restype = i32
    lib.higgs_linear_host.argtypes = [P, vp, i64, vp, vp, vp, vp, i32, vp, sz, vp]
    lib.higgs_linear_share.restype = i32
    lib.higgs_linear_share.argtypes = [P, vp, i64, vp, vp, vp, vp, i32, vp, vp, sz, vp]
    lib.higgs_linear_gather.restype = i32
    lib.higgs_linear_gather.argtypes = [P, vp, i64, vp, vp, vp, vp, i32, i64, i64, i32, vp, sz, vp]
    lib.higgs_linear_host_batch.restype = i32
    lib.higgs_linear_host_batch.argtypes = [i32, vp, vp, i64, vp, vp, vp, vp, i32, vp, vp, vp]
    lib.higgs_linear_host_workspace_bytes.restype = sz
    lib.higgs_linear_host_workspace_bytes.argtypes = [P, i64, i32]
    lib.higgs_rotated_bytes.restype = sz
    lib.higgs_rotated_bytes.argtypes = [P, i64]
    lib.higgs_rotated_layout.restype = i32
    lib.higgs_rotated_layout.argtypes = [P, i64]
    lib.higgs_linear_k_splits.restype = i32
    lib.higgs_linear_k_splits.argtypes = [P, i64]
    lib.higgs_linear_uses_atomics.restype = i32
    lib.higgs_linear_uses_atomics.argtypes = [P, i64]
    lib.higgs_linear_launch_count.restype = i32
    lib.higgs_linear_launch_count.argtypes = [P, i64, i32]
    lib.higgs_linear_static.restype = i32
    lib.higgs_linear_static.argtypes = [P, vp, i64, vp, vp, vp, vp, i32, vp]
    lib.higgs_linear_static_capacity.restype = sz
    lib.higgs_linear_static_capacity.argtypes = []
    lib.higgs_device_status.restype = i32
    lib.higgs_device_status.argtypes = [vp, i32]
    lib.higgs_rht.restype = i32
    lib.higgs_rht.argtypes = [P, vp, i32, i64, vp, i32, vp]
    lib.higgs_pack_codes.restype = i32
    lib.higgs_pack_codes.argtypes = [P, vp, vp, vp]
    lib.higgs_unpack_codes.restype = i32
    lib.higgs_unpack_codes.argtypes = [P, vp, vp, vp]
    lib.higgs_make_uniform_grid.restype = i32
    lib.higgs_make_uniform_grid.argtypes = [i32, vp, vp, vp, vp]
    lib.higgs_layer_error.restype = i32
    lib.higgs_layer_error.argtypes = [P, vp, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.higgs_allocate_bits.restype = i32
    lib.higgs_allocate_bits.argtypes = [i32, i32, vp, vp, vp, vp, i64, vp, vp]
    lib.higgs_general_tuples.restype = i32
    lib.higgs_general_tuples.argtypes = [i32]
    lib.higgs_quantize_general.restype = i32
    lib.higgs_quantize_general.argtypes = [i32, i32, i64, i64, u64, vp, i32, vp, vp, vp, vp, vp]
    lib.higgs_dequantize.restype = i32
    lib.higgs_dequantize.argtypes = [P, vp, vp, vp, vp, i32, vp, sz, vp]
    lib.higgs_make_grid_seeded.restype = i32
    lib.higgs_make_grid_seeded.argtypes = [i32, i32, u64, i32, i32, vp, vp, vp, vp, sz, vp]
    lib.higgs_gaussian_samples.restype = i32
    lib.higgs_gaussian_samples.argtypes = [i32, u64, i64, vp, vp]
    lib.higgs_shard_rows.restype = i32
    lib.higgs_shard_rows.argtypes = [i64, i32, i32, i32, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.higgs_linear_multi.restype = i32
    lib.higgs_linear_multi.argtypes = [i32, vp, vp, i64, vp, vp, vp, vp, i32, vp, sz, vp]
    lib.higgs_linear_multi_workspace_bytes.restype = sz
    lib.higgs_linear_multi_workspace_bytes.argtypes = [i32, vp, i64]
    lib.higgs_linear_multi_launch_count.restype = i32
    lib.higgs_linear_multi_launch_count.argtypes = [i32, vp, i64, i32]
    lib.higgs_linear_host_block.restype = i32
    lib.higgs_linear_host_block.argtypes = [i32, vp, vp, sz, vp, i64, vp, vp, vp, vp, sz, vp, i32, vp, sz, vp]
    lib.higgs_linear_host_block_workspace_bytes.restype = sz
    lib.higgs_linear_host_block_workspace_bytes.argtypes = [i32, vp, i64, sz, sz]
    lib.higgs_shard_seed.restype = u64
    lib.higgs_shard_seed.argtypes = [u64, i64]
    lib.higgs_linear_kshard.restype = i32
    lib.higgs_linear_kshard.argtypes = [P, vp, i64, vp, vp, vp, vp, i32, i32, vp, sz, vp]
    lib.higgs_reduce_slots.restype = i32
    lib.higgs_reduce_slots.argtypes = [vp, i32, i64, vp, i32, vp]
    lib.higgs_launch_floor.restype = i32
    lib.higgs_launch_floor.argtypes = [i32, i32, sz, vp]
    lib.higgs_selftest_wait.restype = i32
    lib.higgs_selftest_wait.argtypes = [i32, ctypes.c_uint32, vp, vp]
    return lib


lib = _load()


def make_desc(p: int, n: int, N: int, K: int, rht_seed: int, g: int = 1024) -> higgs_desc:
    return higgs_desc(p, n, g, HIGGS_F16, rht_seed & (2**64 - 1), N, K, HIGGS_LAYOUT_VERSION, 0)


def status_string(status: int) -> str:
    return lib.higgs_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != HIGGS_OK:
        raise HiggsError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    return {torch.float32: HIGGS_F32, torch.float16: HIGGS_F16, torch.bfloat16: HIGGS_BF16}[t.dtype]


def higgs_sign(rht_seed: int, j: int) -> int:
    return int(lib.higgs_sign(ctypes.c_uint64(rht_seed & (2**64 - 1)), int(j)))


def higgs_packed_bytes(desc: higgs_desc) -> int:
    return int(lib.higgs_packed_bytes(ctypes.byref(desc)))


def higgs_scales_bytes(desc: higgs_desc) -> int:
    return int(lib.higgs_scales_bytes(ctypes.byref(desc)))


def higgs_canonical_bytes(desc: higgs_desc) -> int:
    return int(lib.higgs_canonical_bytes(ctypes.byref(desc)))


def higgs_workspace_bytes(desc: higgs_desc, op: int, B: int = 0) -> int:
    return int(lib.higgs_workspace_bytes(ctypes.byref(desc), int(op), int(B)))


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def higgs_make_grid(p: int, n: int, samples: torch.Tensor, max_iters: int = 4000, workspace: Optional[torch.Tensor] = None):
    """samples: cuda fp32 [m][p].  Returns (grid [n][p] fp32, mse fp32 scalar tensor, iters int32 scalar tensor)."""
    assert samples.is_cuda and samples.dtype == torch.float32 and samples.is_contiguous()
    m = samples.numel() // p
    d = higgs_desc(p, n, 0, HIGGS_F16, 0, 0, m, HIGGS_LAYOUT_VERSION, 0)
    if workspace is None:
        workspace = _workspace(higgs_workspace_bytes(d, HIGGS_OP_MAKE_GRID), samples.device)
    grid = torch.empty((n, p), dtype=torch.float32, device=samples.device)
    mse = torch.empty((), dtype=torch.float32, device=samples.device)
    iters = torch.empty((), dtype=torch.int32, device=samples.device)
    _check(lib.higgs_make_grid(p, n, _ptr(samples), m, int(max_iters), _ptr(grid), _ptr(mse), _ptr(iters),
                               _ptr(workspace), workspace.numel(), _stream()), "higgs_make_grid")
    return grid, mse, iters


def higgs_make_grid_seeded(p: int, n: int, sample_seed: int, log2_samples: int = 18, max_iters: int = 4000, device=None):
    """Grid fit on samples the library draws from the seed.  Returns (grid, mse, iters) like higgs_make_grid."""
    device = device or torch.device("cuda")
    d = higgs_desc(p, n, 0, HIGGS_F16, 0, 0, 1 << log2_samples, HIGGS_LAYOUT_VERSION, 0)
    workspace = _workspace(higgs_workspace_bytes(d, HIGGS_OP_MAKE_GRID_SEEDED), device)
    grid = torch.empty((n, p), dtype=torch.float32, device=device)
    mse = torch.empty((), dtype=torch.float32, device=device)
    iters = torch.empty((), dtype=torch.int32, device=device)
    _check(lib.higgs_make_grid_seeded(p, n, sample_seed & (2**64 - 1), log2_samples, int(max_iters), _ptr(grid), _ptr(mse),
                                      _ptr(iters), _ptr(workspace), workspace.numel(), _stream()), "higgs_make_grid_seeded")
    return grid, mse, iters


def higgs_gaussian_samples(p: int, sample_seed: int, num_samples: int, device=None) -> torch.Tensor:
    device = device or torch.device("cuda")
    out = torch.empty((num_samples, p), dtype=torch.float32, device=device)
    _check(lib.higgs_gaussian_samples(p, sample_seed & (2**64 - 1), num_samples, _ptr(out), _stream()), "higgs_gaussian_samples")
    return out


def higgs_launch_floor(blocks: int, threads: int, shared_bytes: int) -> None:
    _check(lib.higgs_launch_floor(blocks, threads, shared_bytes, _stream()), "higgs_launch_floor")


def higgs_selftest_wait(which: int, polls: int, device=None) -> torch.Tensor:
    """Runs the bounded-wait self-check; returns the device int32[2] result (0 = that wait ran out)."""
    device = device or torch.device("cuda")
    out = torch.full((2,), -1, dtype=torch.int32, device=device)
    _check(lib.higgs_selftest_wait(which, polls, _ptr(out), _stream()), "higgs_selftest_wait")
    return out


def higgs_make_encoder_table(p: int, n: int, grid: torch.Tensor) -> torch.Tensor:
    """The encoder's search table for a grid (cuda [n][p] fp32), to be passed to higgs_quantize(..., table=...) for
    every layer that uses this grid."""
    assert grid.is_cuda and grid.dtype == torch.float32 and grid.is_contiguous() and tuple(grid.shape) == (n, p)
    size = lib.higgs_encoder_table_bytes(p, n)
    if size == 0:
        raise HiggsError(HIGGS_ERR_UNSUPPORTED, "higgs_encoder_table_bytes")
    table = torch.empty(size, dtype=torch.uint8, device=grid.device)
    _check(lib.higgs_make_encoder_table(p, n, _ptr(grid), _ptr(table), _stream()), "higgs_make_encoder_table")
    return table


def higgs_quantize(desc: higgs_desc, W: torch.Tensor, grid: torch.Tensor, want_canonical: bool = False,
                   workspace: Optional[torch.Tensor] = None, out=None, table: Optional[torch.Tensor] = None):
    """W: cuda [N][K] fp32 or bf16; grid: cuda [n][p] fp32.  Returns (packed u8, scales fp16 tile-major [N/16][K/g][16], canonical u8 or None).
    out = (packed, scales) reuses existing output tensors; table = higgs_make_encoder_table(p, n, grid) skips building
    the search table in this call."""
    assert W.is_cuda and W.is_contiguous() and grid.is_cuda and grid.dtype == torch.float32 and grid.is_contiguous()
    dev = W.device
    if out is not None:
        packed, scales = out
        assert packed.is_cuda and packed.dtype == torch.uint8 and packed.numel() >= higgs_packed_bytes(desc)
        assert scales.is_cuda and scales.dtype == torch.float16 and scales.numel() * 2 >= higgs_scales_bytes(desc)
    else:
        packed = torch.empty(max(higgs_packed_bytes(desc), 16), dtype=torch.uint8, device=dev)
        scales = torch.empty((desc.N // 16, max(desc.K // desc.g, 0), 16), dtype=torch.float16, device=dev)
    canonical = torch.empty((desc.N, desc.K // desc.p), dtype=torch.uint8, device=dev) if want_canonical else None
    if workspace is None:
        workspace = _workspace(higgs_workspace_bytes(desc, HIGGS_OP_QUANTIZE), dev)
    elif workspace is False:          # lend none (allowed with want_canonical): the library then packs in a second kernel
        assert want_canonical
        workspace = torch.empty(0, dtype=torch.uint8, device=dev)
    if table is not None:
        assert table.is_cuda and table.dtype == torch.uint8 and table.numel() >= lib.higgs_encoder_table_bytes(desc.p, desc.n)
        _check(lib.higgs_quantize_prepared(ctypes.byref(desc), _ptr(W), _dtype_code(W), _ptr(grid), _ptr(table), _ptr(packed),
                                           _ptr(scales), _ptr(canonical), _ptr(workspace), workspace.numel(), _stream()),
               "higgs_quantize_prepared")
    else:
        _check(lib.higgs_quantize(ctypes.byref(desc), _ptr(W), _dtype_code(W), _ptr(grid), _ptr(packed), _ptr(scales),
                                  _ptr(canonical), _ptr(workspace), workspace.numel(), _stream()), "higgs_quantize")
    return packed, scales, canonical


def higgs_linear(desc: higgs_desc, x: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor, grid: torch.Tensor,
                 out_dtype: torch.dtype = torch.float32, workspace: Optional[torch.Tensor] = None,
                 y: Optional[torch.Tensor] = None) -> torch.Tensor:
    """x: cuda [B][K] bf16.  Returns y [B][N] of out_dtype (fp32 or bf16)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    B = x.shape[0]
    if y is None:
        y = torch.empty((B, desc.N), dtype=out_dtype, device=x.device)
    if workspace is None:
        workspace = _workspace(higgs_workspace_bytes(desc, HIGGS_OP_LINEAR, B), x.device)
    _check(lib.higgs_linear(ctypes.byref(desc), _ptr(x), B, _ptr(packed), _ptr(scales), _ptr(grid), _ptr(y),
                            _dtype_code(y), _ptr(workspace), workspace.numel(), _stream()), "higgs_linear")
    return y


def higgs_linear_share(desc: higgs_desc, x: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor, grid: torch.Tensor,
                       xdag_out: Optional[torch.Tensor] = None, out_dtype: torch.dtype = torch.float32,
                       workspace: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None):
    """higgs_linear that also leaves the rotated activations in xdag_out for the other layers reading the same x
    (pass it to higgs_linear_prerotated).  Returns (y, xdag_out)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    B = x.shape[0]
    if y is None:
        y = torch.empty((B, desc.N), dtype=out_dtype, device=x.device)
    if xdag_out is None:
        nb = higgs_rotated_bytes(desc, B)
        xdag_out = torch.empty(x.shape if nb == x.numel() * 2 else (nb // 2,), dtype=torch.float16, device=x.device)
    if workspace is None:
        workspace = _workspace(higgs_workspace_bytes(desc, HIGGS_OP_LINEAR, B), x.device)
    _check(lib.higgs_linear_share(ctypes.byref(desc), _ptr(x), B, _ptr(packed), _ptr(scales), _ptr(grid), _ptr(y),
                                  _dtype_code(y), _ptr(xdag_out), _ptr(workspace), workspace.numel(), _stream()),
           "higgs_linear_share")
    return y, xdag_out


def higgs_rotate_activations(desc: higgs_desc, x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """x: cuda [B][K] bf16 -> rotated activations, cuda fp16 (higgs_rotated_bytes(desc, B) bytes; row-major [B][K]
    when higgs_rotated_layout(desc, B) == 0)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    if out is None:
        nb = higgs_rotated_bytes(desc, x.shape[0])
        out = torch.empty(x.shape if nb == x.numel() * 2 else (nb // 2,), dtype=torch.float16, device=x.device)
    _check(lib.higgs_rotate_activations(ctypes.byref(desc), _ptr(x), x.shape[0], _ptr(out), _stream()),
           "higgs_rotate_activations")
    return out


def higgs_linear_prerotated(desc: higgs_desc, xdag: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor,
                            grid: torch.Tensor, out_dtype: torch.dtype = torch.float32,
                            workspace: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None,
                            B: Optional[int] = None) -> torch.Tensor:
    """xdag: cuda fp16 from higgs_rotate_activations for the same batch B (pass B when xdag is not [B][K]).
    Returns y [B][N]."""
    assert xdag.is_cuda and xdag.dtype == torch.float16 and xdag.is_contiguous()
    B = xdag.shape[0] if B is None else B
    if y is None:
        y = torch.empty((B, desc.N), dtype=out_dtype, device=xdag.device)
    if workspace is None:
        workspace = _workspace(higgs_workspace_bytes(desc, HIGGS_OP_LINEAR, B), xdag.device)
    _check(lib.higgs_linear_prerotated(ctypes.byref(desc), _ptr(xdag), B, _ptr(packed), _ptr(scales), _ptr(grid),
                                       _ptr(y), _dtype_code(y), _ptr(workspace), workspace.numel(), _stream()),
           "higgs_linear_prerotated")
    return y


def higgs_linear_host_workspace_bytes(desc: higgs_desc, B: int, y_dtype: int = HIGGS_F32) -> int:
    return int(lib.higgs_linear_host_workspace_bytes(ctypes.byref(desc), int(B), int(y_dtype)))


def higgs_linear_host(desc: higgs_desc, x_host: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor,
                      grid: torch.Tensor, y_host: torch.Tensor, workspace: torch.Tensor) -> torch.Tensor:
    """x_host: CPU (pinned) [B][K] bf16; y_host: CPU (pinned) [B][N] fp32/bf16; workspace: cuda uint8.
    Enqueues copy-in, the layer and copy-out on the current stream; synchronise before reading y_host."""
    assert (not x_host.is_cuda) and x_host.dtype == torch.bfloat16 and x_host.is_contiguous()
    assert (not y_host.is_cuda) and y_host.is_contiguous() and workspace.is_cuda
    B = x_host.shape[0]
    _check(lib.higgs_linear_host(ctypes.byref(desc), _ptr(x_host), B, _ptr(packed), _ptr(scales), _ptr(grid),
                                 _ptr(y_host), _dtype_code(y_host), _ptr(workspace), workspace.numel(), _stream()),
           "higgs_linear_host")
    return y_host


def shard_rows(N: int, world: int, rank: int, multiple: int = 128):
    """Rows [begin, end) of an N-row layer that rank `rank` of `world` holds (higgs_shard_rows: contiguous ranges of whole
    units of `multiple` rows, the remainder spread over the first ranks)."""
    begin, count = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(lib.higgs_shard_rows(int(N), int(world), int(rank), int(multiple), ctypes.byref(begin), ctypes.byref(count)),
           "higgs_shard_rows")
    return begin.value, begin.value + count.value


def higgs_linear_gather(desc: higgs_desc, x: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor, grid: torch.Tensor,
                        y_dsts, row_offset: int, workspace: Optional[torch.Tensor] = None) -> None:
    """Row-sharded layer: this device's shard (desc, packed, scales) times x, written into columns
    [row_offset, row_offset + desc.N) of every tensor of y_dsts ([B][ld] each; this device's own first, then
    peer-mapped tensors of the other devices).  The caller orders the ranks (see include/higgs.h)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    B = x.shape[0]
    ld = y_dsts[0].shape[1]
    for t in y_dsts:
        assert t.is_contiguous() and t.dtype == y_dsts[0].dtype and tuple(t.shape) == (B, ld)
    if workspace is None:
        workspace = _workspace(higgs_workspace_bytes(desc, HIGGS_OP_LINEAR, B), x.device)
    ptrs = (ctypes.c_void_p * len(y_dsts))(*[t.data_ptr() for t in y_dsts])
    _check(lib.higgs_linear_gather(ctypes.byref(desc), _ptr(x), B, _ptr(packed), _ptr(scales), _ptr(grid), ptrs, len(y_dsts),
                                   ld, int(row_offset), _dtype_code(y_dsts[0]), _ptr(workspace), workspace.numel(), _stream()),
           "higgs_linear_gather")


class HostBlock:
    """Argument arrays of higgs_linear_host_block, marshalled once: the layers of one step with ONE pinned input block and
    ONE pinned output block.  inputs: list of (key, x) with x a [B][K] bf16 host tensor per distinct input; layer i reads
    the input named x_keys[i].  After the call and a stream synchronisation, self.y[i] is layer i's [B][N_i] output (a view
    of the output block)."""

    def __init__(self, descs, x_keys, inputs, packed, scales, grids, B, y_dtype=torch.float32, device=None):
        n = len(descs)
        assert n == len(x_keys) == len(packed) == len(scales) == len(grids)
        device = device or packed[0].device
        self.count, self.B = n, int(B)
        off, pos = {}, 0
        for key, x in inputs:
            assert (not x.is_cuda) and x.dtype == torch.bfloat16 and x.is_contiguous() and x.shape[0] == B
            off[key] = pos
            pos += (x.numel() * 2 + 255) // 256 * 256
        self.x_block = torch.empty(max(pos, 256), dtype=torch.uint8).pin_memory()
        self.x_views = {}
        for key, x in inputs:
            v = self.x_block[off[key]: off[key] + x.numel() * 2].view(torch.bfloat16).view(x.shape)
            v.copy_(x)
            self.x_views[key] = v
        esz = 4 if y_dtype == torch.float32 else 2
        y_off, pos = [], 0
        for d in descs:
            y_off.append(pos)
            pos += (B * d.N * esz + 255) // 256 * 256
        self.y_block = torch.empty(max(pos, 256), dtype=torch.uint8).pin_memory()
        self.y = [self.y_block[o: o + B * d.N * esz].view(y_dtype).view(B, d.N) for o, d in zip(y_off, descs)]
        self.keep = (list(descs), list(packed), list(scales), list(grids))
        arr = ctypes.c_void_p * n
        szs = ctypes.c_size_t * n
        self.descs = arr(*[ctypes.addressof(d) for d in descs])
        self.x_offsets = szs(*[off[k] for k in x_keys])
        self.y_offsets = szs(*y_off)
        self.packed = arr(*[t.data_ptr() for t in packed])
        self.scales = arr(*[t.data_ptr() for t in scales])
        self.grids = arr(*[t.data_ptr() for t in grids])
        self.y_dtype = HIGGS_F32 if y_dtype == torch.float32 else HIGGS_BF16
        need = int(lib.higgs_linear_host_block_workspace_bytes(n, self.descs, self.B, self.x_block.numel(), self.y_block.numel()))
        self.workspace = _workspace(need, device)

    def set_weights(self, packed, scales):
        self.keep = (self.keep[0], list(packed), list(scales), self.keep[3])
        for i, (p, s) in enumerate(zip(packed, scales)):
            self.packed[i] = p.data_ptr()
            self.scales[i] = s.data_ptr()


def higgs_linear_host_block(hbk: HostBlock) -> None:
    """One host-to-device copy, the step's products, one device-to-host copy, enqueued with one library call."""
    _check(lib.higgs_linear_host_block(hbk.count, hbk.descs, hbk.x_block.data_ptr(), hbk.x_block.numel(), hbk.x_offsets, hbk.B,
                                       hbk.packed, hbk.scales, hbk.grids, hbk.y_block.data_ptr(), hbk.y_block.numel(),
                                       hbk.y_offsets, hbk.y_dtype, _ptr(hbk.workspace), hbk.workspace.numel(), _stream()),
           "higgs_linear_host_block")


class MultiLinear:
    """Argument arrays of higgs_linear_multi, marshalled once: several matrices (same K, grid and seed) that read the
    same activations and run as one product over their concatenated rows."""

    def __init__(self, descs, packed, scales, grid, ys, B, workspace=None):
        n = len(descs)
        assert n == len(packed) == len(scales) == len(ys)
        self.keep = (list(descs), list(packed), list(scales), grid, list(ys))
        self.count, self.B, self.grid = n, int(B), grid
        arr = ctypes.c_void_p * n
        self.descs = arr(*[ctypes.addressof(d) for d in descs])
        self.packed = arr(*[t.data_ptr() for t in packed])
        self.scales = arr(*[t.data_ptr() for t in scales])
        self.ys = arr(*[t.data_ptr() for t in ys])
        self.y_dtype = _dtype_code(ys[0])
        need = int(lib.higgs_linear_multi_workspace_bytes(n, self.descs, self.B))
        self.workspace = workspace if workspace is not None else _workspace(need, ys[0].device)
        assert self.workspace.numel() >= need
        self.launches = int(lib.higgs_linear_multi_launch_count(n, self.descs, self.B, self.y_dtype))

    def set_weights(self, packed, scales):
        self.keep = (self.keep[0], list(packed), list(scales)) + self.keep[3:]
        for i, (p, s) in enumerate(zip(packed, scales)):
            self.packed[i] = p.data_ptr()
            self.scales[i] = s.data_ptr()


def higgs_linear_multi(m: MultiLinear, x: torch.Tensor) -> None:
    """Enqueues the product of every matrix of `m` with x ([B][K] bf16) on the current stream; outputs land in m's ys."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.shape[0] == m.B
    _check(lib.higgs_linear_multi(m.count, m.descs, _ptr(x), m.B, m.packed, m.scales, _ptr(m.grid), m.ys, m.y_dtype,
                                  _ptr(m.workspace), m.workspace.numel(), _stream()), "higgs_linear_multi")


def higgs_shard_seed(rht_seed: int, k_offset: int) -> int:
    return int(lib.higgs_shard_seed(rht_seed & (2**64 - 1), int(k_offset)))


def higgs_linear_kshard(desc: higgs_desc, x_shard: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor, grid: torch.Tensor,
                        slot_bufs, rank: int, workspace: Optional[torch.Tensor] = None) -> None:
    """K-sharded layer: this device's fp32 partial product into slot `rank` of every tensor of slot_bufs
    ([world][B][N] fp32 each, slot_bufs[i] on device i or peer-mapped)."""
    assert x_shard.is_cuda and x_shard.dtype == torch.bfloat16 and x_shard.is_contiguous()
    B, world = x_shard.shape[0], len(slot_bufs)
    for t in slot_bufs:
        assert t.is_contiguous() and t.dtype == torch.float32 and tuple(t.shape) == (world, B, desc.N)
    if workspace is None:
        workspace = _workspace(higgs_workspace_bytes(desc, HIGGS_OP_LINEAR, B), x_shard.device)
    ptrs = (ctypes.c_void_p * world)(*[t.data_ptr() for t in slot_bufs])
    _check(lib.higgs_linear_kshard(ctypes.byref(desc), _ptr(x_shard), B, _ptr(packed), _ptr(scales), _ptr(grid), ptrs, world,
                                   int(rank), _ptr(workspace), workspace.numel(), _stream()), "higgs_linear_kshard")


def higgs_reduce_slots(slots: torch.Tensor, out_dtype: torch.dtype = torch.float32) -> torch.Tensor:
    """slots: cuda fp32 [world][B][N] -> y [B][N] = the slots summed in slot order."""
    assert slots.is_cuda and slots.dtype == torch.float32 and slots.is_contiguous() and slots.dim() == 3
    world, B, N = slots.shape
    y = torch.empty((B, N), dtype=out_dtype, device=slots.device)
    _check(lib.higgs_reduce_slots(_ptr(slots), world, B * N, _ptr(y), _dtype_code(y), _stream()), "higgs_reduce_slots")
    return y


class HostBatch:
    """Argument arrays of higgs_linear_host_batch, marshalled once: `count` layers of one step.  x_hosts may name the
    same pinned tensor for layers that read the same activations (they then share one host-to-device copy)."""

    def __init__(self, descs, x_hosts, packed, scales, grids, y_hosts, workspaces):
        n = len(descs)
        assert all(len(a) == n for a in (x_hosts, packed, scales, grids, y_hosts, workspaces))
        for x, y, w in zip(x_hosts, y_hosts, workspaces):
            assert (not x.is_cuda) and x.dtype == torch.bfloat16 and x.is_contiguous()
            assert (not y.is_cuda) and y.is_contiguous() and y.dtype == y_hosts[0].dtype and w.is_cuda
        self.keep = (list(descs), list(x_hosts), list(packed), list(scales), list(grids), list(y_hosts), list(workspaces))
        self.count = n
        self.B = int(x_hosts[0].shape[0]) if n else 0
        self.y_dtype = _dtype_code(y_hosts[0]) if n else HIGGS_F32
        arr = ctypes.c_void_p * max(n, 1)
        self.descs = arr(*[ctypes.addressof(d) for d in descs])
        self.x = arr(*[t.data_ptr() for t in x_hosts])
        self.y = arr(*[t.data_ptr() for t in y_hosts])
        self.ws = arr(*[t.data_ptr() for t in workspaces])
        self.ws_bytes = (ctypes.c_size_t * max(n, 1))(*[t.numel() for t in workspaces])
        self.packed = arr(*[t.data_ptr() for t in packed])
        self.scales = arr(*[t.data_ptr() for t in scales])
        self.grids = arr(*[t.data_ptr() for t in grids])

    def set_weights(self, packed, scales):
        """Point the batch at another copy of the packed weights (same shapes)."""
        self.keep = self.keep[:2] + (list(packed), list(scales)) + self.keep[4:]
        for i, (p, s) in enumerate(zip(packed, scales)):
            self.packed[i] = p.data_ptr()
            self.scales[i] = s.data_ptr()


def higgs_linear_host_batch(batch: HostBatch) -> None:
    """Enqueues copy-in, the layers and copy-out of every layer of `batch` on the current stream with one library call;
    synchronise before reading the y_hosts."""
    _check(lib.higgs_linear_host_batch(batch.count, batch.descs, batch.x, batch.B, batch.packed, batch.scales, batch.grids,
                                       batch.y, batch.y_dtype, batch.ws, batch.ws_bytes, _stream()), "higgs_linear_host_batch")


def higgs_linear_static_capacity() -> int:
    return int(lib.higgs_linear_static_capacity())


def higgs_linear_static(desc: higgs_desc, x: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor,
                        grid: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
    """higgs_linear for callers that cannot allocate: no workspace argument, the scratch is the library's own
    fixed array.  x: cuda [B][K] bf16; y: caller-owned cuda [B][N] fp32 or bf16, written in place.  Raises
    HiggsError(HIGGS_ERR_STATIC_SCRATCH) when the shape does not fit the array."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and y.is_cuda and y.is_contiguous()
    _check(lib.higgs_linear_static(ctypes.byref(desc), _ptr(x), x.shape[0], _ptr(packed), _ptr(scales), _ptr(grid),
                                   _ptr(y), _dtype_code(y), _stream()), "higgs_linear_static")
    return y


def higgs_device_status(clear: bool = True) -> int:
    """Synchronises the current stream and returns the library's device status word (HIGGS_OK unless a bounded
    device-side wait ran out)."""
    return int(lib.higgs_device_status(_stream(), int(bool(clear))))


def scales_to_tile_major(scales: torch.Tensor) -> torch.Tensor:
    """[N][K/g] fp16 -> the tile-major storage order higgs_linear reads (pure data movement)."""
    N, Gn = scales.shape
    return scales.reshape(N // 16, 16, Gn).permute(0, 2, 1).contiguous()


def scales_from_tile_major(scales: torch.Tensor, N: int) -> torch.Tensor:
    """Inverse of scales_to_tile_major: returns [N][K/g]."""
    Gn = scales.numel() // N
    return scales.reshape(N // 16, Gn, 16).permute(0, 2, 1).reshape(N, Gn).contiguous()


def higgs_rotated_bytes(desc: higgs_desc, B: int) -> int:
    return int(lib.higgs_rotated_bytes(ctypes.byref(desc), int(B)))


def higgs_rotated_layout(desc: higgs_desc, B: int) -> int:
    return int(lib.higgs_rotated_layout(ctypes.byref(desc), int(B)))


def higgs_linear_k_splits(desc: higgs_desc, B: int) -> int:
    return int(lib.higgs_linear_k_splits(ctypes.byref(desc), int(B)))


def higgs_linear_uses_atomics(desc: higgs_desc, B: int) -> bool:
    return bool(lib.higgs_linear_uses_atomics(ctypes.byref(desc), B))


def higgs_linear_launch_count(desc: higgs_desc, B: int, y_dtype: int = HIGGS_F32) -> int:
    return int(lib.higgs_linear_launch_count(ctypes.byref(desc), int(B), int(y_dtype)))


def higgs_rht(desc: higgs_desc, x: torch.Tensor, normalised: bool) -> torch.Tensor:
    """x: cuda [rows][K] fp32 or bf16 -> fp32 [rows][K], the transform of Algorithm 1 / Appendix F per group."""
    assert x.is_cuda and x.is_contiguous()
    out = torch.empty(x.shape, dtype=torch.float32, device=x.device)
    _check(lib.higgs_rht(ctypes.byref(desc), _ptr(x), _dtype_code(x), x.shape[0], _ptr(out), int(bool(normalised)),
                         _stream()), "higgs_rht")
    return out


def higgs_pack_codes(desc: higgs_desc, canonical: torch.Tensor) -> torch.Tensor:
    assert canonical.is_cuda and canonical.dtype == torch.uint8 and canonical.is_contiguous()
    packed = torch.empty(max(higgs_packed_bytes(desc), 16), dtype=torch.uint8, device=canonical.device)
    _check(lib.higgs_pack_codes(ctypes.byref(desc), _ptr(canonical), _ptr(packed), _stream()), "higgs_pack_codes")
    return packed


def higgs_make_uniform_grid(n: int, device=None):
    """The MSE-optimal uniform n-level grid (constrained HIGGS; n = 256 is 'CH8').  Returns (grid [n][1], step, mse)."""
    device = device or torch.device("cuda", torch.cuda.current_device())
    grid = torch.empty((n, 1), dtype=torch.float32, device=device)
    out = torch.zeros(2, dtype=torch.float32, device=device)
    _check(lib.higgs_make_uniform_grid(int(n), _ptr(grid), out.data_ptr(), out.data_ptr() + 4, _stream()), "higgs_make_uniform_grid")
    return grid, out[0], out[1]


def higgs_layer_error(desc: higgs_desc, W: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor, grid: torch.Tensor) -> float:
    """Relative quantisation error t^2 = ||W^ - W||^2 / ||W||^2 of the layer (Section 5, 'Measuring Grid Parameters')."""
    assert W.is_cuda and W.is_contiguous() and W.dtype in (torch.float32, torch.bfloat16)
    sums = torch.zeros(3, dtype=torch.float64, device=W.device)
    ws = _workspace(higgs_workspace_bytes(desc, HIGGS_OP_QUANTIZE, 0), W.device)
    _check(lib.higgs_layer_error(ctypes.byref(desc), _ptr(W), _dtype_code(W), _ptr(packed), _ptr(scales), _ptr(grid), _ptr(sums),
                                 _ptr(ws), ws.numel(), _stream()), "higgs_layer_error")
    return float(sums[2].item())


def higgs_quantize_general(p: int, n: int, W: torch.Tensor, grid: torch.Tensor, rht_seed: int, want_error: bool = True):
    """Algorithm 1 for any grid (p <= 4, n <= 4096).  Returns (codes int16-as-uint16 [N][K/1024][ceil(1024/p)],
    scales fp16 [N][K/1024] row-major, t^2 or None)."""
    assert W.is_cuda and W.is_contiguous() and W.dtype in (torch.float32, torch.bfloat16)
    assert grid.is_cuda and grid.dtype == torch.float32 and grid.is_contiguous() and tuple(grid.shape) == (n, p)
    N, K = W.shape
    tuples = lib.higgs_general_tuples(p)
    codes = torch.empty((N, K // 1024, max(tuples, 1)), dtype=torch.uint16, device=W.device)
    scales = torch.empty((N, K // 1024), dtype=torch.float16, device=W.device)
    sums = torch.zeros(3, dtype=torch.float64, device=W.device) if want_error else None
    _check(lib.higgs_quantize_general(p, n, N, K, rht_seed, _ptr(W), _dtype_code(W), _ptr(grid), _ptr(codes), _ptr(scales),
                                      _ptr(sums), _stream()), "higgs_quantize_general")
    return codes, scales, (float(sums[2].item()) if want_error else None)


def higgs_allocate_bits(alpha, t2, bits64, sizes, budget64: int):
    """Eq. 4 on the host: returns (choice per layer, objective).  bits64 / budget64 in units of 1/64 bit per weight."""
    import numpy as np
    a = np.ascontiguousarray(alpha, dtype=np.float64)
    t = np.ascontiguousarray(t2, dtype=np.float64)
    b = np.ascontiguousarray(bits64, dtype=np.int32)
    d = np.ascontiguousarray(sizes, dtype=np.int64)
    L, J = t.shape
    assert a.shape == (L,) and b.shape == (J,) and d.shape == (L,)
    choice = np.zeros(L, dtype=np.int32)
    obj = ctypes.c_double(0.0)
    _check(lib.higgs_allocate_bits(L, J, a.ctypes.data, t.ctypes.data, b.ctypes.data, d.ctypes.data, int(budget64),
                                   choice.ctypes.data, ctypes.addressof(obj)), "higgs_allocate_bits")
    return choice, float(obj.value)


def higgs_dequantize(desc: higgs_desc, packed: torch.Tensor, scales: torch.Tensor, grid: torch.Tensor,
                     out_dtype: torch.dtype = torch.float32) -> torch.Tensor:
    """packed codes + scales -> the matrix [N][K] the quantised layer stands for (Appendix F, 'Dequantization')."""
    W = torch.empty((desc.N, desc.K), dtype=out_dtype, device=packed.device)
    ws = _workspace(higgs_workspace_bytes(desc, HIGGS_OP_QUANTIZE, 0), packed.device)
    _check(lib.higgs_dequantize(ctypes.byref(desc), _ptr(packed), _ptr(scales), _ptr(grid), _ptr(W), _dtype_code(W),
                                _ptr(ws), ws.numel(), _stream()), "higgs_dequantize")
    return W


def higgs_unpack_codes(desc: higgs_desc, packed: torch.Tensor) -> torch.Tensor:
    assert packed.is_cuda and packed.dtype == torch.uint8
    canonical = torch.empty((desc.N, desc.K // desc.p), dtype=torch.uint8, device=packed.device)
    _check(lib.higgs_unpack_codes(ctypes.byref(desc), _ptr(packed), _ptr(canonical), _stream()), "higgs_unpack_codes")
    return canonical
