"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its host logic
(size queries, argument validation, the sign function) behaves as include/higgs.h documents."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2411_17525_b200 as hb
from paper_2411_17525_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(higgs_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 12 and "higgs_linear" in names and "higgs_quantize" in names and "higgs_make_grid" in names
    lib = ctypes.CDLL(hb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) <= set(names)


def test_sign_function_matches_oracle_statement():
    for seed in (0, 1, 0x48494747, 2**64 - 1, 0x123456789ABCDEF0):
        got = [hb.higgs_sign(seed, j) for j in range(512)]
        want = [int(oracle.sign(seed, j)) for j in range(512)]
        assert got == want
    assert hb.higgs_sign(7, 10**12) == int(oracle.sign(7, 10**12))


def test_size_queries():
    d = hb.make_desc(2, 256, 4096, 14336, 1)
    assert hb.higgs_packed_bytes(d) == 4096 * 14336 // 2          # 4 bits per weight
    assert hb.higgs_scales_bytes(d) == 4096 * 14 * 2              # one fp16 per (row, group)
    assert hb.higgs_canonical_bytes(d) == 4096 * 14336 // 2
    d = hb.make_desc(2, 64, 4096, 4096, 1)
    assert hb.higgs_packed_bytes(d) == 4096 * 4096 * 3 // 8       # 3 bits per weight
    d = hb.make_desc(1, 16, 1024, 4096, 1)
    assert hb.higgs_packed_bytes(d) == 1024 * 4096 // 2
    assert hb.higgs_canonical_bytes(d) == 1024 * 4096
    assert hb.higgs_workspace_bytes(d, hb.HIGGS_OP_LINEAR, 16) >= 16 * 4096 * 2
    assert hb.higgs_workspace_bytes(d, hb.HIGGS_OP_LINEAR, 0) == 0
    # effective bits per weight incl. scales, as the paper counts them: 4 + 16/1024
    d = hb.make_desc(2, 256, 4096, 4096, 1)
    bpw = 8.0 * (hb.higgs_packed_bytes(d) + hb.higgs_scales_bytes(d)) / (4096 * 4096)
    assert round(bpw, 2) == 4.02


@pytest.mark.parametrize("p,n,g,N,K", [(2, 100, 1024, 16, 1024), (3, 256, 1024, 16, 1024), (2, 256, 512, 16, 1024),
                                       (2, 256, 1024, 15, 1024), (2, 256, 1024, 16, 1000), (1, 64, 1024, 16, 1024)])
def test_unsupported_descriptors_are_refused(p, n, g, N, K):
    d = hb.make_desc(p, n, N, K, 1, g=g)
    assert hb.higgs_packed_bytes(d) == 0
    rc = binding.lib.higgs_linear(ctypes.byref(d), None, 1, None, None, None, None, 0, None, 0, None)
    assert rc == hb.HIGGS_ERR_UNSUPPORTED
    rc = binding.lib.higgs_quantize(ctypes.byref(d), None, 0, None, None, None, None, None, 0, None)
    assert rc == hb.HIGGS_ERR_UNSUPPORTED


def test_invalid_arguments_are_refused_before_any_cuda_call():
    d = hb.make_desc(2, 256, 16, 1024, 1)
    L = binding.lib
    assert L.higgs_linear(None, None, 1, None, None, None, None, 0, None, 0, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_linear(ctypes.byref(d), None, 1, None, None, None, None, 0, None, 0, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_linear(ctypes.byref(d), None, -1, None, None, None, None, 0, None, 0, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_linear(ctypes.byref(d), None, 0, None, None, None, None, 0, None, 0, None) == hb.HIGGS_OK  # empty batch
    assert L.higgs_linear(ctypes.byref(d), None, 1, None, None, None, None, 7, None, 0, None) == hb.HIGGS_ERR_UNSUPPORTED
    assert L.higgs_quantize(ctypes.byref(d), None, 0, None, None, None, None, None, 0, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_quantize(ctypes.byref(d), None, 1, None, None, None, None, None, 0, None) == hb.HIGGS_ERR_UNSUPPORTED
    # misaligned and undersized workspace (fake non-null addresses are never dereferenced on these paths)
    a = ctypes.c_void_p(0x1000)
    assert L.higgs_linear(ctypes.byref(d), a, 1, a, a, a, a, 0, ctypes.c_void_p(0x1010), 1 << 20, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_linear(ctypes.byref(d), a, 1, a, a, a, a, 0, a, 16, None) == hb.HIGGS_ERR_WORKSPACE
    assert L.higgs_quantize(ctypes.byref(d), a, 0, a, a, a, None, a, 16, None) == hb.HIGGS_ERR_WORKSPACE
    assert L.higgs_make_grid(2, 256, a, 100, 10, a, None, None, a, 1 << 30, None) == hb.HIGGS_ERR_INVALID_ARG  # fewer samples than points
    assert L.higgs_make_grid(5, 256, a, 1000, 10, a, None, None, a, 1 << 30, None) == hb.HIGGS_ERR_UNSUPPORTED
    assert L.higgs_make_grid(2, 4097, a, 10000, 10, a, None, None, a, 1 << 30, None) == hb.HIGGS_ERR_UNSUPPORTED
    # batched host call
    assert L.higgs_linear_host_batch(-1, None, None, 1, None, None, None, None, 0, None, None, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_linear_host_batch(0, None, None, 1, None, None, None, None, 0, None, None, None) == hb.HIGGS_OK
    assert L.higgs_linear_host_batch(2, None, None, 1, None, None, None, None, 0, None, None, None) == hb.HIGGS_ERR_INVALID_ARG
    # general-grid encoder
    assert L.higgs_general_tuples(3) == 342 and L.higgs_general_tuples(2) == 512 and L.higgs_general_tuples(5) == 0
    assert L.higgs_quantize_general(5, 16, 16, 1024, 1, a, 0, a, a, a, None, None) == hb.HIGGS_ERR_UNSUPPORTED
    assert L.higgs_quantize_general(3, 830, 16, 1000, 1, a, 0, a, a, a, None, None) == hb.HIGGS_ERR_UNSUPPORTED
    assert L.higgs_quantize_general(3, 830, 16, 1024, 1, None, 0, a, a, a, None, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_quantize_general(3, 830, 0, 1024, 1, None, 0, None, None, None, None, None) == hb.HIGGS_OK
    assert L.higgs_make_grid(2, 256, a, 1000, 10, a, None, None, a, 16, None) == hb.HIGGS_ERR_WORKSPACE
    empty = hb.make_desc(2, 256, 0, 1024, 1)
    assert L.higgs_quantize(ctypes.byref(empty), None, 0, None, None, None, None, None, 0, None) == hb.HIGGS_OK
    for s in range(7):
        assert isinstance(hb.status_string(s), str) and hb.status_string(s)


def test_layout_version_is_checked():
    d = hb.make_desc(2, 256, 16, 1024, 1)
    assert d.layout_version == hb.HIGGS_LAYOUT_VERSION and hb.higgs_packed_bytes(d) > 0
    d.layout_version = hb.HIGGS_LAYOUT_VERSION + 1          # a stream written by some other version of the layouts
    assert hb.higgs_packed_bytes(d) == 0
    assert binding.lib.higgs_linear(ctypes.byref(d), None, 1, None, None, None, None, 0, None, 0, None) == hb.HIGGS_ERR_UNSUPPORTED


def test_shard_rows_partitions_the_rows():
    for N, world, mult in ((28672, 8, 128), (4096, 3, 128), (1024, 8, 128), (512, 5, 16), (14336, 7, 128)):
        spans = [hb.shard_rows(N, world, r, mult) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == N
        for (b0, e0), (b1, e1) in zip(spans, spans[1:]):
            assert e0 == b1                                                      # contiguous, in rank order
        sizes = [e - b for b, e in spans]
        assert all(s % mult == 0 for s in sizes) and max(sizes) - min(sizes) <= mult
        assert sizes == sorted(sizes, reverse=True)                              # the remainder goes to the first ranks
    b, c = ctypes.c_int64(), ctypes.c_int64()
    L = binding.lib
    assert L.higgs_shard_rows(1000, 4, 0, 128, ctypes.byref(b), ctypes.byref(c)) == hb.HIGGS_ERR_UNSUPPORTED
    assert L.higgs_shard_rows(1024, 4, 4, 128, ctypes.byref(b), ctypes.byref(c)) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_shard_rows(1024, 4, 0, 24, ctypes.byref(b), ctypes.byref(c)) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_shard_rows(1024, 4, 0, 128, None, ctypes.byref(c)) == hb.HIGGS_ERR_INVALID_ARG


def test_seeded_grid_and_helper_arguments():
    a = ctypes.c_void_p(0x1000)
    L = binding.lib
    assert L.higgs_make_grid_seeded(2, 256, 1, 5, 10, a, None, None, a, 1 << 30, None) == hb.HIGGS_ERR_INVALID_ARG   # 32 samples < 256 points
    assert L.higgs_make_grid_seeded(2, 256, 1, 30, 10, a, None, None, a, 1 << 30, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_make_grid_seeded(5, 256, 1, 18, 10, a, None, None, a, 1 << 30, None) == hb.HIGGS_ERR_UNSUPPORTED
    assert L.higgs_make_grid_seeded(2, 256, 1, 18, 10, a, None, None, a, 1024, None) == hb.HIGGS_ERR_WORKSPACE
    d = hb.make_desc(2, 256, 0, 1 << 18, 0)
    assert hb.higgs_workspace_bytes(d, hb.HIGGS_OP_MAKE_GRID_SEEDED) >= hb.higgs_workspace_bytes(d, hb.HIGGS_OP_MAKE_GRID) + (1 << 18) * 2 * 4
    assert L.higgs_gaussian_samples(2, 1, 0, None, None) == hb.HIGGS_OK
    assert L.higgs_gaussian_samples(2, 1, 16, None, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_launch_floor(0, 32, 0, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_launch_floor(148, 2048, 0, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_selftest_wait(0, 100, None, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_selftest_wait(2, 100, a, None) == hb.HIGGS_ERR_INVALID_ARG


def test_encoder_table_queries_and_arguments():
    """The prepared search table: one 32-bit list per cell (128 x 128 cells for p = 2, 1024 for p = 1); argument
    checks run before any CUDA call."""
    L = binding.lib
    a, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1008)
    assert L.higgs_encoder_table_bytes(2, 256) == 128 * 128 * 4
    assert L.higgs_encoder_table_bytes(2, 64) == 128 * 128 * 4
    assert L.higgs_encoder_table_bytes(1, 16) == 1024 * 4
    assert L.higgs_encoder_table_bytes(3, 830) == 0 and L.higgs_encoder_table_bytes(2, 100) == 0
    assert L.higgs_make_encoder_table(3, 830, a, a, None) == hb.HIGGS_ERR_UNSUPPORTED
    assert L.higgs_make_encoder_table(2, 256, None, a, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_make_encoder_table(2, 256, a, None, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_make_encoder_table(2, 256, a, odd, None) == hb.HIGGS_ERR_INVALID_ARG
    d = hb.make_desc(2, 256, 4096, 4096, 1)
    P = ctypes.byref(d)
    ws = hb.higgs_workspace_bytes(d, hb.HIGGS_OP_QUANTIZE)
    assert ws >= L.higgs_encoder_table_bytes(2, 256)         # a large layer's workspace always holds the table
    assert L.higgs_quantize_prepared(P, None, hb.HIGGS_BF16, a, a, a, a, None, a, ws, None) == hb.HIGGS_ERR_INVALID_ARG
    assert L.higgs_quantize_prepared(P, a, hb.HIGGS_BF16, a, odd, a, a, None, a, ws, None) == hb.HIGGS_ERR_INVALID_ARG    # table alignment
    assert L.higgs_quantize_prepared(P, a, hb.HIGGS_BF16, a, a, a, a, odd, a, ws, None) == hb.HIGGS_ERR_INVALID_ARG      # canonical alignment
    assert L.higgs_quantize_prepared(P, a, hb.HIGGS_BF16, a, a, a, a, None, None, 0, None) == hb.HIGGS_ERR_INVALID_ARG   # no canonical_out: workspace needed
    assert L.higgs_quantize_prepared(P, a, hb.HIGGS_BF16, a, a, a, a, None, a, 16, None) == hb.HIGGS_ERR_WORKSPACE
    empty = hb.make_desc(2, 256, 0, 4096, 1)
    assert L.higgs_quantize_prepared(ctypes.byref(empty), None, hb.HIGGS_BF16, None, None, None, None, None, None, 0, None) == hb.HIGGS_OK
