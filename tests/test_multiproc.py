"""world_size-2 gloo test of the benchmark's multi-rank logic (replicas only: no data-path collective): the timed
region's duration is the MAX over ranks, the reported value the sum of all ranks' bytes over that time."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        ms = bench.max_over_ranks(local_ms, torch.device("cpu"), world)
        value = bench.aggregate_value(bytes_per_step=1_000_000, steps=4, ms=ms, world=world)
        out.put((rank, ms, value))
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_value():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in res:
        assert ms == 15.0                                  # the slowest rank's time on every rank
        assert abs(value - 2 * 1_000_000 / (15.0 / 4 * 1e-3) / 1e9) < 1e-9


def test_single_rank_is_identity():
    assert bench.max_over_ranks(3.5, torch.device("cpu"), 1) == 3.5
    assert abs(bench.aggregate_value(2_000_000, 2, 4.0, 1) - 1.0) < 1e-12


# ---- row-sharded layer: the host-side protocol of higgs_linear_gather on two CPU ranks --------------------------------
def _gather_worker(rank, world, port, out):
    import numpy as np

    import oracle
    from paper_2411_17525_b200 import binding
    from synth import inputs
    from tests.golden import make_grids

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        N, K, B, g, xi = 384, 1024, 3, 1024, 5
        grid = make_grids.load(2, 64)
        W = inputs.make_weights(N, K, seed=9, bf16=True).astype(np.float64)      # every rank can draw the full matrix...
        x = inputs.make_activations(B, K, seed=10).astype(np.float64)
        r0, r1 = binding.shard_rows(N, world, rank)                               # ...but encodes and multiplies only its rows
        q = oracle.quantize(W[r0:r1], g, grid, xi)
        sc = oracle.round_scales_fp16(q.scales).astype(np.float64)
        y_shard = oracle.linear_dense(x, q.codes, sc, g, grid, xi)              # [B][r1 - r0]
        # what the fused epilogue does over peer memory: this shard's columns land in every rank's [B][N] buffer
        spans = [None] * world
        dist.all_gather_object(spans, (r0, r1))
        blocks = [None] * world
        dist.all_gather_object(blocks, y_shard)
        y = np.full((B, N), np.nan)
        for (a, b), blk in zip(spans, blocks):
            y[:, a:b] = blk
        dist.barrier()                                                            # "all shards written" before any reader
        q_all = oracle.quantize(W, g, grid, xi)
        y_ref = oracle.linear_dense(x, q_all.codes, oracle.round_scales_fp16(q_all.scales).astype(np.float64), g, grid, xi)
        out.put((rank, spans, float(np.max(np.abs(y - y_ref)))))
    finally:
        dist.destroy_process_group()


def test_row_sharded_layer_protocol_on_two_ranks():
    """Rows are independent in Algorithm 1 and in the product of Appendix F, so shards encoded and multiplied separately
    and gathered by column blocks reproduce the unsharded layer exactly; the shard spans tile [0, N) in 128-row units."""
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gather_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=300) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, spans, err in res:
        assert spans == [(0, 256), (256, 384)]          # three 128-row units over two ranks: 2 + 1
        assert err == 0.0


# ---- K-sharded layer: the host-side protocol of higgs_linear_kshard + higgs_reduce_slots on two CPU ranks ------------
def _kshard_worker(rank, world, port, out):
    import numpy as np

    import oracle
    from paper_2411_17525_b200 import binding
    from synth import inputs
    from synth import grids as stored

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        N, K, B, g, xi = 64, 4096, 2, 1024, 0x48494747
        grid = stored.load(2, 64)
        W = inputs.make_weights(N, K, seed=19, bf16=True).astype(np.float64)
        x = inputs.make_activations(B, K, seed=20).astype(np.float64)
        Kr = K // world
        k0 = rank * Kr                                                            # a multiple of the group size
        xi_r = binding.higgs_shard_seed(xi, k0)                                   # the shard's signs are the layer's, shifted
        q = oracle.quantize(W[:, k0:k0 + Kr], g, grid, xi_r)
        sc = oracle.round_scales_fp16(q.scales).astype(np.float64)
        part = oracle.linear_dense(x[:, k0:k0 + Kr], q.codes, sc, g, grid, xi_r)  # this rank's fp partial [B][N]
        slots = [None] * world                                                    # what the epilogues write into every rank's slot buffer
        dist.all_gather_object(slots, part)
        dist.barrier()                                                            # "all partials written" before the reduction
        y = np.zeros((B, N))
        for r in range(world):                                                    # higgs_reduce_slots: slot order
            y = y + slots[r]
        q_all = oracle.quantize(W, g, grid, xi)
        same_codes = bool(np.array_equal(q_all.codes[:, k0 // 2:(k0 + Kr) // 2], q.codes))
        y_ref = oracle.linear_dense(x, q_all.codes, oracle.round_scales_fp16(q_all.scales).astype(np.float64), g, grid, xi)
        out.put((rank, same_codes, float(np.max(np.abs(y - y_ref)) / np.max(np.abs(y_ref)))))
    finally:
        dist.destroy_process_group()


def test_k_sharded_layer_protocol_on_two_ranks():
    """The rotation is local to a 1024-group (Appendix F), so a layer cut along K on group boundaries is a sum of
    independent layers; with the shifted seed each shard carries exactly the codes of its columns of the unsharded
    layer, and the slot-ordered sum of the partial outputs is the unsharded output (up to fp64 summation order)."""
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_kshard_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=300) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, same_codes, err in res:
        assert same_codes
        assert err < 1e-12


def test_shard_seed_shifts_the_sign_sequence():
    import oracle
    from paper_2411_17525_b200 import binding
    for xi in (0, 7, 0x48494747, 2**64 - 5):
        for k0 in (0, 1024, 4096, 28672 - 1024):
            s = binding.higgs_shard_seed(xi, k0)
            assert [oracle.sign(s, j) for j in range(0, 2048, 37)] == [oracle.sign(xi, k0 + j) for j in range(0, 2048, 37)]


def test_shard_rows_tiles_the_layer():
    from paper_2411_17525_b200 import binding
    for N, world in [(4096, 8), (14336, 8), (1024, 3), (128, 2), (8192, 5)]:
        spans = [binding.shard_rows(N, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == N
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        assert all(s[0] % 128 == 0 and s[1] % 128 == 0 for s in spans)
        sizes = [s[1] - s[0] for s in spans]
        assert max(sizes) - min(sizes) <= 128


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` (the oracle timed on the host cores) runs without a GPU and prints one JSON line with
    the keys of the benchmark contract, on the same metric, unit and workload name as the CUDA arm."""
    import json
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1"],
                         capture_output=True, text=True, timeout=600, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["metric"] == "higgs_linear_effective_weight_bandwidth" and line["unit"] == "GB/s"
    assert line["steps"] == 2 and line["value"] > 0 and line["dtype"] == "f64" and line["vs_baseline"] is None
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("llama-3.1-70b layer set (7 matrices), grid mixed ")
    assert line["config"]["workload"].endswith("g=1024, batch 1")
