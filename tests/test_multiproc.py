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
