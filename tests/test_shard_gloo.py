"""Multi-rank host logic on CPU: two gloo ranks shard the units, reduce their timings with a max
and agree on the whole-job throughput."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_05534_b200 import shard


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        units = shard.rank_units(3, 2, rank, world)
        gathered = [None] * world
        dist.all_gather_object(gathered, units)
        ms = shard.max_over_ranks(10.0 + 5.0 * rank)            # rank 1 is the slow one
        value = shard.aggregate_throughput(1000, world, ms)
        if rank == 0:
            out.put((gathered, ms, value))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_units_and_reduce_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, ms, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    a, b = gathered
    assert len(a) == len(b) == 6
    assert not set(a) & set(b), "ranks must not share a (layer, sequence) unit"
    assert {s for _, s in a} == {0, 1} and {s for _, s in b} == {2, 3}
    assert {l for l, _ in a} == {0, 1, 2}
    assert ms == 15.0                                            # max over ranks, not the mean
    assert value == pytest.approx(2 * 1000 / 15e-3)


def test_single_process_is_identity():
    assert shard.max_over_ranks(3.5) == 3.5
    assert shard.rank_units(2, 1, 0, 1) == [(0, 0), (1, 0)]
    with pytest.raises(ValueError):
        shard.rank_units(2, 1, 2, 2)
    assert shard.seed_offset(1, 3) != shard.seed_offset(0, 3)
