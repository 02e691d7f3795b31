"""Host-side sharding of a workload over ranks (one process per GPU).

The (layer, sequence) units of the compression are independent problems, so ranks share
nothing on the data path: every rank compresses its own sequences through the whole layer
stack (weak scaling; per-rank work is fixed) and only the timing is reduced (max over ranks).
This module holds that bookkeeping; it has none of the method's arithmetic and works with
any torch.distributed backend (nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def rank_units(n_layers: int, n_seqs: int, rank: int, world: int) -> List[Tuple[int, int]]:
    """(layer, global sequence id) units of `rank`: the full layer stack for its own
    `n_seqs` sequences, numbered rank * n_seqs ... so that no two ranks share a sequence."""
    if not 0 <= rank < world:
        raise ValueError("rank %d outside world of %d" % (rank, world))
    return [(layer, rank * n_seqs + s) for layer in range(n_layers) for s in range(n_seqs)]


def seed_offset(rank: int, input_set: int) -> int:
    """Distinct generator offset per (rank, rotating input set)."""
    return rank * 100 + input_set


def max_over_ranks(ms: float, device=None) -> float:
    """The slowest rank's time; identity when no process group is up."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(tokens_layers_per_rank: int, world: int, ms_step_max: float) -> float:
    """Whole-job tokens x layers per second: every rank did `tokens_layers_per_rank` in the
    slowest rank's step time."""
    return world * tokens_layers_per_rank / (ms_step_max * 1e-3)
