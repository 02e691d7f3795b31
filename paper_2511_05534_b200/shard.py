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


# ---- sharding one layer by KV head (tensor-parallel ownership of the cache) -------------------------
#
# Inside a unit the KV heads share exactly one number: rho, the mean over all query heads of the
# cross-modal mass (Eq. 6).  A rank that owns a contiguous range of KV heads (and their query heads)
# therefore runs the whole path on its own heads and takes part in ONE collective, a sum of n_units
# floats between the scoring step and the matching step; K and V never move.

def head_range(n_kv_heads: int, rank: int, world: int) -> Tuple[int, int]:
    """[first, last) KV head of `rank`; equal contiguous shares (rho is then the plain mean of the ranks' means)."""
    if not 0 <= rank < world:
        raise ValueError("rank %d outside world of %d" % (rank, world))
    if n_kv_heads % world != 0:
        raise ValueError("%d KV heads do not split evenly over %d ranks" % (n_kv_heads, world))
    per = n_kv_heads // world
    return rank * per, (rank + 1) * per


def compress_layer_head_sharded(p_local, q_win, k, v, modality, out, ws, group=None, steps=None):
    """The compression path on this rank's heads, with the layer's rho taken over all ranks' heads.

    p_local describes the rank's share (its own n_q_heads / n_kv_heads); q_win, k, v hold only those
    heads.  `out` is a dict of preallocated tensors: importance, cross_mass, rho, strategy,
    retained, evicted, match, match_sim, k_out, v_out (rho / strategy sized [n_units]) and
    rho_local [n_units], strategy_local [n_units] as scratch.  `steps` is the module that provides
    the step entry points (default: the CUDA binding).  Every arithmetic step runs in those entry
    points; this function only orders them around the one all-reduce.
    """
    import dataclasses
    import torch.distributed as dist
    if steps is None:
        from . import binding as steps
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    steps.flowmm_score(p_local, q_win, k, modality, out["importance"], out["cross_mass"], ws)
    # head mean over this rank's heads ...
    steps.flowmm_layer_flow(p_local, out["cross_mass"], out["rho_local"], out["strategy_local"])
    # ... summed over the ranks (the one collective: n_units floats) ...
    if world > 1:
        dist.all_reduce(out["rho_local"], op=dist.ReduceOp.SUM, group=group)
    # ... and divided by their number together with the theta rule, again by the layer-flow step: a single
    # pseudo-head per unit whose "window" is the number of ranks
    p_flow = dataclasses.replace(p_local, n_q_heads=1, n_kv_heads=1, seq_len=max(world, 1), window=world, n_keep=1,
                                 keep_window=0)
    steps.flowmm_layer_flow(p_flow, out["rho_local"].view(-1, 1), out["rho"], out["strategy"])
    steps.flowmm_select(p_local, out["importance"], out["retained"], out["evicted"], ws)
    steps.flowmm_match(p_local, k, out["importance"], modality, out["retained"], out["evicted"], out["strategy"],
                       out["match"], out["match_sim"], ws)
    steps.flowmm_merge(p_local, k, v, out["retained"], out["evicted"], out["match"], out["match_sim"],
                       out["k_out"], out["v_out"], ws)
    return out
