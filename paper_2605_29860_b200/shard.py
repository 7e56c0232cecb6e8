"""Row sharding across GPUs for the ESPO hot path.

Trajectories are independent units: neither ``espo_step`` nor ``espo_advantages`` exchanges data
between rows, so N GPUs run N disjoint row ranges with no data-path collective.  This module holds
the little host-side logic that goes with it: which rows and seeds a rank owns, and the reduction
of per-rank timings (the only communication the benchmark does).
"""
from __future__ import annotations

from typing import List, Tuple

import torch


def shard_rows(n_rows: int, world: int) -> List[Tuple[int, int]]:
    """Contiguous, disjoint row ranges [lo, hi) that cover 0..n_rows, sizes differing by at most one."""
    if world < 1 or n_rows < 0:
        raise ValueError("world must be >= 1 and n_rows >= 0")
    return [(r * n_rows // world, (r + 1) * n_rows // world) for r in range(world)]


def rank_plan(rank: int, world: int, rows_per_rank: int, base_seed: int = 1234) -> dict:
    """Weak-scaling plan: every rank owns ``rows_per_rank`` trajectories of one global batch.

    Returns the rank's slice of global trajectory ids, the Philox seed of its state and the seed offset
    of its synthetic inputs; both seeds differ between ranks so that no two GPUs draw the same noise.
    """
    if not 0 <= rank < world:
        raise ValueError("rank outside [0, world)")
    lo = rank * rows_per_rank
    return {"rows": (lo, lo + rows_per_rank), "state_seed": base_seed + rank, "data_seed_offset": 10 * rank,
            "global_rows": world * rows_per_rank}


def max_over_ranks(values, dist=None, device="cpu") -> list:
    """Element-wise maximum of a list of floats over all ranks (the timings of a multi-GPU run)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def sum_over_ranks(values, dist=None, device="cpu") -> list:
    """Element-wise sum over all ranks (rows processed, rows stopped)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t.tolist()


# ---- vocabulary shards (tensor-parallel LM head): espo_step_partial on every rank, one all-gather, espo_step_merge ----

def vocab_shards(V: int, world: int, multiple: int = 128) -> List[Tuple[int, int]]:
    """Contiguous (offset, size) shards of the vocabulary, one per rank; every offset is a multiple of ``multiple``
    (espo_step_partial wants a multiple of 4, and of 1024 with the hierarchical sampler, whose draws belong to blocks of
    1024 ids; 128 keeps rows of bf16 shards 256-byte aligned).  Trailing ranks may get
    an empty shard when V is small."""
    if world < 1 or V < 1 or multiple < 4 or multiple % 4:
        raise ValueError("need world >= 1, V >= 1 and a shard granularity that is a multiple of 4")
    units = (V + multiple - 1) // multiple
    out = []
    for r in range(world):
        lo = min((r * units // world) * multiple, V)
        hi = min(((r + 1) * units // world) * multiple, V)
        out.append((lo, hi - lo))
    return out


def all_gather_partials(local: torch.Tensor, dist=None) -> torch.Tensor:
    """Brings every rank's partials (float32 [rows, 8], one espo_partial per row) together as [world, rows, 8], in rank
    order, which is the layout espo_step_merge reads.  The only data-path collective of the vocabulary-sharded step:
    32 bytes per row and rank."""
    if local.dim() != 2 or local.shape[1] != 8 or local.dtype != torch.float32:
        raise ValueError("partials must be float32 [rows, 8]")
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local.contiguous().unsqueeze(0)
    world = dist.get_world_size()
    out = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    dist.all_gather(list(out.unbind(0)), local.contiguous())
    return out


def all_gather_batch_stats(stats, dist=None, device="cpu") -> list:
    """Every rank's six batch statistics (the numbers espo_end_batch returns: mean, variance, stop rate, tokens,
    trajectories, stopped), in rank order -- the input of espo_end_batch_merge.  The only collective the row-sharded
    method needs, once per training batch."""
    row = [float(x) for x in stats]
    if len(row) != 6:
        raise ValueError("six numbers per rank")
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [row]
    mine = torch.tensor(row, dtype=torch.float64, device=device)
    out = [torch.empty_like(mine) for _ in range(dist.get_world_size())]
    dist.all_gather(out, mine)
    return [t.tolist() for t in out]
