"""Multi-GPU plumbing: requests are independent, so a batch shards over ranks with no data-path
collective.  The only communication is the reduction of the benchmark's timings (max over ranks)
and work counts (sum over ranks), over whatever process group the caller initialised
(NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import Dict

import torch


def reduce_timings(times_ms: Dict[str, float], counts: Dict[str, float], dist=None, device="cpu"):
    """Max of every timing and sum of every count over the ranks of the default process group.

    With dist=None (single process) the inputs are returned unchanged.
    """
    if dist is None:
        return dict(times_ms), dict(counts)
    keys_t, keys_c = sorted(times_ms), sorted(counts)
    t = torch.tensor([times_ms[k] for k in keys_t], dtype=torch.float64, device=device)
    c = torch.tensor([counts[k] for k in keys_c], dtype=torch.float64, device=device)
    if keys_t:       # an empty dictionary is not reduced at all (no zero-element collective)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if keys_c:
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return ({k: float(v) for k, v in zip(keys_t, t.tolist())},
            {k: float(v) for k, v in zip(keys_c, c.tolist())})


def whole_job_throughput(total_bytes: float, max_ms_per_step: float) -> float:
    """GB/s of the whole job: bytes all ranks processed per step over the slowest rank's step time."""
    return total_bytes / (max_ms_per_step * 1e-3) / 1e9


# --------------------------------------------------------------------------------------------------
# One request's cache split over devices (Section 5): every device sweeps the shards it holds and
# returns (O, log Z) per shard; the owner merges.  The states are tiny (one "j-th" of the sweep's
# bytes), so the exchange is a gather of [B, S_local, Hq, D] + [B, S_local, Hq] per rank.  On GPUs
# the same exchange needs no collective at all: with out_shards / out_shard_offset in the parameters
# (rank_sweep_params) every rank's qf_decode_partial writes its slots of the OWNER's [B, S, Hq, D] arrays,
# passed as peer-mapped pointers; the sweep kernel writes shard states with plain stores, so its epilogue
# is the transfer (Section 3: results are left where the other side reads them), and the owner merges after a barrier.
# --------------------------------------------------------------------------------------------------
def shard_slice(max_shards: int, world_size: int, rank: int) -> range:
    """Shard slots [lo, hi) of every request that ``rank`` sweeps: equal blocks of ceil(S/world)."""
    per = -(-max_shards // world_size)
    lo = min(max_shards, rank * per)
    return range(lo, min(max_shards, lo + per))


def local_shard_ranges(shard_ranges, max_shards: int, world_size: int, rank: int):
    """The rank's view of the shard table: [B, S_local, 2] with S_local = ceil(S/world), padded with
    empty ranges (0, 0) so that every rank sweeps the same number of slots."""
    per = -(-max_shards // world_size)
    sl = shard_slice(max_shards, world_size, rank)
    out = torch.zeros((shard_ranges.shape[0], per, 2), dtype=shard_ranges.dtype, device=shard_ranges.device)
    out[:, :len(sl)] = shard_ranges[:, sl.start:sl.stop]
    return out


def rank_sweep_params(p, world_size: int, rank: int):
    """Parameters of ``rank``'s sweep when every rank writes its shard states straight into the merging device's
    arrays (no gather): the rank sweeps S_local = ceil(S/world) slots (``local_shard_ranges``) and places them at
    slots [rank * S_local, (rank + 1) * S_local) of arrays laid out for world * S_local slots per request.
    The merging device then calls qf_combine with max_shards = world * S_local (padded slots are empty)."""
    import copy
    per = -(-int(p.max_shards) // world_size)
    q = copy.copy(p)
    q.max_shards = per
    q.out_shards = per * world_size
    q.out_shard_offset = rank * per
    return q


def gather_shard_states(o_local: torch.Tensor, lse_local: torch.Tensor, max_shards: int, dist):
    """All ranks' shard states, concatenated in shard order: o [B, S, Hq, D], lse [B, S, Hq].

    o_local [B, S_local, Hq, D], lse_local [B, S_local, Hq]; padded slots carry lse = -inf and are
    dropped.  Every rank receives the result (an all-gather keeps the code path identical on gloo and
    NCCL); only the owner needs it.
    """
    world = dist.get_world_size()
    o_all = [torch.empty_like(o_local) for _ in range(world)]
    l_all = [torch.empty_like(lse_local) for _ in range(world)]
    dist.all_gather(o_all, o_local.contiguous())
    dist.all_gather(l_all, lse_local.contiguous())
    o = torch.cat(o_all, dim=1)[:, :max_shards]
    lse = torch.cat(l_all, dim=1)[:, :max_shards]
    return o, lse
