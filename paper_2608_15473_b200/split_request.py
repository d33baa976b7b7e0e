"""One request's cache split over devices (Section 5: a cache may be split anywhere, every part returns
(O, log Z), and the parts merge in any order; Section 3: a result is left in memory the other side reads).

One process per GPU.  Rank r holds the pages of the shards it owns and nothing else; the cache never moves.
A step is:

    1. the owner's query goes to every rank                       (the only bytes that travel out:
                                                                   B * Hq * D * 2, a broadcast)
    2. every rank sweeps its own shards with qf_decode_partial,    (K/V stay local to the GPU that holds them;
       writing the shard states straight into ITS SLOTS of the      the states, B * S_local * Hq * (D + 2) * 4
       owner's [B, S, Hq, D] / [B, S, Hq] arrays                    bytes, leave through the sweep's own
                                                                   epilogue stores into peer-mapped memory)
    3. a barrier on the stream (a one-element all-reduce)
    4. the owner merges with qf_combine

Steps follow one another without any other synchronisation: the next step's broadcast is enqueued by the owner
after its merge, so no rank receives the next query (and none starts overwriting its slots) before the owner
has finished reading them.

The owner's arrays are ordinary device memory of the owner's GPU, exported as CUDA IPC handles over the
process group and opened by the other ranks; a rank's kernels reach them with plain stores over NVLink.
No TMA load, bulk copy or library kernel is ever given a peer pointer: every K/V tile a rank reads lives in
its own memory, and the peer arrays are only ever the destination of ordinary stores.

``transport="gather"`` is the comparison arm: every rank sweeps into local arrays and the states are
all-gathered (NCCL on GPUs, gloo in the CPU tests).

The sweep and the merge themselves are passed in as callables, so that the CPU tests can drive exactly this
control flow over gloo with a checker standing in for the kernels; on GPUs they are the library's calls.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, List, Optional, Sequence

import numpy as np
import torch

from .workloads import PAGE, Workload


@dataclass
class SplitPlan:
    """Which shard slots of every request a rank sweeps, and where they land in the owner's arrays."""
    world: int
    rank: int
    max_shards: int          # S of the whole request table
    owner: int = 0

    @property
    def per_rank(self) -> int:
        return -(-self.max_shards // self.world)

    @property
    def padded_shards(self) -> int:
        """Shard slots per request of the owner's arrays: world * per_rank (padded slots stay empty)."""
        return self.per_rank * self.world

    def slots(self, rank: Optional[int] = None) -> range:
        """Shard indices [lo, hi) of the request table that ``rank`` owns."""
        r = self.rank if rank is None else rank
        lo = min(self.max_shards, r * self.per_rank)
        return range(lo, min(self.max_shards, lo + self.per_rank))

    @property
    def out_offset(self) -> int:
        return self.rank * self.per_rank


def rank_workload(w: Workload, plan: SplitPlan) -> Workload:
    """The part of ``w`` that ``plan.rank`` holds: only the pages its shards touch, in a pool of its own,
    behind a block table of the same width whose other entries are -1 (never read: no shard of this rank
    reaches them), and a shard table of ``per_rank`` slots padded with empty ranges.  A page on the boundary
    of two ranks' shards (unaligned shards) is held by both."""
    sl = plan.slots()
    B, per = w.batch, plan.per_rank
    ranges = np.zeros((B, per, 2), np.int32)
    ranges[:, :len(sl)] = w.shard_ranges[:, sl.start:sl.stop]
    table = np.full_like(w.block_table, -1)
    keep: List[int] = []
    for b in range(B):
        L = int(w.seq_lens[b])
        need = np.zeros(w.max_pages_per_req, bool)
        for s in range(len(sl)):
            lo, hi = max(0, int(ranges[b, s, 0])), min(L, int(ranges[b, s, 1]))
            if hi > lo:
                need[lo // PAGE:(hi - 1) // PAGE + 1] = True
        lp = np.nonzero(need)[0]
        table[b, lp] = len(keep) + np.arange(len(lp), dtype=np.int32)
        keep.extend(int(x) for x in w.block_table[b, lp])
    if not keep:                      # a rank with nothing to sweep still needs a (one-page) pool to point at
        keep = [int(max(0, w.block_table.max()))]
    idx = np.asarray(keep, np.int64)
    counts = np.clip(w.shard_counts.astype(np.int64) - sl.start, 0, per).astype(np.int32)
    return Workload(f"{w.name}/rank{plan.rank}", B, w.num_q_heads, w.num_kv_heads, w.max_pages_per_req, per,
                    len(idx), w.q, np.ascontiguousarray(w.k_cache[idx]), np.ascontiguousarray(w.v_cache[idx]),
                    table, w.seq_lens, ranges, counts, meta=dict(w.meta, split_rank=plan.rank))


# ---------------------------------------------------------------------------------------------------------
# the owner's arrays in every rank's address space
# ---------------------------------------------------------------------------------------------------------
def share_from_owner(tensors: Optional[Sequence[torch.Tensor]], dist, plan: SplitPlan):
    """CUDA tensors of the owner, opened in every other rank's process through CUDA IPC handles that travel
    over the process group.  Returns the owner's own tensors on the owner and peer-mapped views elsewhere
    (keep them referenced: dropping a view closes the mapping)."""
    from torch.multiprocessing.reductions import reduce_tensor
    payload = [None]
    if plan.rank == plan.owner:
        payload = [[reduce_tensor(t) for t in tensors]]
    dist.broadcast_object_list(payload, src=plan.owner)
    if plan.rank == plan.owner:
        return list(tensors)
    return [fn(*fn_args) for fn, fn_args in payload[0]]


class SplitRequestRunner:
    """The per-step control flow of one rank.  ``sweep(q, o, m, lse)`` runs this rank's sweep into the given
    arrays (the owner's, with this rank's slot offset already in its parameters, or local ones for the gather
    arm); ``merge(o, lse)`` runs on the owner only."""

    def __init__(self, plan: SplitPlan, dist, q: torch.Tensor, sweep: Callable, merge: Callable,
                 owner_arrays: Optional[Sequence[torch.Tensor]] = None,
                 local_arrays: Optional[Sequence[torch.Tensor]] = None, transport: str = "parked"):
        assert transport in ("parked", "gather")
        self.plan, self.dist, self.q, self.sweep, self.merge = plan, dist, q, sweep, merge
        self.transport = transport
        self.owner_arrays, self.local_arrays = owner_arrays, local_arrays
        self._token = torch.zeros(1, dtype=torch.float32, device=q.device)
        if transport == "parked":
            assert owner_arrays is not None and len(owner_arrays) == 3
        else:
            assert local_arrays is not None and len(local_arrays) == 3
        self.exchange_bytes_out = q.numel() * q.element_size()          # per receiving rank
        self.last_gathered = None

    def step(self):
        plan, dist = self.plan, self.dist
        # 1. only the query travels out
        if plan.world > 1:
            dist.broadcast(self.q.view(torch.uint8), src=plan.owner)    # as bytes: every backend moves those
        if self.transport == "parked":
            o, m, lse = self.owner_arrays
            # 2. the sweep's epilogue stores are the transfer
            self.sweep(self.q, o, m, lse)
            # 3. every rank's states are in the owner's memory once every rank's sweep has completed
            if plan.world > 1:
                dist.all_reduce(self._token)
            # 4. the owner merges
            if plan.rank == plan.owner:
                self.merge(o, lse)
        else:
            o, m, lse = self.local_arrays
            self.sweep(self.q, o, m, lse)
            o_all, l_all = gather_states(o, lse, plan, dist)
            self.last_gathered = (o_all, l_all)
            if plan.rank == plan.owner:
                self.merge(o_all, l_all)


def gather_states(o_local: torch.Tensor, lse_local: torch.Tensor, plan: SplitPlan, dist):
    """All ranks' shard states in slot order: o [B, world * per_rank, Hq, D], lse [B, world * per_rank, Hq]."""
    if plan.world == 1:
        return o_local, lse_local
    o_all = [torch.empty_like(o_local) for _ in range(plan.world)]
    l_all = [torch.empty_like(lse_local) for _ in range(plan.world)]
    dist.all_gather(o_all, o_local.contiguous())
    dist.all_gather(l_all, lse_local.contiguous())
    return torch.cat(o_all, dim=1), torch.cat(l_all, dim=1)


# ---------------------------------------------------------------------------------------------------------
# the GPU instantiation: library calls behind the two callables
# ---------------------------------------------------------------------------------------------------------
def cuda_runner(w: Workload, plan: SplitPlan, dist, device, transport: str = "parked", flags: int = 0):
    """Uploads this rank's part of ``w``, allocates (owner) or opens (others) the shard-state arrays and
    returns (runner, out, lse, device_workload); out / lse are the owner's result tensors (None elsewhere)."""
    from . import binding as qf
    from .runtime import DeviceWorkload
    import copy

    wr = rank_workload(w, plan)
    dw = DeviceWorkload(wr, device=device, flags=flags)
    B, Hq, D, St = w.batch, w.num_q_heads, w.head_dim, plan.padded_shards
    is_owner = plan.rank == plan.owner
    out = lse = None
    merge_params = qf.params(B, Hq, w.num_kv_heads, w.max_pages_per_req, St, max(1, wr.num_pages))
    if is_owner:
        out = torch.empty((B, Hq, D), dtype=torch.float32, device=device)
        lse = torch.empty((B, Hq), dtype=torch.float32, device=device)

    def merge(o, l):
        qf.combine(o, l, None, out, lse, merge_params)

    if transport == "parked":
        arrays = None
        if is_owner:
            arrays = [torch.zeros((B, St, Hq, D), dtype=torch.float32, device=device),
                      torch.full((B, St, Hq), float("-inf"), dtype=torch.float32, device=device),
                      torch.full((B, St, Hq), float("-inf"), dtype=torch.float32, device=device)]
        if plan.world > 1:
            arrays = share_from_owner(arrays, dist, plan)
            if not is_owner:
                # this rank's kernels store into the owner's memory: its device must be allowed to
                qf.enable_peer_access(arrays[0].device.index)
        sp = copy.copy(dw.params)
        sp.out_shards, sp.out_shard_offset = St, plan.out_offset

        def sweep(q, o, m, l):
            qf.decode_partial(q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, dw.shard_ranges, o, m, l, sp,
                              dw.workspace, dw.ws_bytes)

        runner = SplitRequestRunner(plan, dist, dw.q, sweep, merge, owner_arrays=arrays, transport="parked")
    else:
        def sweep(q, o, m, l):
            qf.decode_partial(q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, dw.shard_ranges, o, m, l,
                              dw.params, dw.workspace, dw.ws_bytes)

        runner = SplitRequestRunner(plan, dist, dw.q, sweep, merge,
                                    local_arrays=[dw.o_part, dw.m_part, dw.lse_part], transport="gather")
    return runner, out, lse, dw
