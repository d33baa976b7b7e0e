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
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return ({k: float(v) for k, v in zip(keys_t, t.tolist())},
            {k: float(v) for k, v in zip(keys_c, c.tolist())})


def whole_job_throughput(total_bytes: float, max_ms_per_step: float) -> float:
    """GB/s of the whole job: bytes all ranks processed per step over the slowest rank's step time."""
    return total_bytes / (max_ms_per_step * 1e-3) / 1e9
