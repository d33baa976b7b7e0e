"""Q-First cache-side decode attention for B200 (sm_100a).

Single-token grouped-query decode attention over a paged bf16 KV cache,
returned per KV shard as the mergeable pair (O, log Z) plus the running max,
and the log-sum-exp combine that merges shards into the full-context result.

The arithmetic lives in hand-written CUDA behind a C ABI (``include/qf.h``);
``binding`` marshals arguments and nothing else.  There is no CPU fallback:
using the binding without the built library raises.
"""

__all__ = ["binding", "workloads", "build"]
