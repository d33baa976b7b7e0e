"""Device-memory plumbing around the binding: torch owns buffers and streams,
the CUDA library does all the arithmetic.

``DeviceWorkload`` uploads a host ``Workload`` once and pre-allocates every
output and the scratch, so that ``sweep()`` / ``merge()`` / ``step()`` only
enqueue kernels.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as qf
from .workloads import Workload


def _to_dev(a: np.ndarray, device, dtype=None) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.to(device, non_blocking=False)


class DeviceWorkload:
    """A workload resident in HBM plus its outputs and scratch."""

    def __init__(self, w: Workload, device="cuda:0", flags: int = 0, identity_table_as_null: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU path)")
        self.w = w
        self.device = torch.device(device)
        dev = self.device
        B, Hq, D, S = w.batch, w.num_q_heads, w.head_dim, w.max_shards
        self.params = qf.params(B, Hq, w.num_kv_heads, w.max_pages_per_req, S, w.num_pages, flags=flags)
        self.q = _to_dev(w.q.view(np.int16), dev, torch.bfloat16)
        # the host workload keeps pages head-major [page, Hkv, 16, D]; with QF_FLAG_KV_NHD the device copy is
        # the token-major [page, 16, Hkv, D] arrangement of the same values
        self.kv_nhd = bool(flags & qf.QF_FLAG_KV_NHD)
        order = (0, 2, 1, 3) if self.kv_nhd else (0, 1, 2, 3)
        self.k_cache = _to_dev(w.k_cache.view(np.int16).transpose(order), dev, torch.bfloat16)
        self.v_cache = _to_dev(w.v_cache.view(np.int16).transpose(order), dev, torch.bfloat16)
        self.block_table = None if identity_table_as_null else _to_dev(w.block_table, dev)
        self.seq_lens = _to_dev(w.seq_lens, dev)
        self.shard_ranges = _to_dev(w.shard_ranges, dev)
        self.shard_counts = _to_dev(w.shard_counts, dev)
        self.o_part = torch.empty((B, S, Hq, D), dtype=torch.float32, device=dev)
        self.m_part = torch.empty((B, S, Hq), dtype=torch.float32, device=dev)
        self.lse_part = torch.empty((B, S, Hq), dtype=torch.float32, device=dev)
        self.out = torch.empty((B, Hq, D), dtype=torch.float32, device=dev)
        self.lse = torch.empty((B, Hq), dtype=torch.float32, device=dev)
        self.ws_bytes = qf.workspace_bytes(self.params)
        if self.ws_bytes == 0:
            raise qf.QFError(qf.QF_ERR_UNSUPPORTED, "qf_workspace_bytes")
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        assert self.workspace.data_ptr() % 256 == 0

    def cache_head_major(self, which: str = "k") -> np.ndarray:
        """Host copy (uint16 bit patterns) of a device pool in the host workload's [page, Hkv, 16, D] order."""
        t = self.k_cache if which == "k" else self.v_cache
        a = t.view(torch.int16).cpu().numpy().view(np.uint16)
        return np.ascontiguousarray(a.transpose(0, 2, 1, 3)) if self.kv_nhd else a

    def poison_outputs(self) -> None:
        for t in (self.o_part, self.m_part, self.lse_part, self.out, self.lse):
            t.fill_(float("nan"))

    def sweep(self, stream=None) -> None:
        """qf_decode_partial: shard states into o_part / m_part / lse_part."""
        qf.decode_partial(self.q, self.k_cache, self.v_cache, self.block_table, self.seq_lens,
                          self.shard_ranges, self.o_part, self.m_part, self.lse_part, self.params,
                          self.workspace, self.ws_bytes, stream)

    def merge(self, stream=None) -> None:
        """qf_combine: shard states into out / lse."""
        qf.combine(self.o_part, self.lse_part, self.shard_counts, self.out, self.lse, self.params, stream)

    def step(self, stream=None) -> int:
        """One pass of the whole hot path (qf_decode_step: shard states and the merged result; the sweep, the merge
        of cut units and the merge of shards, the last two as one kernel when the sweep is small); returns the number
        of kernels enqueued."""
        qf.decode_step(self.q, self.k_cache, self.v_cache, self.block_table, self.seq_lens, self.shard_ranges,
                       self.shard_counts, self.o_part, self.m_part, self.lse_part, self.out, self.lse, self.params,
                       self.workspace, self.ws_bytes, stream)
        return qf.last_launch_count()

    def step_two_calls(self, stream=None) -> int:
        """The same pass as two calls, qf_decode_partial then qf_combine."""
        self.sweep(stream)
        n = qf.last_launch_count()
        self.merge(stream)
        return n + qf.last_launch_count()

    def status(self) -> int:
        return qf.read_status(self.workspace)

    def results(self):
        """Host copies (float64) of (o_part, m_part, lse_part, out, lse)."""
        torch.cuda.synchronize(self.device)
        return tuple(t.detach().cpu().numpy().astype(np.float64)
                     for t in (self.o_part, self.m_part, self.lse_part, self.out, self.lse))


class HostStepper:
    """End-to-end stepping from pinned host buffers through qf_decode_step_host."""

    def __init__(self, dw: DeviceWorkload, pinned: bool = True):
        """pinned=True: page-locked (and therefore mapped) host buffers, which the library's kernels read and
        write directly; pinned=False: ordinary pageable buffers, which take the library's copy path."""
        self.dw = dw
        w = dw.w
        pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
        self.q_host = pin(torch.from_numpy(w.q.view(np.int16).copy()))
        self.seq_lens_host = pin(torch.from_numpy(w.seq_lens.copy()))
        self.shard_ranges_host = pin(torch.from_numpy(w.shard_ranges.copy()))
        self.shard_counts_host = pin(torch.from_numpy(w.shard_counts.copy()))
        self.out_host = pin(torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32))
        self.lse_host = pin(torch.empty((w.batch, w.num_q_heads), dtype=torch.float32))
        self.scratch_bytes = qf.step_scratch_bytes(dw.params)
        self.scratch = torch.empty(self.scratch_bytes, dtype=torch.uint8, device=dw.device)
        self.h2d_bytes = (self.q_host.numel() * 2 + self.seq_lens_host.numel() * 4 +
                          self.shard_ranges_host.numel() * 4 + self.shard_counts_host.numel() * 4)
        self.d2h_bytes = self.out_host.numel() * 4 + self.lse_host.numel() * 4

        # raw addresses once: the per-step call then only crosses the C boundary
        import ctypes
        self._fn = qf.lib().qf_decode_step_host
        self._args = [qf._ptr(x) for x in (self.q_host, dw.k_cache, dw.v_cache, dw.block_table, self.seq_lens_host,
                                           self.shard_ranges_host, self.shard_counts_host, self.out_host,
                                           self.lse_host)]
        self._tail = [ctypes.byref(dw.params), qf._ptr(self.scratch), int(self.scratch_bytes)]

    def step(self, stream=None) -> None:
        st = int(torch.cuda.current_stream().cuda_stream) if stream is None else qf._stream(stream)
        rc = self._fn(*self._args, *self._tail, st)
        if rc != qf.QF_OK:
            raise qf.QFError(rc, "qf_decode_step_host")


class HostPipeline:
    """Steps from pinned host buffers with ``depth`` steps in flight (qf_host_pipe_*): a step's query travels in and
    the previous step's result travels out while a sweep runs.  Holds ``depth`` rotating sets of host buffers;
    ``submit`` takes the step's query (bf16 bit patterns, any integer-16 tensor or array of the right size) and
    returns a ticket, ``wait`` returns that step's (out, lse) host tensors, valid until the slot is reused."""

    def __init__(self, dw: DeviceWorkload, depth: int = 2):
        self.dw, self.depth = dw, depth
        w = dw.w
        pin = lambda t: t.pin_memory()
        self.q_host = [pin(torch.from_numpy(w.q.view(np.int16).copy())) for _ in range(depth)]
        self.seq_lens_host = [pin(torch.from_numpy(w.seq_lens.copy())) for _ in range(depth)]
        self.shard_ranges_host = [pin(torch.from_numpy(w.shard_ranges.copy())) for _ in range(depth)]
        self.shard_counts_host = [pin(torch.from_numpy(w.shard_counts.copy())) for _ in range(depth)]
        self.out_host = [pin(torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32)) for _ in range(depth)]
        self.lse_host = [pin(torch.empty((w.batch, w.num_q_heads), dtype=torch.float32)) for _ in range(depth)]
        self.scratch_bytes = qf.host_pipe_scratch_bytes(dw.params, depth)
        self.scratch = torch.empty(self.scratch_bytes, dtype=torch.uint8, device=dw.device)
        self.pipe = qf.host_pipe_create(dw.params, self.scratch, self.scratch_bytes, depth)
        self.h2d_bytes = (self.q_host[0].numel() * 2 + self.seq_lens_host[0].numel() * 4 +
                          self.shard_ranges_host[0].numel() * 4 + self.shard_counts_host[0].numel() * 4)
        self.d2h_bytes = self.out_host[0].numel() * 4 + self.lse_host[0].numel() * 4
        self._next = 0

    def submit(self, q_bits=None, stream=None) -> int:
        """Enqueue one step (with a new query if given: written into the slot's pinned buffer first)."""
        slot = self._next % self.depth
        if self._next >= self.depth:
            qf.host_pipe_wait(self.pipe, self._next - self.depth)     # the slot's host buffers are free again
        if q_bits is not None:
            src = torch.as_tensor(np.ascontiguousarray(q_bits).view(np.int16)) if not torch.is_tensor(q_bits) else q_bits
            self.q_host[slot].copy_(src.view(torch.int16).reshape(self.q_host[slot].shape))
        dw = self.dw
        t = qf.host_pipe_submit(self.pipe, self.q_host[slot], dw.k_cache, dw.v_cache, dw.block_table,
                                self.seq_lens_host[slot], self.shard_ranges_host[slot], self.shard_counts_host[slot],
                                self.out_host[slot], self.lse_host[slot], stream)
        assert t == self._next
        self._next += 1
        return t

    def wait(self, ticket: int):
        qf.host_pipe_wait(self.pipe, ticket)
        slot = ticket % self.depth
        return self.out_host[slot], self.lse_host[slot]

    def close(self) -> None:
        if self.pipe:
            qf.host_pipe_destroy(self.pipe)
            self.pipe = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class CacheSideStack:
    """The cache side of a stack of layers for one batch of co-resident requests (Section 4): per layer its KV
    pool, W_o, W_q and the normalisation gain.  A stage of layer l is what the cache side does per token and layer:

        sweep layer l's cache with the query it already holds        (qf_decode_partial)
        fold in the current token's (k, v), which arrive with z,
        write them into the cache and advance the lengths            (qf_fold_append)
        u' = z + W_o a  ->  the wire;  q = W_q N_1(u')  ->  layer l+1 (qf_project_pair)

    Only enqueues library calls; ``capture`` records a whole token, every layer's stage in order, into one CUDA
    graph whose replays see the lengths grow on the device.
    """

    def __init__(self, layers, w_o: torch.Tensor, w_q: torch.Tensor, gain: torch.Tensor, eps: float = 1e-6):
        self.layers = list(layers)
        L = len(self.layers)
        d0 = self.layers[0]
        self.batch, self.n_q = d0.w.batch, d0.w.num_q_heads * d0.w.head_dim
        self.d_model = int(w_o.shape[1])
        assert tuple(w_o.shape) == (L, self.d_model, self.n_q) and tuple(w_q.shape) == (L, self.n_q, self.d_model)
        assert tuple(gain.shape) == (L, self.d_model)
        for t in (w_o, w_q, gain):
            assert t.dtype == torch.bfloat16 and t.is_contiguous()
        self.w_o, self.w_q, self.gain, self.eps = w_o, w_q, gain, float(eps)
        n = qf.project_workspace_bytes(self.batch, self.d_model, self.n_q)
        if n == 0:
            raise qf.QFError(qf.QF_ERR_UNSUPPORTED, "qf_project_workspace_bytes")
        self.proj_ws = torch.empty(n, dtype=torch.uint8, device=d0.device)
        self.launches_per_token = 0

    def stage(self, l: int, z, k_new, v_new, u_out, stream=None) -> int:
        """Enqueue layer l's stage; the next query lands in layer (l + 1) mod L's q buffer.  Returns launches."""
        dw, nxt = self.layers[l], self.layers[(l + 1) % len(self.layers)]
        dw.sweep(stream)
        n = qf.last_launch_count()
        qf.fold_append(dw.o_part, dw.lse_part, dw.shard_counts, dw.q, k_new, v_new, dw.out, dw.lse, dw.k_cache,
                       dw.v_cache, dw.block_table, dw.seq_lens, dw.params, advance_lengths=True, stream=stream)
        n += qf.last_launch_count()
        qf.project_pair(dw.out.view(self.batch, self.n_q), z, self.w_o[l], self.gain[l], self.w_q[l], u_out,
                        nxt.q.view(self.batch, self.n_q), self.eps, self.proj_ws, stream)
        return n + qf.last_launch_count()

    def token(self, z, k_new, v_new, u_out, stream=None) -> int:
        """One token through every layer: z, k_new, v_new, u_out are [L, ...] stacks, one slice per layer."""
        n = 0
        for l in range(len(self.layers)):
            n += self.stage(l, z[l], k_new[l], v_new[l], u_out[l], stream)
        self.launches_per_token = n
        return n

    def capture(self, z, k_new, v_new, u_out, stream: torch.cuda.Stream) -> torch.cuda.CUDAGraph:
        """One token as a CUDA graph on ``stream``.  Call ``token`` once un-captured before this: the first call
        of a shape sets kernel attributes and builds descriptors."""
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            self.token(z, k_new, v_new, u_out, stream)
        return graph

    def status(self) -> int:
        st = qf.project_status(self.proj_ws)
        for dw in self.layers:
            st |= dw.status()
        return st
