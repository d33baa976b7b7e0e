"""Thin ctypes binding over the C ABI in ``include/qf.h``.

Covers ``include/qf.h`` and the test hooks of ``include/qf_testing.h``.
Argument marshalling only: every step of the path runs in the CUDA library.
Functions carry the same names as the C entry points (without the ``qf_``
prefix).  Tensor arguments may be torch tensors (their ``data_ptr()`` is
taken), integers (raw addresses) or ``None`` (NULL).

There is no fallback: if ``libqf.so`` has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libqf.so"

QF_OK = 0
QF_ERR_NULL = -1
QF_ERR_BAD_SHAPE = -2
QF_ERR_UNSUPPORTED = -3
QF_ERR_WORKSPACE = -4
QF_ERR_CUDA = -5
QF_ERR_DEVICE = -6
QF_ERR_STATIC_SCRATCH = -7
QF_STATIC_SCRATCH_BYTES = 8 << 20

QF_FLAG_CHECK_BOUNDS = 1
QF_FLAG_SIMPLE_KERNEL = 2
QF_FLAG_DRAW_ALWAYS = 8
QF_FLAG_KV_NHD = 16
QF_FLAG_NO_SMALL_MERGE = 32

QF_STATUS_BAD_PAGE = 1
QF_STATUS_TIMEOUT = 2

# every symbol include/qf.h declares
EXPORTS = (
    "qf_version", "qf_strerror", "qf_workspace_bytes", "qf_decode_partial", "qf_combine",
    "qf_step_scratch_bytes", "qf_decode_step_host", "qf_read_status", "qf_last_launch_count",
    "qf_set_profile_events", "qf_decode_partial_static", "qf_static_scratch_error",
    "qf_combine_self", "qf_append_kv", "qf_selftest_bounded_wait", "qf_plan_pieces",
    "qf_project_workspace_bytes", "qf_project_pair", "qf_project_status", "qf_fold_append",
    "qf_static_scratch_status", "qf_project_status_inject", "qf_enable_peer_access", "qf_decode_step",
    "qf_host_pipe_scratch_bytes", "qf_host_pipe_create", "qf_host_pipe_submit", "qf_host_pipe_wait",
    "qf_host_pipe_destroy",
)


class QFParams(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("page_size", ctypes.c_int32),
        ("max_pages_per_req", ctypes.c_int32),
        ("max_shards", ctypes.c_int32),
        ("flags", ctypes.c_int32),
        ("num_pages", ctypes.c_int64),
        ("sm_scale", ctypes.c_float),
        ("out_shards", ctypes.c_int32),
        ("out_shard_offset", ctypes.c_int32),
        ("max_seq_len", ctypes.c_int32),
    ]


class QFError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where} failed with status {status}: {strerror(status)}")


_lib = None


def lib() -> ctypes.CDLL:
    """Load libqf.so (built by ``paper_2608_15473_b200.build``).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2608_15473_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, i32p = ctypes.c_void_p, ctypes.c_void_p
        pp = ctypes.POINTER(QFParams)
        L.qf_version.restype = ctypes.c_int
        L.qf_strerror.restype = ctypes.c_char_p
        L.qf_strerror.argtypes = [ctypes.c_int]
        L.qf_workspace_bytes.restype = ctypes.c_size_t
        L.qf_workspace_bytes.argtypes = [pp]
        L.qf_step_scratch_bytes.restype = ctypes.c_size_t
        L.qf_step_scratch_bytes.argtypes = [pp]
        L.qf_decode_partial.restype = ctypes.c_int
        L.qf_decode_partial.argtypes = [vp, vp, vp, i32p, i32p, i32p, vp, vp, vp, pp, vp, ctypes.c_size_t, vp]
        L.qf_decode_step.restype = ctypes.c_int
        L.qf_decode_step.argtypes = [vp, vp, vp, i32p, i32p, i32p, i32p, vp, vp, vp, vp, vp, pp, vp, ctypes.c_size_t, vp]
        L.qf_combine.restype = ctypes.c_int
        L.qf_combine.argtypes = [vp, vp, i32p, vp, vp, pp, vp]
        L.qf_decode_step_host.restype = ctypes.c_int
        L.qf_decode_step_host.argtypes = [vp, vp, vp, i32p, i32p, i32p, i32p, vp, vp, pp, vp, ctypes.c_size_t, vp]
        L.qf_read_status.restype = ctypes.c_int
        L.qf_read_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), vp]
        L.qf_last_launch_count.restype = ctypes.c_int
        L.qf_set_profile_events.restype = ctypes.c_int
        L.qf_set_profile_events.argtypes = [vp, vp]
        L.qf_combine_self.restype = ctypes.c_int
        L.qf_combine_self.argtypes = [vp, vp, i32p, vp, vp, vp, vp, vp, pp, vp]
        L.qf_append_kv.restype = ctypes.c_int
        L.qf_append_kv.argtypes = [vp, vp, i32p, i32p, vp, vp, pp, vp]
        L.qf_selftest_bounded_wait.restype = ctypes.c_int
        L.qf_selftest_bounded_wait.argtypes = [vp, vp]
        L.qf_decode_partial_static.restype = ctypes.c_int
        L.qf_decode_partial_static.argtypes = [vp, vp, vp, i32p, i32p, i32p, vp, vp, vp, pp, vp]
        L.qf_static_scratch_error.restype = ctypes.c_char_p
        L.qf_static_scratch_status.restype = ctypes.c_int
        L.qf_static_scratch_status.argtypes = [ctypes.POINTER(ctypes.c_int32), vp]
        L.qf_host_pipe_scratch_bytes.restype = ctypes.c_size_t
        L.qf_host_pipe_scratch_bytes.argtypes = [pp, ctypes.c_int]
        L.qf_host_pipe_create.restype = ctypes.c_int
        L.qf_host_pipe_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), pp, vp, ctypes.c_size_t, ctypes.c_int]
        L.qf_host_pipe_submit.restype = ctypes.c_longlong
        L.qf_host_pipe_submit.argtypes = [vp, vp, vp, vp, i32p, i32p, i32p, i32p, vp, vp, vp]
        L.qf_host_pipe_wait.restype = ctypes.c_int
        L.qf_host_pipe_wait.argtypes = [vp, ctypes.c_longlong]
        L.qf_host_pipe_destroy.restype = ctypes.c_int
        L.qf_host_pipe_destroy.argtypes = [vp]
        L.qf_enable_peer_access.restype = ctypes.c_int
        L.qf_enable_peer_access.argtypes = [ctypes.c_int]
        L.qf_project_status_inject.restype = ctypes.c_int
        L.qf_project_status_inject.argtypes = [vp, ctypes.c_int32, vp]
        L.qf_fold_append.restype = ctypes.c_int
        L.qf_fold_append.argtypes = [vp, vp, i32p, vp, vp, vp, vp, vp, vp, vp, i32p, i32p, ctypes.c_int, pp, vp]
        L.qf_project_workspace_bytes.restype = ctypes.c_size_t
        L.qf_project_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int]
        L.qf_project_pair.restype = ctypes.c_int
        L.qf_project_pair.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_float, vp, ctypes.c_size_t, vp]
        L.qf_project_status.restype = ctypes.c_int
        L.qf_project_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), vp]
        L.qf_plan_pieces.restype = ctypes.c_int
        L.qf_plan_pieces.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, i32p, i32p, ctypes.c_int]
        _lib = L
    return _lib


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    if hasattr(x, "ctypes"):  # numpy (host buffers of decode_step_host)
        return int(x.ctypes.data)
    raise TypeError(f"cannot take the address of {type(x)}")


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def params(batch: int, num_q_heads: int, num_kv_heads: int, max_pages_per_req: int, max_shards: int,
           num_pages: int, head_dim: int = 128, page_size: int = 16, flags: int = 0,
           sm_scale: float = 0.0, out_shards: int = 0, out_shard_offset: int = 0, max_seq_len: int = 0) -> QFParams:
    return QFParams(batch, num_q_heads, num_kv_heads, head_dim, page_size, max_pages_per_req, max_shards,
                    flags, num_pages, sm_scale, out_shards, out_shard_offset, max_seq_len)


def version() -> int:
    return int(lib().qf_version())


def strerror(status: int) -> str:
    return lib().qf_strerror(int(status)).decode()


def workspace_bytes(p: QFParams) -> int:
    return int(lib().qf_workspace_bytes(ctypes.byref(p)))


def step_scratch_bytes(p: QFParams) -> int:
    return int(lib().qf_step_scratch_bytes(ctypes.byref(p)))


def last_launch_count() -> int:
    return int(lib().qf_last_launch_count())


def set_profile_events(start_event, stop_event) -> None:
    """cudaEvent_t handles (ints) recorded around the sweep kernel; (None, None) switches it off."""
    lib().qf_set_profile_events(start_event, stop_event)


def decode_partial(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part,
                   p: QFParams, workspace, workspace_bytes: int, stream=None, check: bool = True) -> int:
    rc = lib().qf_decode_partial(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table), _ptr(seq_lens),
                                 _ptr(shard_ranges), _ptr(o_part), _ptr(m_part), _ptr(lse_part),
                                 ctypes.byref(p), _ptr(workspace), int(workspace_bytes), _stream(stream))
    if check and rc != QF_OK:
        raise QFError(rc, "qf_decode_partial")
    return rc


def decode_partial_static(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part,
                          p: QFParams, stream=None, check: bool = True) -> int:
    """The sweep with the library's built-in scratch array: for callers that cannot allocate."""
    rc = lib().qf_decode_partial_static(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                        _ptr(seq_lens), _ptr(shard_ranges), _ptr(o_part), _ptr(m_part),
                                        _ptr(lse_part), ctypes.byref(p), _stream(stream))
    if check and rc != QF_OK:
        detail = lib().qf_static_scratch_error().decode()
        raise QFError(rc, "qf_decode_partial_static" + (f" ({detail})" if detail else ""))
    return rc


def decode_step(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, shard_counts, o_part, m_part, lse_part,
                out, lse, p: QFParams, workspace, workspace_bytes: int, stream=None, check: bool = True) -> int:
    """Sweep and merge as one call (a small sweep is followed by one merging kernel instead of two)."""
    rc = lib().qf_decode_step(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table), _ptr(seq_lens),
                              _ptr(shard_ranges), _ptr(shard_counts), _ptr(o_part), _ptr(m_part), _ptr(lse_part),
                              _ptr(out), _ptr(lse), ctypes.byref(p), _ptr(workspace), int(workspace_bytes),
                              _stream(stream))
    if check and rc != QF_OK:
        raise QFError(rc, "qf_decode_step")
    return rc


def static_scratch_status(stream=None) -> int:
    """Status bits of the last decode_partial_static on the current device (synchronises the stream)."""
    st = ctypes.c_int32(0)
    rc = lib().qf_static_scratch_status(ctypes.byref(st), _stream(stream))
    if rc != QF_OK:
        raise QFError(rc, "qf_static_scratch_status")
    return int(st.value)


def enable_peer_access(peer_device: int, check: bool = True) -> int:
    """Let the current device's kernels store into memory of ``peer_device`` (shard states left in the merging
    GPU's arrays)."""
    rc = lib().qf_enable_peer_access(int(peer_device))
    if check and rc != QF_OK:
        raise QFError(rc, "qf_enable_peer_access")
    return rc


def project_status_inject(workspace, bits: int, stream=None) -> None:
    """Test hook: OR status bits into the projection pair's status word as a timed-out kernel would."""
    rc = lib().qf_project_status_inject(_ptr(workspace), int(bits), _stream(stream))
    if rc != QF_OK:
        raise QFError(rc, "qf_project_status_inject")


def combine(o_part, lse_part, shard_counts, out, lse, p: QFParams, stream=None, check: bool = True) -> int:
    rc = lib().qf_combine(_ptr(o_part), _ptr(lse_part), _ptr(shard_counts), _ptr(out), _ptr(lse),
                          ctypes.byref(p), _stream(stream))
    if check and rc != QF_OK:
        raise QFError(rc, "qf_combine")
    return rc


def combine_self(o_part, lse_part, shard_counts, q, k_new, v_new, out, lse, p: QFParams, stream=None,
                 check: bool = True) -> int:
    """Shard merge with the current token (k_new, v_new) folded in."""
    rc = lib().qf_combine_self(_ptr(o_part), _ptr(lse_part), _ptr(shard_counts), _ptr(q), _ptr(k_new),
                               _ptr(v_new), _ptr(out), _ptr(lse), ctypes.byref(p), _stream(stream))
    if check and rc != QF_OK:
        raise QFError(rc, "qf_combine_self")
    return rc


def append_kv(k_cache, v_cache, block_table, seq_lens, k_new, v_new, p: QFParams, stream=None,
              check: bool = True) -> int:
    """Write the current token's key and value at position seq_lens[b] of every request."""
    rc = lib().qf_append_kv(_ptr(k_cache), _ptr(v_cache), _ptr(block_table), _ptr(seq_lens), _ptr(k_new),
                            _ptr(v_new), ctypes.byref(p), _stream(stream))
    if check and rc != QF_OK:
        raise QFError(rc, "qf_append_kv")
    return rc


def fold_append(o_part, lse_part, shard_counts, q, k_new, v_new, out, lse, k_cache, v_cache, block_table, seq_lens,
                p: QFParams, advance_lengths: bool = True, stream=None, check: bool = True) -> int:
    """combine_self and append_kv in one launch; advance_lengths also adds one to the stored requests' lengths."""
    rc = lib().qf_fold_append(_ptr(o_part), _ptr(lse_part), _ptr(shard_counts), _ptr(q), _ptr(k_new), _ptr(v_new),
                              _ptr(out), _ptr(lse), _ptr(k_cache), _ptr(v_cache), _ptr(block_table), _ptr(seq_lens),
                              1 if advance_lengths else 0, ctypes.byref(p), _stream(stream))
    if check and rc != QF_OK:
        raise QFError(rc, "qf_fold_append")
    return rc


def decode_step_host(q_host, k_cache, v_cache, block_table, seq_lens_host, shard_ranges_host,
                     shard_counts_host, out_host, lse_host, p: QFParams, dev_scratch, dev_scratch_bytes: int,
                     stream=None, check: bool = True) -> int:
    rc = lib().qf_decode_step_host(_ptr(q_host), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                   _ptr(seq_lens_host), _ptr(shard_ranges_host), _ptr(shard_counts_host),
                                   _ptr(out_host), _ptr(lse_host), ctypes.byref(p), _ptr(dev_scratch),
                                   int(dev_scratch_bytes), _stream(stream))
    if check and rc != QF_OK:
        raise QFError(rc, "qf_decode_step_host")
    return rc


def host_pipe_scratch_bytes(p: QFParams, depth: int) -> int:
    return int(lib().qf_host_pipe_scratch_bytes(ctypes.byref(p), int(depth)))


def host_pipe_create(p: QFParams, dev_scratch, dev_scratch_bytes: int, depth: int) -> int:
    """A pipelined host-buffer stepper; returns its handle (an integer address)."""
    h = ctypes.c_void_p(None)
    rc = lib().qf_host_pipe_create(ctypes.byref(h), ctypes.byref(p), _ptr(dev_scratch), int(dev_scratch_bytes), int(depth))
    if rc != QF_OK:
        raise QFError(rc, "qf_host_pipe_create")
    return int(h.value)


def host_pipe_submit(pipe: int, q_host, k_cache, v_cache, block_table, seq_lens_host, shard_ranges_host,
                     shard_counts_host, out_host, lse_host, stream=None) -> int:
    """Enqueue one step; returns its ticket."""
    t = lib().qf_host_pipe_submit(pipe, _ptr(q_host), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                  _ptr(seq_lens_host), _ptr(shard_ranges_host), _ptr(shard_counts_host),
                                  _ptr(out_host), _ptr(lse_host), _stream(stream))
    if t < 0:
        raise QFError(int(t), "qf_host_pipe_submit")
    return int(t)


def host_pipe_wait(pipe: int, ticket: int) -> None:
    rc = lib().qf_host_pipe_wait(pipe, int(ticket))
    if rc != QF_OK:
        raise QFError(rc, "qf_host_pipe_wait")


def host_pipe_destroy(pipe: int) -> None:
    lib().qf_host_pipe_destroy(pipe)


def selftest_bounded_wait(workspace, stream=None) -> None:
    """Enqueue the kernel whose wait can never be satisfied; read_status must then report a timeout."""
    rc = lib().qf_selftest_bounded_wait(_ptr(workspace), _stream(stream))
    if rc != QF_OK:
        raise QFError(rc, "qf_selftest_bounded_wait")


def project_workspace_bytes(batch: int, d_model: int, n_q: int) -> int:
    return int(lib().qf_project_workspace_bytes(int(batch), int(d_model), int(n_q)))


def project_pair(a, z, w_o, g, w_q, u_out, q_out, eps, workspace, stream=None, check=True) -> int:
    """u' = z + W_o a, q = W_q N_1(u') for a batch of co-resident requests (device tensors; marshalling only)."""
    batch, n_q = int(a.shape[0]), int(a.shape[1])
    d_model = int(z.shape[1])
    rc = lib().qf_project_pair(_ptr(a), _ptr(z), _ptr(w_o), _ptr(g), _ptr(w_q), _ptr(u_out), _ptr(q_out), batch,
                               d_model, n_q, float(eps), _ptr(workspace),
                               int(workspace.numel() * workspace.element_size()), _stream(stream))
    if check and rc != QF_OK:
        raise QFError(rc, "qf_project_pair")
    return rc


def project_status(workspace, stream=None) -> int:
    st = ctypes.c_int32(0)
    rc = lib().qf_project_status(_ptr(workspace), ctypes.byref(st), _stream(stream))
    if rc != QF_OK:
        raise QFError(rc, "qf_project_status")
    return int(st.value)


def plan_pieces(total_units: int, n_ctas: int, draw_always: bool = False):
    """The sweep's schedule for (total_units, n_ctas): a list of [begin, end) ranges, one per piece
    (static slices first, then the drawn chunks).  Host arithmetic only: no GPU is touched."""
    cap = n_ctas + 4096
    b = (ctypes.c_int32 * cap)()
    e = (ctypes.c_int32 * cap)()
    n = lib().qf_plan_pieces(int(total_units), int(n_ctas), int(bool(draw_always)), b, e, cap)
    if n < 0:
        raise QFError(n, "qf_plan_pieces")
    return [(int(b[i]), int(e[i])) for i in range(n)]


def read_status(workspace, stream=None) -> int:
    st = ctypes.c_int32(0)
    rc = lib().qf_read_status(_ptr(workspace), ctypes.byref(st), _stream(stream))
    if rc != QF_OK:
        raise QFError(rc, "qf_read_status")
    return int(st.value)
