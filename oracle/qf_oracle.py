"""ctypes loader for the fp64 CPU oracle (``qf_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It imports nothing from
the CUDA package and the CUDA package imports nothing from here.

Arrays cross as NumPy: bf16 tensors as ``uint16`` bit patterns, metadata as
``int32``, results as ``float64``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from pathlib import Path
from typing import Optional

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "qf_oracle.c"
_LIB = _HERE / "libqf_oracle.so"


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no fast-math: summation order is the source's)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall", "-Wextra",
               str(_SRC), "-o", str(tmp), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _Shape(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("page_size", ctypes.c_int32),
        ("max_pages_per_req", ctypes.c_int32),
        ("max_shards", ctypes.c_int32),
        ("sm_scale", ctypes.c_double),
    ]


@dataclass
class Shape:
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int = 128
    page_size: int = 16
    max_pages_per_req: int = 0
    max_shards: int = 1
    sm_scale: float = 0.0  # <= 0: 1/sqrt(head_dim)

    def c(self) -> _Shape:
        return _Shape(self.batch, self.num_q_heads, self.num_kv_heads, self.head_dim, self.page_size,
                      self.max_pages_per_req, self.max_shards, float(self.sm_scale))


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.qfo_num_threads.restype = ctypes.c_int
        _lib.qfo_set_num_threads.argtypes = [ctypes.c_int]
        _lib.qfo_attend_range.restype = None
    return _lib


def num_threads() -> int:
    return int(lib().qfo_num_threads())


def set_num_threads(n: int) -> None:
    lib().qfo_set_num_threads(int(n))


def _p(a: Optional[np.ndarray], dtype) -> ctypes.c_void_p:
    if a is None:
        return ctypes.c_void_p(None)
    assert a.dtype == dtype, (a.dtype, dtype)
    assert a.flags["C_CONTIGUOUS"]
    return ctypes.c_void_p(a.ctypes.data)


def attend_range(q, k_cache, v_cache, block_table, sh: Shape, b: int, h: int, beg: int, end: int,
                 want_scores: bool = False):
    """One head over tokens [beg, end) of request b (already clamped by the caller).

    Returns dict(o, m, lse, w_rel[, scores]).
    """
    D = sh.head_dim
    o = np.zeros(D, np.float64)
    w = np.zeros(D, np.float64)
    m = ctypes.c_double(0.0)
    lse = ctypes.c_double(0.0)
    n = max(0, end - beg)
    scores = np.zeros(max(n, 1), np.float64) if want_scores else None
    shc = sh.c()
    lib().qfo_attend_range(_p(q, np.uint16), _p(k_cache, np.uint16), _p(v_cache, np.uint16),
                           _p(block_table, np.int32), ctypes.byref(shc),
                           ctypes.c_int(b), ctypes.c_int(h), ctypes.c_int64(beg), ctypes.c_int64(end),
                           _p(o, np.float64), ctypes.byref(m), ctypes.byref(lse), _p(w, np.float64),
                           _p(scores, np.float64))
    res = dict(o=o, m=m.value, lse=lse.value, w_rel=w)
    if want_scores:
        res["scores"] = scores[:n]
    return res


def decode_partial(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, sh: Shape):
    """All shard states: o_part [B,S,Hq,D], m_part, lse_part [B,S,Hq] (float64)."""
    B, S, H, D = sh.batch, sh.max_shards, sh.num_q_heads, sh.head_dim
    o = np.zeros((B, S, H, D), np.float64)
    m = np.zeros((B, S, H), np.float64)
    l = np.zeros((B, S, H), np.float64)
    shc = sh.c()
    rc = lib().qfo_decode_partial(_p(q, np.uint16), _p(k_cache, np.uint16), _p(v_cache, np.uint16),
                                  _p(block_table, np.int32), _p(seq_lens, np.int32),
                                  _p(shard_ranges, np.int32), ctypes.byref(shc),
                                  _p(o, np.float64), _p(m, np.float64), _p(l, np.float64))
    assert rc == 0
    return o, m, l


def decode_partial_pick(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, sh: Shape, pick):
    """Shard states of the listed (b, s, h) triples only: o [n,D], m [n], lse [n]."""
    pick = np.ascontiguousarray(np.asarray(pick, np.int32).reshape(-1, 3))
    n = pick.shape[0]
    o = np.zeros((n, sh.head_dim), np.float64)
    m = np.zeros(n, np.float64)
    l = np.zeros(n, np.float64)
    shc = sh.c()
    rc = lib().qfo_decode_partial_pick(_p(q, np.uint16), _p(k_cache, np.uint16), _p(v_cache, np.uint16),
                                       _p(block_table, np.int32), _p(seq_lens, np.int32),
                                       _p(shard_ranges, np.int32), ctypes.byref(shc),
                                       _p(pick, np.int32), ctypes.c_int64(n),
                                       _p(o, np.float64), _p(m, np.float64), _p(l, np.float64))
    assert rc == 0
    return o, m, l


def decode_full(q, k_cache, v_cache, block_table, seq_lens, sh: Shape, pick=None):
    """Unsharded result over [0, seq_lens[b]).

    pick=None: out [B,Hq,D], lse [B,Hq].  Otherwise pick is a list of (b, h)
    pairs and the result is out [n,D], lse [n].
    """
    H, D = sh.num_q_heads, sh.head_dim
    shc = sh.c()
    if pick is None:
        out = np.zeros((sh.batch, H, D), np.float64)
        lse = np.zeros((sh.batch, H), np.float64)
        pk, n = None, 0
    else:
        pk = np.ascontiguousarray(np.asarray(pick, np.int32).reshape(-1, 2))
        n = pk.shape[0]
        out = np.zeros((n, D), np.float64)
        lse = np.zeros(n, np.float64)
    rc = lib().qfo_decode_full(_p(q, np.uint16), _p(k_cache, np.uint16), _p(v_cache, np.uint16),
                               _p(block_table, np.int32), _p(seq_lens, np.int32), ctypes.byref(shc),
                               _p(pk, np.int32), ctypes.c_int64(n), _p(out, np.float64), _p(lse, np.float64))
    assert rc == 0
    return out, lse


def combine(o_part, lse_part, shard_counts, sh: Shape):
    """n-way merge of shard states: out [B,Hq,D], lse [B,Hq]."""
    out = np.zeros((sh.batch, sh.num_q_heads, sh.head_dim), np.float64)
    lse = np.zeros((sh.batch, sh.num_q_heads), np.float64)
    shc = sh.c()
    o_part, lse_part = np.ascontiguousarray(o_part), np.ascontiguousarray(lse_part)  # kept alive over the call
    rc = lib().qfo_combine(_p(o_part, np.float64), _p(lse_part, np.float64),
                           _p(shard_counts, np.int32), ctypes.byref(shc),
                           _p(out, np.float64), _p(lse, np.float64))
    assert rc == 0
    return out, lse


def combine_fold(o_part, lse_part, shard_counts, sh: Shape, perm=None):
    """The pairwise lerp / sigmoid / logaddexp fold, in shard order ``perm``."""
    out = np.zeros((sh.batch, sh.num_q_heads, sh.head_dim), np.float64)
    lse = np.zeros((sh.batch, sh.num_q_heads), np.float64)
    pm = None if perm is None else np.ascontiguousarray(np.asarray(perm, np.int32))
    shc = sh.c()
    o_part, lse_part = np.ascontiguousarray(o_part), np.ascontiguousarray(lse_part)  # kept alive over the call
    rc = lib().qfo_combine_fold(_p(o_part, np.float64), _p(lse_part, np.float64),
                                _p(shard_counts, np.int32), _p(pm, np.int32), ctypes.byref(shc),
                                _p(out, np.float64), _p(lse, np.float64))
    assert rc == 0
    return out, lse


def self_fold(o_prev, lse_prev, q, k_new, v_new, sh: Shape):
    """Fold the current token into the swept state: out [B,Hq,D], lse [B,Hq], s_self [B,Hq]."""
    out = np.zeros((sh.batch, sh.num_q_heads, sh.head_dim), np.float64)
    lse = np.zeros((sh.batch, sh.num_q_heads), np.float64)
    s_self = np.zeros((sh.batch, sh.num_q_heads), np.float64)
    shc = sh.c()
    o_prev, lse_prev = np.ascontiguousarray(o_prev), np.ascontiguousarray(lse_prev)  # kept alive over the call
    rc = lib().qfo_self_fold(_p(o_prev, np.float64), _p(lse_prev, np.float64), _p(q, np.uint16),
                             _p(k_new, np.uint16), _p(v_new, np.uint16), ctypes.byref(shc),
                             _p(out, np.float64), _p(lse, np.float64), _p(s_self, np.float64))
    assert rc == 0
    return out, lse, s_self



def project_pair(a, z, w_o, g, w_q, eps=1e-6, exact=False):
    """The cache side's projection pair (Section 4; the appendix paragraph on batching at the cache side):
    u' = z + W_o a, q = W_q N_1(u') with bf16 roundings of a, u', N_1(u') and q.
    a: float32 [M, n_q]; z: bf16 bits [M, d_model]; w_o: [d_model, n_q]; g: [d_model]; w_q: [n_q, d_model].
    Returns (u bf16 bits, q bf16 bits) and, with exact=True, the fp64 values before the last rounding."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    z, w_o, g, w_q = (np.ascontiguousarray(t, dtype=np.uint16) for t in (z, w_o, g, w_q))
    M, n_q = a.shape
    d_model = z.shape[1]
    assert z.shape == (M, d_model) and w_o.shape == (d_model, n_q) and w_q.shape == (n_q, d_model) and g.shape == (d_model,)
    u = np.empty((M, d_model), np.uint16)
    q = np.empty((M, n_q), np.uint16)
    ue = np.empty((M, d_model), np.float64) if exact else None
    qe = np.empty((M, n_q), np.float64) if exact else None
    f = lib().qfo_project_pair
    f.restype = ctypes.c_int
    vp = ctypes.c_void_p
    f.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp, vp, vp, ctypes.c_double, vp, vp, vp, vp, vp]
    rc = f(M, d_model, n_q, a.ctypes.data, z.ctypes.data, w_o.ctypes.data, g.ctypes.data, float(eps), w_q.ctypes.data,
           u.ctypes.data, q.ctypes.data, ue.ctypes.data if exact else None, qe.ctypes.data if exact else None)
    if rc != 0:
        raise RuntimeError(f"qfo_project_pair failed: {rc}")
    return (u, q, ue, qe) if exact else (u, q)
