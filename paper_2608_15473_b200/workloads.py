"""Seeded synthetic inputs for the decode-attention path.

This module only *draws inputs*: tensor shapes, value distributions, block
tables and shard ranges.  It contains none of the attention arithmetic and is
the one module that both the CUDA tests/benchmark and the CPU checker's tests
use, so that both sides see identical bit patterns.

Everything is NumPy on the host.  bf16 tensors are carried as ``uint16`` bit
patterns (round-to-nearest-even from fp32 draws).

Layouts (shared by every consumer):
  q            uint16 [B, Hq, D]
  k_cache,
  v_cache      uint16 [num_pages, Hkv, page_size, D]
  block_table  int32  [B, max_pages_per_req]  logical page -> physical page, -1 = unused
  seq_lens     int32  [B]                      cached positions per request
  shard_ranges int32  [B, S, 2]                half-open token ranges; unused slots are (0, 0)
  shard_counts int32  [B]
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional

import numpy as np

PAGE = 16
HEAD_DIM = 128
_NAN_BF16 = np.uint16(0x7FC0)


# --------------------------------------------------------------------------
# bf16 bit helpers (conversion only; no arithmetic of the method)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even (NaN stays NaN)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        r[nan] = _NAN_BF16
    return r


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def _round_inplace_to_bf16(buf32: np.ndarray, out16: np.ndarray) -> None:
    """RNE-round a scratch fp32 buffer (destroyed) into a uint16 destination."""
    u = buf32.view(np.uint32)
    lsb = u >> np.uint32(16)
    lsb &= np.uint32(1)
    lsb += np.uint32(0x7FFF)
    u += lsb  # no finite N(0,1)-scale draw can carry into the exponent's top
    u >>= np.uint32(16)
    out16[...] = u


# --------------------------------------------------------------------------
# workload container
# --------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    max_pages_per_req: int
    max_shards: int
    num_pages: int
    q: np.ndarray
    k_cache: np.ndarray
    v_cache: np.ndarray
    block_table: np.ndarray
    seq_lens: np.ndarray
    shard_ranges: np.ndarray
    shard_counts: np.ndarray
    head_dim: int = HEAD_DIM
    page_size: int = PAGE
    meta: Dict = field(default_factory=dict)

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def total_tokens(self) -> int:
        return int(self.seq_lens.astype(np.int64).sum())

    def swept_tokens(self) -> int:
        """Tokens inside the (clamped) shard ranges, summed over requests."""
        r = self.shard_ranges.astype(np.int64)
        L = self.seq_lens.astype(np.int64)[:, None]
        beg = np.clip(r[..., 0], 0, L)
        end = np.clip(r[..., 1], 0, L)
        return int(np.maximum(end - beg, 0).sum())

    def algorithmic_bytes(self) -> int:
        """Bytes the method must move for one pass (partials + combine).

        Per swept token 2*Hkv*D*2 bytes of K and V plus 4 bytes of block table
        per page; per request Hq*D*2 bytes of q; per (request, shard, head)
        (D+2)*4 bytes written by the partial step and (D+1)*4 read back by the
        combine; per (request, head) (D+1)*4 bytes of result.
        """
        D, Hq, Hkv = self.head_dim, self.num_q_heads, self.num_kv_heads
        tok = self.swept_tokens()
        n_sh = int(self.shard_counts.astype(np.int64).sum())
        kv = tok * 2 * Hkv * D * 2
        table = 4 * ((tok + self.page_size - 1) // self.page_size)
        qb = self.batch * Hq * D * 2
        part = n_sh * Hq * ((D + 2) * 4 + (D + 1) * 4)
        res = self.batch * Hq * (D + 1) * 4
        return kv + table + qb + part + res


# --------------------------------------------------------------------------
# bulk N(0,1) fill of a paged pool, chunked and threaded
# --------------------------------------------------------------------------
def _n_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def _fill_pool(pool: np.ndarray, seed_seq: np.random.SeedSequence,
               used_pages: Optional[np.ndarray] = None,
               row_scale: Optional[np.ndarray] = None,
               col_scale: Optional[np.ndarray] = None,
               chunk_pages: int = 128) -> None:
    """Fill ``pool`` [P, Hkv, page, D] (uint16) with bf16(N(0,1) * scales).

    used_pages: bool [P]; pages that are False are left untouched.
    row_scale:  float32 [P, page] multiplier per physical token slot (all heads).
    col_scale:  float32 [D] multiplier per channel.
    The stream of chunk c depends only on (seed_seq, c): results do not depend
    on the thread count.
    """
    P, Hkv, page, D = pool.shape
    n_chunks = (P + chunk_pages - 1) // chunk_pages
    children = seed_seq.spawn(n_chunks)

    def work(c: int) -> None:
        lo, hi = c * chunk_pages, min(P, (c + 1) * chunk_pages)
        if used_pages is not None and not used_pages[lo:hi].any():
            return
        gen = np.random.Generator(np.random.SFC64(children[c]))
        buf = gen.standard_normal((hi - lo, Hkv, page, D), dtype=np.float32)
        if row_scale is not None:
            buf *= row_scale[lo:hi, None, :, None]
        if col_scale is not None:
            buf *= col_scale[None, None, None, :]
        if used_pages is None or used_pages[lo:hi].all():
            _round_inplace_to_bf16(buf, pool[lo:hi])
        else:
            tmp = np.empty(buf.shape, np.uint16)
            _round_inplace_to_bf16(buf, tmp)
            sel = used_pages[lo:hi]
            pool[lo:hi][sel] = tmp[sel]

    nt = min(_n_threads(), n_chunks)
    if nt <= 1:
        for c in range(n_chunks):
            work(c)
    else:
        with ThreadPoolExecutor(nt) as ex:
            list(ex.map(work, range(n_chunks)))


def _normal_bf16(shape, seed_seq: np.random.SeedSequence) -> np.ndarray:
    gen = np.random.Generator(np.random.SFC64(seed_seq))
    return f32_to_bf16_bits(gen.standard_normal(shape, dtype=np.float32))


def _pages_for(L: np.ndarray, page: int = PAGE) -> np.ndarray:
    return (L.astype(np.int64) + page - 1) // page


def _build_table(n_pages_req: np.ndarray, phys_order: np.ndarray, max_pages: int) -> np.ndarray:
    """Rows of logical->physical pages; request b takes the next n_b entries of phys_order."""
    B = len(n_pages_req)
    table = np.full((B, max_pages), -1, np.int32)
    pos = 0
    for b in range(B):
        n = int(n_pages_req[b])
        table[b, :n] = phys_order[pos:pos + n]
        pos += n
    return table


def _slot_mask_from_tokens(table: np.ndarray, tokens_per_req: List[np.ndarray], num_pages: int,
                           page: int = PAGE) -> np.ndarray:
    """bool [num_pages, page]: physical slots of the listed logical tokens."""
    mask = np.zeros((num_pages, page), bool)
    for b, toks in enumerate(tokens_per_req):
        if len(toks) == 0:
            continue
        toks = np.asarray(toks, np.int64)
        mask[table[b, toks // page], toks % page] = True
    return mask


# --------------------------------------------------------------------------
# generic small/medium workload for tests
# --------------------------------------------------------------------------
def make_workload(name: str, seq_lens, shard_ranges, num_q_heads: int, num_kv_heads: int, seed: int = 0,
                  table: str = "shuffled", pool_factor: float = 1.0, poison_unused: bool = False,
                  poison_tails: bool = False, k_row_scale_fn: Optional[Callable] = None,
                  k_col_scale: Optional[np.ndarray] = None, max_pages_per_req: Optional[int] = None,
                  shard_counts=None, q_scale: float = 1.0) -> Workload:
    """A paged workload with N(0,1) q, K, V.

    seq_lens:     list of ints.
    shard_ranges: list (per request) of lists of (beg, end).
    table:        "identity" (block_table rows are b*max_pages+p), "shuffled"
                  (random permutation of the pool) .
    pool_factor:  pool size / pages needed (>1 leaves unused pages).
    poison_unused / poison_tails: NaN-fill unused pool pages / the unused tail
                  slots of each request's last page (K and V).
    k_row_scale_fn(rng, b, L) -> int array of logical tokens whose K row is x10.
    """
    ss = np.random.SeedSequence([seed, 0x51F1])
    s_tab, s_q, s_k, s_v, s_misc = ss.spawn(5)
    L = np.asarray(seq_lens, np.int32)
    B = len(L)
    npg = _pages_for(L)
    S = max(1, max(len(r) for r in shard_ranges))
    mp = int(max_pages_per_req if max_pages_per_req is not None else max(1, int(npg.max()) if B else 1))
    needed = int(npg.sum())
    if table == "identity":
        num_pages = B * mp
        bt = np.full((B, mp), -1, np.int32)
        for b in range(B):
            bt[b, :npg[b]] = b * mp + np.arange(npg[b])
    else:
        num_pages = max(1, int(math.ceil(needed * pool_factor)))
        perm = np.random.Generator(np.random.SFC64(s_tab)).permutation(num_pages)
        bt = _build_table(npg, perm.astype(np.int32), mp)
    used = np.zeros(num_pages, bool)
    used[bt[bt >= 0]] = True

    Hkv, Hq = num_kv_heads, num_q_heads
    kc = np.zeros((num_pages, Hkv, PAGE, HEAD_DIM), np.uint16)
    vc = np.zeros((num_pages, Hkv, PAGE, HEAD_DIM), np.uint16)
    row_scale = None
    if k_row_scale_fn is not None:
        rng = np.random.Generator(np.random.SFC64(s_misc))
        toks = [np.asarray(k_row_scale_fn(rng, b, int(L[b])), np.int64) for b in range(B)]
        m = _slot_mask_from_tokens(bt, toks, num_pages)
        row_scale = np.where(m, np.float32(10.0), np.float32(1.0)).astype(np.float32)
    _fill_pool(kc, s_k, None, row_scale, k_col_scale)
    _fill_pool(vc, s_v)
    if poison_unused:
        kc[~used] = _NAN_BF16
        vc[~used] = _NAN_BF16
    if poison_tails:
        for b in range(B):
            r = int(L[b]) % PAGE
            if L[b] > 0 and r:
                p = bt[b, npg[b] - 1]
                kc[p, :, r:, :] = _NAN_BF16
                vc[p, :, r:, :] = _NAN_BF16
    q = _normal_bf16((B, Hq, HEAD_DIM), s_q)
    if q_scale != 1.0:
        q = f32_to_bf16_bits(bf16_bits_to_f32(q) * np.float32(q_scale))

    sr = np.zeros((B, S, 2), np.int32)
    sc = np.zeros(B, np.int32)
    for b in range(B):
        for s, (lo, hi) in enumerate(shard_ranges[b]):
            sr[b, s] = (lo, hi)
        sc[b] = len(shard_ranges[b])
    if shard_counts is not None:
        sc = np.asarray(shard_counts, np.int32)
    return Workload(name, B, Hq, Hkv, mp, S, num_pages, q, kc, vc, bt, L, sr, sc,
                    meta=dict(seed=seed, table=table))


def even_shards(L: int, n: int) -> List[tuple]:
    """n contiguous near-equal token ranges covering [0, L)."""
    cuts = [round(k * L / n) for k in range(n + 1)]
    return [(cuts[k], cuts[k + 1]) for k in range(n)]


def fixed_shards(L: int, size: int) -> List[tuple]:
    """Ranges [k*size, min((k+1)*size, L)) covering [0, L)."""
    n = max(1, (L + size - 1) // size)
    return [(k * size, min((k + 1) * size, L)) for k in range(n)]


# --------------------------------------------------------------------------
# the five benchmark configurations (synthetic stand-ins for Qwen3 layers)
# --------------------------------------------------------------------------
def config1(seed: int = 0) -> Workload:
    """0.6B shape, batch 1, 16q/8kv, context 4,096, one shard, contiguous KV."""
    w = make_workload("cfg1_0p6b_single", [4096], [[(0, 4096)]], 16, 8, seed=seed, table="identity")
    return w


def config2(seed: int = 0, batch: int = 64, ctx: int = 4608, n_shards: int = 4) -> Workload:
    """0.6B shape, batch 64, context 4,608, shuffled table, 4 shards; 4 outlier K channels x8."""
    ss = np.random.SeedSequence([seed, 0xC2])
    ch = np.random.Generator(np.random.SFC64(ss)).choice(HEAD_DIM, size=4, replace=False)
    col = np.ones(HEAD_DIM, np.float32)
    col[ch] = 8.0
    w = make_workload("cfg2_0p6b_batched", [ctx] * batch, [even_shards(ctx, n_shards)] * batch, 16, 8,
                      seed=seed, table="shuffled", k_col_scale=col)
    w.meta["outlier_channels"] = sorted(int(c) for c in ch)
    return w


def config3(seed: int = 0, batch: int = 32, lo: int = 1024, hi: int = 36480, shard: int = 4096) -> Workload:
    """4B shape (32q/8kv), ragged contexts U[lo, hi], shuffled pages, shards of 4,096 tokens."""
    ss = np.random.SeedSequence([seed, 0xC3])
    L = np.random.Generator(np.random.SFC64(ss)).integers(lo, hi + 1, size=batch)
    w = make_workload("cfg3_4b_batched", L.tolist(), [fixed_shards(int(l), shard) for l in L], 32, 8,
                      seed=seed, table="shuffled", max_pages_per_req=(hi + PAGE - 1) // PAGE)
    return w


def config4(seed: int = 0, ctx: int = 1 << 20, n_shards: int = 16, n_plant: int = 400,
            target: float = 85.0, table: str = "identity") -> Workload:
    """1M-token split-KV, 16q/8kv, 16 shards; 400 planted positions with scaled logits near 85.

    The planted positions are shared by all KV heads and drawn from the first
    three quarters of the shards, so the last quarter stays unplanted.  A
    planted key is the minimum-norm correction of its N(0,1) draw n that gives
    every query head of the group the target logit:
    k = n + Qc^T (Qc Qc^T)^-1 (target*sqrt(D)*1 - Qc n), then rounded to bf16.
    """
    shards = even_shards(ctx, n_shards)
    w = make_workload("cfg4_1m_splitkv", [ctx], [shards], 16, 8, seed=seed, table=table)
    ss = np.random.SeedSequence([seed, 0xC4])
    rng = np.random.Generator(np.random.SFC64(ss))
    plant_hi = shards[max(0, (3 * n_shards) // 4 - 1)][1]
    pos = np.sort(rng.choice(plant_hi, size=min(n_plant, plant_hi), replace=False))
    G = w.group
    qf = bf16_bits_to_f64(w.q[0])  # [Hq, D]
    pages = w.block_table[0, pos // PAGE]
    slots = pos % PAGE
    rhs_val = target * math.sqrt(HEAD_DIM)
    for c in range(w.num_kv_heads):
        Qc = qf[c * G:(c + 1) * G]                          # [G, D]
        n = bf16_bits_to_f64(w.k_cache[pages, c, slots])    # [n_plant, D]
        gram_inv = np.linalg.inv(Qc @ Qc.T)
        resid = rhs_val - n @ Qc.T                          # [n_plant, G]
        k = n + (resid @ gram_inv) @ Qc
        w.k_cache[pages, c, slots] = f32_to_bf16_bits(k.astype(np.float32))
    w.meta["planted"] = pos
    w.meta["target_logit"] = target
    return w


def config5(seed: int = 0, batch: int = 256, lo: int = 512, hi: int = 32768, max_shards: int = 8,
            pool_factor: float = 1.5, boost_frac: float = 0.01) -> Workload:
    """4B shape mixed batch: log-uniform contexts, fragmented pool, 1-8 page-aligned shards, 1% keys x10."""
    ss = np.random.SeedSequence([seed, 0xC5])
    rng = np.random.Generator(np.random.SFC64(ss))
    L = np.floor(np.exp(rng.uniform(math.log(lo), math.log(hi), size=batch))).astype(np.int64)
    nsh = rng.integers(1, max_shards + 1, size=batch)
    ranges = []
    for l, n in zip(L, nsh):
        npg = (int(l) + PAGE - 1) // PAGE
        cuts = [min(int(l), PAGE * int(round(k * npg / int(n)))) for k in range(int(n) + 1)]
        cuts[-1] = int(l)
        ranges.append([(cuts[k], cuts[k + 1]) for k in range(int(n))])

    def boost(r, b, Lb):
        return np.nonzero(r.random(Lb) < boost_frac)[0]

    w = make_workload("cfg5_4b_mixed", L.tolist(), ranges, 32, 8, seed=seed, table="shuffled",
                      pool_factor=pool_factor, poison_unused=True, k_row_scale_fn=boost,
                      max_pages_per_req=(hi + PAGE - 1) // PAGE)
    w.max_shards = max_shards
    if w.shard_ranges.shape[1] < max_shards:
        pad = np.zeros((batch, max_shards, 2), np.int32)
        pad[:, :w.shard_ranges.shape[1]] = w.shard_ranges
        w.shard_ranges = pad
    return w


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}


def split_requests(n_requests: int, world_size: int, rank: int) -> range:
    """Contiguous block of request indices owned by ``rank`` (requests are independent)."""
    base, rem = divmod(n_requests, world_size)
    lo = rank * base + min(rank, rem)
    return range(lo, lo + base + (1 if rank < rem else 0))
