"""Shared helpers for the GPU parity tests: run the CUDA path, run the oracle, compare."""
import numpy as np

from oracle import qf_oracle as orc

# contract (max-abs on outputs; |d| <= tol * max(1, |ref|) on log-sum-exp and running max)
TOL_OUT = 2e-3
TOL_LSE = 1e-5
# what a correct fp32-accumulating kernel is expected to reach; anything worse is a bug to find
ENG_OUT = 5e-5
ENG_LSE = 1e-6


def oracle_shape(w, **kw):
    d = dict(batch=w.batch, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads,
             max_pages_per_req=w.max_pages_per_req, max_shards=w.max_shards)
    d.update(kw)
    return orc.Shape(**d)


def lse_err(got, ref):
    """Relative error with -inf required to match exactly; returns max over finite entries."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    ninf = np.isneginf(ref)
    assert np.array_equal(np.isneginf(got), ninf), "-inf pattern differs"
    fin = ~ninf
    assert np.isfinite(got[fin]).all(), "non-finite log-sum-exp"
    if not fin.any():
        return 0.0
    return float((np.abs(got[fin] - ref[fin]) / np.maximum(1.0, np.abs(ref[fin]))).max())


def out_err(got, ref):
    got = np.asarray(got, np.float64)
    assert np.isfinite(got).all(), "non-finite output"
    return float(np.abs(got - np.asarray(ref, np.float64)).max()) if got.size else 0.0


def covers_context(w):
    """True if every request's counted shards tile [0, L) exactly (so combine == unsharded sweep)."""
    for b in range(w.batch):
        L = int(w.seq_lens[b])
        pos = 0
        for s in range(int(w.shard_counts[b])):
            lo, hi = (int(x) for x in w.shard_ranges[b, s])
            lo, hi = max(0, min(lo, L)), max(0, min(hi, L))
            if hi <= lo:
                continue
            if lo != pos:
                return False
            pos = hi
        if pos != L:
            return False
    return True


def oracle_all(w):
    sh = oracle_shape(w)
    op, mp, lp = orc.decode_partial(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh)
    if covers_context(w):
        out, lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
    else:
        out, lse = orc.combine(op, lp, w.shard_counts, sh)
    return op, mp, lp, out, lse


def compare_all(dw, w, eng=True, tag=""):
    """Element-by-element comparison of every output with the oracle. Returns the error dict."""
    got_op, got_mp, got_lp, got_out, got_lse = dw.results()
    op, mp, lp, out, lse = oracle_all(w)
    errs = dict(o_part=out_err(got_op, op), m_part=lse_err(got_mp, mp), lse_part=lse_err(got_lp, lp),
                out=out_err(got_out, out), lse=lse_err(got_lse, lse))
    assert errs["o_part"] <= TOL_OUT and errs["out"] <= TOL_OUT, (tag, errs)
    assert errs["m_part"] <= TOL_LSE and errs["lse_part"] <= TOL_LSE and errs["lse"] <= TOL_LSE, (tag, errs)
    if eng:
        assert errs["o_part"] <= ENG_OUT and errs["out"] <= ENG_OUT, ("engineering gate", tag, errs)
        assert max(errs["m_part"], errs["lse_part"], errs["lse"]) <= ENG_LSE, ("engineering gate", tag, errs)
    return errs


def compare_sampled(dw, w, n_full=24, n_part=48, seed=0, eng=True, tag=""):
    """Full-size check on sampled outputs the oracle computes one by one."""
    rng = np.random.default_rng(seed)
    sh = oracle_shape(w)
    got_op, got_mp, got_lp, got_out, got_lse = dw.results()
    B, S, Hq = w.batch, w.max_shards, w.num_q_heads
    # shard states: sample among real shards, always include each request's last (ragged) shard of a few
    cand = [(b, s) for b in range(B) for s in range(int(w.shard_counts[b]))]
    idx = rng.choice(len(cand), size=min(n_part, len(cand)), replace=False)
    pick = [(cand[i][0], cand[i][1], int(rng.integers(Hq))) for i in idx]
    op, mp, lp = orc.decode_partial_pick(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens,
                                         w.shard_ranges, sh, pick)
    pk = np.asarray(pick)
    errs = dict(o_part=out_err(got_op[pk[:, 0], pk[:, 1], pk[:, 2]], op),
                m_part=lse_err(got_mp[pk[:, 0], pk[:, 1], pk[:, 2]], mp),
                lse_part=lse_err(got_lp[pk[:, 0], pk[:, 1], pk[:, 2]], lp))
    assert covers_context(w)
    bh = [(int(rng.integers(B)), int(rng.integers(Hq))) for _ in range(n_full)]
    out, lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh, pick=bh)
    bh = np.asarray(bh)
    errs["out"] = out_err(got_out[bh[:, 0], bh[:, 1]], out)
    errs["lse"] = lse_err(got_lse[bh[:, 0], bh[:, 1]], lse)
    # properties that hold at any size: unused shard slots follow the empty convention, outputs finite
    for b in range(B):
        for s in range(int(w.shard_counts[b]), S):
            assert np.isneginf(got_lp[b, s]).all() and np.isneginf(got_mp[b, s]).all() and (got_op[b, s] == 0).all()
    assert np.isfinite(got_out).all() and np.isfinite(got_lse).all()
    assert errs["o_part"] <= TOL_OUT and errs["out"] <= TOL_OUT, (tag, errs)
    assert errs["m_part"] <= TOL_LSE and errs["lse_part"] <= TOL_LSE and errs["lse"] <= TOL_LSE, (tag, errs)
    if eng:
        assert errs["o_part"] <= ENG_OUT and errs["out"] <= ENG_OUT, ("engineering gate", tag, errs)
        assert max(errs["m_part"], errs["lse_part"], errs["lse"]) <= ENG_LSE, ("engineering gate", tag, errs)
    return errs
