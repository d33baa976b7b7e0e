"""Pins for the fp64 CPU oracle: closed forms, invariants, library routines,
exact brute force and the values the paper prints.  CPU only.

Each pin is chosen so that a plausible mistake in the oracle (a dropped
term, a wrong sign or index, a transposed operand, a wrong head mapping)
fails at least one of them.
"""
import math
from decimal import Decimal, getcontext
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

from oracle import qf_oracle as orc
from paper_2608_15473_b200 import workloads as wl

GOLDEN = Path(__file__).parent / "golden"


def golden_values():
    vals = {}
    for line in (GOLDEN / "paper_values.txt").read_text().splitlines():
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            vals[k.strip()] = float(v)
    return vals


def shape_of(w, **kw):
    d = dict(batch=w.batch, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads,
             max_pages_per_req=w.max_pages_per_req, max_shards=w.max_shards)
    d.update(kw)
    return orc.Shape(**d)


def full(w):
    return orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, shape_of(w))


def partials(w):
    return orc.decode_partial(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, shape_of(w))


def token_rows(w, pool, b, c):
    """fp64 [L, D] rows of request b, kv head c, gathered through the table (test-side gather)."""
    L = int(w.seq_lens[b])
    i = np.arange(L)
    return wl.bf16_bits_to_f64(pool[w.block_table[b, i // 16], c, i % 16])


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("G", [1, 2, 4])
def test_single_key_returns_its_value(G):
    Hkv = 2
    w = wl.make_workload("one", [1, 1], [[(0, 1)], [(0, 1)]], G * Hkv, Hkv, seed=3)
    out, lse = full(w)
    op, mp, lp = partials(w)
    for b in range(2):
        for h in range(G * Hkv):
            c = h // G
            v = token_rows(w, w.v_cache, b, c)[0]
            k = token_rows(w, w.k_cache, b, c)[0]
            qv = wl.bf16_bits_to_f64(w.q[b, h])
            # exact rational dot product, then one rounding
            dot = sum(Fraction(float(a)) * Fraction(float(bb)) for a, bb in zip(qv, k))
            s = float(dot) / math.sqrt(128.0)
            assert np.array_equal(out[b, h], v)
            assert lse[b, h] == pytest.approx(s, rel=1e-14, abs=1e-14)
            assert mp[b, 0, h] == lp[b, 0, h] == lse[b, h]
            assert np.array_equal(op[b, 0, h], v)


def test_identical_keys_give_mean_of_values():
    n = 37
    w = wl.make_workload("same", [n], [[(0, n)]], 4, 2, seed=5, table="identity")
    # copy token 0's key into every token
    for c in range(2):
        for i in range(n):
            w.k_cache[w.block_table[0, i // 16], c, i % 16] = w.k_cache[w.block_table[0, 0], c, 0]
    out, lse = full(w)
    one = wl.make_workload("same", [n], [[(0, 1)]], 4, 2, seed=5, table="identity")
    one.k_cache[:] = w.k_cache
    one.seq_lens[:] = 1
    _, lse1 = full(one)
    for h in range(4):
        v = token_rows(w, w.v_cache, 0, h // 2)
        assert np.allclose(out[0, h], v.mean(axis=0), rtol=1e-14, atol=1e-15)
        assert lse[0, h] == pytest.approx(lse1[0, h] + math.log(n), rel=1e-14)


def test_constant_values_come_back_unchanged():
    w = wl.make_workload("constv", [200, 77], [[(0, 200)], [(0, 77)]], 8, 2, seed=7)
    w.v_cache[:] = wl.f32_to_bf16_bits(np.float32(-1.375))
    out, _ = full(w)
    assert np.allclose(out, -1.375, rtol=1e-15, atol=0)


def test_all_weights_on_one_token_when_its_logit_dominates():
    # q along e_0, one key with huge k_0: out -> that token's value, lse -> its score
    w = wl.make_workload("dom", [50], [[(0, 50)]], 2, 1, seed=9, table="identity")
    w.q[:] = 0
    w.q[0, :, 0] = wl.f32_to_bf16_bits(np.float32(16.0))
    w.k_cache[w.block_table[0, 33 // 16], 0, 33 % 16, 0] = wl.f32_to_bf16_bits(np.float32(512.0)).item()
    out, lse = full(w)
    v = token_rows(w, w.v_cache, 0, 0)[33]
    assert np.allclose(out[0, 0], v, atol=1e-12)
    assert lse[0, 0] == pytest.approx(16.0 * 512.0 / math.sqrt(128), rel=1e-12)


# ------------------------------------------------------------ brute force
def _exact_attention(qv, K, V, scale_dec):
    """Scores as exact rationals, exponentials in 60-digit decimal arithmetic."""
    getcontext().prec = 60
    s = []
    for k in K:
        dot = sum(Fraction(float(a)) * Fraction(float(b)) for a, b in zip(qv, k))
        s.append(Decimal(dot.numerator) / Decimal(dot.denominator) * scale_dec)
    mx = max(s)
    e = [(x - mx).exp() for x in s]
    z = sum(e)
    out = [sum(ei * Decimal(float(v[d])) for ei, v in zip(e, V)) / z for d in range(len(V[0]))]
    return [float(o) for o in out], float(mx + z.ln()), float(mx)


@pytest.mark.parametrize("G", [2, 4])
def test_brute_force_tiny_every_length(G):
    getcontext().prec = 60
    scale = Decimal(1) / Decimal(128).sqrt()
    lens = list(range(1, 49, 5)) + [16, 17, 32, 48]
    w = wl.make_workload("tiny", lens, [[(0, L)] for L in lens], 2 * G, 2, seed=11)
    out, lse = full(w)
    for b, L in enumerate(lens):
        for h in (0, 2 * G - 1):
            c = h // G
            K = token_rows(w, w.k_cache, b, c)
            V = token_rows(w, w.v_cache, b, c)
            eo, el, _ = _exact_attention(wl.bf16_bits_to_f64(w.q[b, h]), K, V, scale)
            assert np.allclose(out[b, h], eo, rtol=1e-12, atol=1e-14)
            assert lse[b, h] == pytest.approx(el, rel=1e-13, abs=1e-13)


# ------------------------------------------------------- library routines
def test_against_torch_sdpa_fp64_with_expanded_kv():
    import torch
    import torch.nn.functional as F
    lens = [130, 47, 512]
    Hq, Hkv = 8, 2
    G = Hq // Hkv
    w = wl.make_workload("sdpa", lens, [[(0, L)] for L in lens], Hq, Hkv, seed=13)
    out, lse = full(w)
    for b, L in enumerate(lens):
        K = np.stack([token_rows(w, w.k_cache, b, c) for c in range(Hkv)])  # [Hkv, L, D]
        V = np.stack([token_rows(w, w.v_cache, b, c) for c in range(Hkv)])
        Kt = torch.from_numpy(K).repeat_interleave(G, dim=0)[None]          # expand per group
        Vt = torch.from_numpy(V).repeat_interleave(G, dim=0)[None]
        qt = torch.from_numpy(wl.bf16_bits_to_f64(w.q[b]))[None, :, None, :]
        ref = F.scaled_dot_product_attention(qt, Kt, Vt)[0, :, 0].numpy()
        assert np.allclose(out[b], ref, rtol=1e-12, atol=1e-14)


def test_against_scipy_logsumexp_and_softmax():
    from scipy.special import logsumexp, softmax
    w = wl.make_workload("scipy", [301], [[(0, 301)]], 4, 1, seed=17)
    sh = shape_of(w)
    for h in range(4):
        r = orc.attend_range(w.q, w.k_cache, w.v_cache, w.block_table, sh, 0, h, 0, 301, want_scores=True)
        K = token_rows(w, w.k_cache, 0, 0)
        V = token_rows(w, w.v_cache, 0, 0)
        s = K @ wl.bf16_bits_to_f64(w.q[0, h]) / np.sqrt(128.0)
        assert np.allclose(r["scores"], s, rtol=1e-13, atol=1e-13)
        assert r["lse"] == pytest.approx(logsumexp(s), rel=1e-14)
        assert r["m"] == s.max() or r["m"] == pytest.approx(s.max(), rel=1e-15)
        assert np.allclose(r["o"], softmax(s) @ V, rtol=1e-12, atol=1e-15)
        # the accumulator relative to m is recoverable from (o, lse, m)
        assert np.allclose(r["w_rel"], r["o"] * math.exp(r["lse"] - r["m"]), rtol=1e-13)


def test_explicit_sm_scale_is_used():
    w = wl.make_workload("scale", [64], [[(0, 64)]], 2, 1, seed=19)
    a = orc.attend_range(w.q, w.k_cache, w.v_cache, w.block_table, shape_of(w, sm_scale=0.25), 0, 1, 0, 64,
                         want_scores=True)
    b = orc.attend_range(w.q, w.k_cache, w.v_cache, w.block_table, shape_of(w), 0, 1, 0, 64, want_scores=True)
    assert np.allclose(a["scores"], b["scores"] * 0.25 * math.sqrt(128.0), rtol=1e-14)


# --------------------------------------------------------------- invariants
def test_gqa_head_mapping_is_contiguous_groups():
    # heads h and h' of one group with the same query must agree; across groups they differ
    w = wl.make_workload("gqa", [90], [[(0, 90)]], 8, 2, seed=23)
    w.q[0, :] = w.q[0, 0]
    out, lse = full(w)
    for h in range(1, 4):
        assert np.array_equal(out[0, h], out[0, 0]) and lse[0, h] == lse[0, 0]
    for h in range(5, 8):
        assert np.array_equal(out[0, h], out[0, 4])
    assert not np.allclose(out[0, 0], out[0, 4])


def test_paging_invariance():
    lens = [100, 33]
    a = wl.make_workload("pg", lens, [[(0, L)] for L in lens], 4, 2, seed=29, table="identity")
    # same logical data under a shuffled table inside a bigger pool
    rng = np.random.default_rng(0)
    npg = [(L + 15) // 16 for L in lens]
    P = 40
    perm = rng.permutation(P)
    bt = np.full((2, a.max_pages_per_req), -1, np.int32)
    kc = np.full((P, 2, 16, 128), 0x7FC0, np.uint16)
    vc = np.full((P, 2, 16, 128), 0x7FC0, np.uint16)
    pos = 0
    for b in range(2):
        for p in range(npg[b]):
            bt[b, p] = perm[pos]
            kc[perm[pos]] = a.k_cache[a.block_table[b, p]]
            vc[perm[pos]] = a.v_cache[a.block_table[b, p]]
            pos += 1
    o1, l1 = full(a)
    o2, l2 = orc.decode_full(a.q, kc, vc, bt, a.seq_lens, shape_of(a))
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)
    # identity table given as NULL
    o3, l3 = orc.decode_full(a.q, a.k_cache, a.v_cache, None, a.seq_lens, shape_of(a))
    assert np.array_equal(o1, o3) and np.array_equal(l1, l3)


def test_garbage_outside_the_range_is_never_read():
    L = 70
    w = wl.make_workload("nan", [L], [[(5, 40), (40, 70)]], 4, 2, seed=31, pool_factor=2.0,
                         poison_unused=True, poison_tails=True)
    ref, lref = full(w)
    assert np.isfinite(ref).all() and np.isfinite(lref).all()
    op, mp, lp = partials(w)
    assert np.isfinite(op).all() and np.isfinite(lp).all()
    # poisoning tokens outside a shard's range must not change that shard's state
    w2 = wl.make_workload("nan", [L], [[(5, 40), (40, 70)]], 4, 2, seed=31, pool_factor=2.0)
    for i in range(0, 5):
        w2.k_cache[w2.block_table[0, 0], :, i] = 0x7FC0
        w2.v_cache[w2.block_table[0, 0], :, i] = 0x7FC0
    op2, _, lp2 = partials(w2)
    assert np.array_equal(op2[0, 0], op[0, 0]) and np.array_equal(lp2[0, 0], lp[0, 0])


def test_shift_invariance():
    # A constant added to every score leaves out unchanged and raises lse by it.
    # Built exactly in bf16: every head's query is 2*e_0, channel 0 of every key is a
    # multiple of 1/4, and the shift adds 4 to that channel, so each score rises by 8/sqrt(D).
    w = wl.make_workload("shift", [120], [[(0, 120)]], 2, 1, seed=37, table="identity")
    w.q[:] = 0
    w.q[0, :, 0] = wl.f32_to_bf16_bits(np.float32(2.0))
    w.k_cache[..., 0] = wl.f32_to_bf16_bits(np.round(wl.bf16_bits_to_f32(w.k_cache[..., 0]) * 4) / 4)
    out1, lse1 = full(w)
    shifted = wl.bf16_bits_to_f32(w.k_cache[..., 0]) + np.float32(4.0)
    w.k_cache[..., 0] = wl.f32_to_bf16_bits(shifted)
    assert np.array_equal(wl.bf16_bits_to_f32(w.k_cache[..., 0]), shifted)  # the shift is exact in bf16
    out2, lse2 = full(w)
    assert np.allclose(out2, out1, rtol=1e-12, atol=1e-14)
    assert np.allclose(lse2, lse1 + 8.0 / math.sqrt(128.0), rtol=1e-14)
    assert np.abs(out1).max() > 1e-3


def test_value_path_gain_is_the_attention_weight():
    # d out / d v_j = A_j: bump one v_j by delta along one channel
    from scipy.special import softmax
    L, j, ch = 60, 41, 7
    w = wl.make_workload("dv", [L], [[(0, L)]], 2, 1, seed=41, table="identity")
    sh = shape_of(w)
    r0 = orc.attend_range(w.q, w.k_cache, w.v_cache, w.block_table, sh, 0, 1, 0, L, want_scores=True)
    A = softmax(r0["scores"])
    old = wl.bf16_bits_to_f64(w.v_cache[j // 16, 0, j % 16, ch:ch + 1])[0]
    new_bits = wl.f32_to_bf16_bits(np.float32(old + 2.0)).item()
    w.v_cache[j // 16, 0, j % 16, ch] = new_bits
    delta = wl.bf16_bits_to_f64(np.array([new_bits], np.uint16))[0] - old
    r1 = orc.attend_range(w.q, w.k_cache, w.v_cache, w.block_table, sh, 0, 1, 0, L)
    d = r1["o"] - r0["o"]
    assert d[ch] == pytest.approx(A[j] * delta, rel=1e-10)
    d[ch] = 0
    assert np.abs(d).max() < 1e-15
    assert A.sum() == pytest.approx(1.0, rel=1e-14)


# ------------------------------------------------- sharding and the combine
def test_sharded_then_combined_equals_unsharded():
    g = golden_values()
    rng = np.random.default_rng(1)
    worst = 0.0
    for trial in range(int(g["shard_trials"]) // 10):
        L = int(rng.integers(4, 400))
        cuts = np.sort(rng.integers(0, L + 1, size=3))
        rngs = [(0, cuts[0]), (cuts[0], cuts[1]), (cuts[1], cuts[2]), (cuts[2], L)]  # four-way, may be empty
        w = wl.make_workload("split", [L], [rngs], 4, 2, seed=100 + trial)
        ref, lref = full(w)
        op, mp, lp = partials(w)
        out, lse = orc.combine(op, lp, w.shard_counts, shape_of(w))
        worst = max(worst, np.abs(out - ref).max(), np.abs(lse - lref).max())
        # empty shards carry -inf and a zero vector
        for s, (a, b) in enumerate(rngs):
            if a == b:
                assert np.isneginf(lp[0, s]).all() and np.isneginf(mp[0, s]).all() and (op[0, s] == 0).all()
    assert worst < 1e-13            # fp64: far inside the paper's printed agreement
    assert worst < g["shard_err"]


def test_pairwise_fold_equals_nway_in_any_order():
    rng = np.random.default_rng(2)
    L = 333
    rngs = wl.even_shards(L, 6)
    rngs[2] = (rngs[2][0], rngs[2][0])  # one empty shard (tokens dropped on purpose from both sides)
    w = wl.make_workload("fold", [L, L // 2], [rngs, wl.even_shards(L // 2, 6)], 4, 1, seed=43)
    op, mp, lp = partials(w)
    sh = shape_of(w)
    out, lse = orc.combine(op, lp, w.shard_counts, sh)
    for _ in range(5):
        perm = rng.permutation(6)
        fo, fl = orc.combine_fold(op, lp, w.shard_counts, sh, perm)
        assert np.allclose(fo, out, rtol=1e-13, atol=1e-15)
        assert np.allclose(fl, lse, rtol=1e-14)
    # poison the empty shard's vector: it must never be read
    op[0, 2] = np.nan
    o2, l2 = orc.combine(op, lp, w.shard_counts, sh)
    f2, _ = orc.combine_fold(op, lp, w.shard_counts, sh)
    assert np.array_equal(o2, out) and np.isfinite(f2).all()


def _two_shard_state(la, lb, D=128, seed=0):
    rng = np.random.default_rng(seed)
    o = rng.standard_normal((1, 2, 1, D))
    l = np.array([[[la], [lb]]], np.float64)
    return o, l, orc.Shape(batch=1, num_q_heads=1, num_kv_heads=1, max_shards=2)


def test_combine_overflow_cases_and_sign_symmetry():
    g = golden_values()
    a = g["logaddexp_overflow_operand"]  # 100: log(e^a + e^a) overflows in fp32, the stabilised form does not
    o, l, sh = _two_shard_state(a, a)
    out, lse = orc.combine(o, l, None, sh)
    assert lse[0, 0] == pytest.approx(a + math.log(2.0), rel=1e-15)
    assert np.allclose(out[0, 0], 0.5 * (o[0, 0, 0] + o[0, 1, 0]), rtol=1e-14)
    with np.errstate(over="ignore"):
        assert np.isinf(np.log(np.exp(np.float32(a)) + np.exp(np.float32(a))))
    # past the exponential form's NaN threshold (e^x/(e^x+e^y) in fp32) the combine stays exact
    thr = g["exp_form_nan_past"]
    with np.errstate(over="ignore", invalid="ignore"):
        x, y = np.float32(thr + 1), np.float32(thr + 2)
        assert np.isnan(np.exp(x) / (np.exp(x) + np.exp(y)))
    for la, lb in [(85.0, 91.0), (thr + 1, thr + 2), (90.0, -90.0), (-90.0, 90.0), (700.0, 701.0)]:
        o, l, sh = _two_shard_state(la, lb, seed=3)
        out, lse = orc.combine(o, l, None, sh)
        t = 1.0 / (1.0 + math.exp(-(la - lb)))
        assert np.allclose(out[0, 0], (1 - t) * o[0, 1, 0] + t * o[0, 0, 0], rtol=1e-13, atol=1e-300)
        assert lse[0, 0] == pytest.approx(max(la, lb) + math.log1p(math.exp(-abs(la - lb))), rel=1e-15)
        # swapping the operands changes nothing (the sign of the difference is not one-directional)
        o_sw, l_sw = o[:, ::-1].copy(), l[:, ::-1].copy()
        out2, lse2 = orc.combine(o_sw, l_sw, None, sh)
        f2, fl2 = orc.combine_fold(o_sw, l_sw, None, sh)
        assert np.allclose(out2, out, rtol=1e-14) and lse2[0, 0] == pytest.approx(lse[0, 0], rel=1e-15)
        assert np.allclose(f2, out, rtol=1e-13) and fl2[0, 0] == pytest.approx(lse[0, 0], rel=1e-15)


def test_combine_empty_operands():
    o, l, sh = _two_shard_state(3.0, -np.inf)
    o[0, 1] = np.nan
    out, lse = orc.combine(o, l, None, sh)
    assert np.array_equal(out[0, 0], o[0, 0, 0]) and lse[0, 0] == 3.0
    o, l, sh = _two_shard_state(-np.inf, -np.inf)
    o[:] = np.nan
    out, lse = orc.combine(o, l, None, sh)
    assert (out == 0).all() and np.isneginf(lse).all()
    f, fl = orc.combine_fold(o, l, None, sh)
    assert (f == 0).all() and np.isneginf(fl).all()
    # shard_counts smaller than max_shards: the tail slot is ignored even if finite
    o, l, sh = _two_shard_state(1.0, 50.0)
    out, lse = orc.combine(o, l, np.array([1], np.int32), sh)
    assert np.array_equal(out[0, 0], o[0, 0, 0]) and lse[0, 0] == 1.0


def test_planted_logits_near_85_combine_without_overflow():
    g = golden_values()
    # the paper's un-logged shard total: ln(8.2e36) = 85.0
    assert math.log(g["shard_Z"]) == pytest.approx(g["shard_logZ"], abs=0.05)
    # a small version of the one-million-token workload: planted scaled logits near 85
    w = wl.config4(seed=0, ctx=4096, n_shards=4, n_plant=40)
    sh = shape_of(w)
    pos = w.meta["planted"]
    r = orc.attend_range(w.q, w.k_cache, w.v_cache, w.block_table, sh, 0, 5, 0, 4096, want_scores=True)
    assert np.abs(r["scores"][pos] - 85.0).max() < 0.15
    with np.errstate(over="ignore"):
        assert np.isinf(np.exp(r["scores"].astype(np.float32)).sum(dtype=np.float32) * np.float32(10))
    ref, lref = full(w)
    assert np.allclose(lref, 85.0 + math.log(40), atol=0.1)
    op, mp, lp = partials(w)
    out, lse = orc.combine(op, lp, w.shard_counts, sh)
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() < 1e-13 and np.abs(lse - lref).max() < 1e-12
    assert (lp[0, 3] < 12).all() and (lp[0, 0] > 80).all()  # unplanted vs planted shards: a ~75 nat gap


def test_byte_model_matches_the_papers_figures():
    g = golden_values()
    w = wl.make_workload("bytes", [1600], [[(0, 1600)]], 16, 8, seed=0)
    per_tok = 2 * w.num_kv_heads * w.head_dim * 2
    assert per_tok / 1000.0 == pytest.approx(g["kv_kb_per_position_per_layer"], abs=0.05)
    assert per_tok * 28 / 1024 == g["kv_kb_per_token_0p6b"]
    assert per_tok * 36 / 1024 == g["kv_kb_per_token_4b"]
    assert w.algorithmic_bytes() >= 1600 * per_tok
    assert w.algorithmic_bytes() < 1600 * per_tok * 1.02


def test_lse_statistics_of_the_normal_workload():
    # law of large numbers for i.i.d. N(0,1) keys: lse ~ ln L + |q|^2 / (2 D)
    L = 4096
    w = wl.make_workload("stat", [L], [[(0, L)]], 4, 2, seed=47)
    _, lse = full(w)
    qn = (wl.bf16_bits_to_f64(w.q[0]) ** 2).sum(axis=1)
    assert np.abs(lse[0] - (math.log(L) + qn / 256.0)).max() < 0.2


# ------------------------------------------------- the current token's fold (Section 2)
def _with_appended_token(w, k_new, v_new):
    """A copy of the workload whose cache holds one more position per request: (k_new, v_new)."""
    lens = [int(L) + 1 for L in w.seq_lens]
    w2 = wl.make_workload("app", lens, [[(0, L)] for L in lens], w.num_q_heads, w.num_kv_heads, seed=0,
                          table="identity")
    for b, L in enumerate(w.seq_lens):
        for i in range(int(L)):
            w2.k_cache[w2.block_table[b, i // 16], :, i % 16] = w.k_cache[w.block_table[b, i // 16], :, i % 16]
            w2.v_cache[w2.block_table[b, i // 16], :, i % 16] = w.v_cache[w.block_table[b, i // 16], :, i % 16]
        L = int(L)
        w2.k_cache[w2.block_table[b, L // 16], :, L % 16] = k_new[b]
        w2.v_cache[w2.block_table[b, L // 16], :, L % 16] = v_new[b]
    w2.q[:] = w.q
    return w2


def test_self_fold_equals_attention_over_one_more_position():
    lens = [0, 1, 15, 16, 100]
    w = wl.make_workload("fold1", lens, [[(0, L)] for L in lens], 8, 2, seed=51)
    rng = np.random.default_rng(51)
    k_new = wl.f32_to_bf16_bits(rng.standard_normal((len(lens), 2, 128)).astype(np.float32))
    v_new = wl.f32_to_bf16_bits(rng.standard_normal((len(lens), 2, 128)).astype(np.float32))
    sh = shape_of(w)
    o_prev, lse_prev = full(w)
    out, lse, s_self = orc.self_fold(o_prev, lse_prev, w.q, k_new, v_new, sh)
    ref_out, ref_lse = full(_with_appended_token(w, k_new, v_new))
    assert np.allclose(out, ref_out, rtol=1e-12, atol=1e-14)
    assert np.allclose(lse, ref_lse, rtol=1e-13, atol=1e-13)
    # empty cache: the step returns the new value and its own score
    assert np.array_equal(out[0], wl.bf16_bits_to_f64(v_new[0]).repeat(4, axis=0))
    assert np.array_equal(lse[0], s_self[0])


def test_self_fold_sign_is_not_one_directional():
    # at cache length one the new score may exceed the cached log-sum-exp by many nats, or fall far below it
    w = wl.make_workload("fold2", [1, 1], [[(0, 1)], [(0, 1)]], 2, 1, seed=53)
    qv = wl.bf16_bits_to_f32(w.q)
    k_new = np.stack([wl.f32_to_bf16_bits(qv[0, :1] * np.float32(1.0)),      # s_jj = |q|^2/sqrt(d) >> lse_prev
                      wl.f32_to_bf16_bits(qv[1, :1] * np.float32(-1.0))])    # s_jj << lse_prev
    v_new = wl.f32_to_bf16_bits(np.ones((2, 1, 128), np.float32) * np.float32(3.0))
    sh = shape_of(w)
    o_prev, lse_prev = full(w)
    out, lse, s_self = orc.self_fold(o_prev, lse_prev, w.q, k_new, v_new, sh)
    assert s_self[0, 0] - lse_prev[0, 0] > 5 and s_self[1, 0] - lse_prev[1, 0] < -5
    for b in range(2):
        for h in range(2):
            t = 1.0 / (1.0 + math.exp(-(lse_prev[b, h] - s_self[b, h])))
            assert np.allclose(out[b, h], (1 - t) * 3.0 + t * o_prev[b, h], rtol=1e-13)
            assert lse[b, h] == pytest.approx(np.logaddexp(lse_prev[b, h], s_self[b, h]), rel=1e-14)
    assert np.abs(out[0, 0] - 3.0).max() < 0.1             # head 0 attends to what just arrived
    assert np.abs(out[1, 0] - o_prev[1, 0]).max() < 0.1    # head 0 attends to what it already had


def test_self_fold_large_magnitudes():
    # lse_prev = 100 and s_jj = 100: log(e^a + e^b) overflows in fp32, the fold does not
    o_prev = np.zeros((1, 1, 128)); o_prev[0, 0, 0] = 1.0
    lse_prev = np.array([[100.0]])
    q = np.zeros((1, 1, 128), np.uint16); k = np.zeros((1, 1, 128), np.uint16)
    q[0, 0, 0] = wl.f32_to_bf16_bits(np.float32(100.0)).item()
    k[0, 0, 0] = wl.f32_to_bf16_bits(np.float32(math.sqrt(128.0))).item()   # bf16(11.3125): s_jj = 99.99...
    v = wl.f32_to_bf16_bits(np.full((1, 1, 128), 2.0, np.float32))
    sh = orc.Shape(batch=1, num_q_heads=1, num_kv_heads=1)
    out, lse, s_self = orc.self_fold(o_prev, lse_prev, q, k, v, sh)
    assert abs(s_self[0, 0] - 100.0) < 0.05
    assert lse[0, 0] == pytest.approx(np.logaddexp(100.0, s_self[0, 0]), rel=1e-15) and np.isfinite(out).all()
    assert abs(out[0, 0, 1] - 1.0) < 0.02   # about half of v = 2 in the channels where o_prev is 0


# ---------------------------------------------------------------- the "pick" entry points
def _pick_workload():
    # ragged lengths; shards that are clamped at both ends, empty, unaligned, overlapping, past the end;
    # a shuffled table with spare pool pages and NaN in everything that must not be read
    lens = [100, 0, 37, 300, 16, 1, 129]
    ranges = [
        [(0, 7), (7, 7), (7, 33), (33, 100)],
        [(0, 0), (0, 5), (3, 2), (0, 0)],
        [(0, 500), (-5, 10), (36, 37), (40, 50)],
        [(0, 128), (128, 129), (129, 257), (250, 300)],
        [(0, 16), (16, 16), (5, 11), (0, 0)],
        [(0, 1), (1, 1), (0, 0), (-3, 9)],
        [(17, 95), (1, 129), (128, 129), (64, 64)],
    ]
    return wl.make_workload("pick", lens, ranges, 12, 4, seed=71, pool_factor=1.4, poison_unused=True,
                            poison_tails=True, max_pages_per_req=24)


def test_picked_shard_states_equal_the_rows_of_the_full_set():
    # qfo_decode_partial_pick is what the full-size GPU checks compare against: a wrong stride on the
    # (b, s, h) triples, a missed clamp or a wrong output row would show here
    w = _pick_workload()
    sh = shape_of(w)
    op, mp, lp = partials(w)
    rng = np.random.default_rng(5)
    B, S, H = w.batch, w.max_shards, w.num_q_heads
    every = [(b, s, h) for b in range(B) for s in range(S) for h in range(H)]
    order = rng.permutation(len(every))
    pick = [every[i] for i in order] + [every[i] for i in rng.integers(len(every), size=40)]   # shuffled, with repeats
    o, m, l = orc.decode_partial_pick(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh, pick)
    pk = np.asarray(pick)
    assert np.array_equal(o, op[pk[:, 0], pk[:, 1], pk[:, 2]])
    assert np.array_equal(m, mp[pk[:, 0], pk[:, 1], pk[:, 2]], equal_nan=False)
    assert np.array_equal(l, lp[pk[:, 0], pk[:, 1], pk[:, 2]], equal_nan=False)
    # a single triple, and the same triple three times
    one = orc.decode_partial_pick(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh, [(3, 2, 7)])
    assert np.array_equal(one[0][0], op[3, 2, 7]) and one[2][0] == lp[3, 2, 7]
    rep = orc.decode_partial_pick(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh,
                                  [(6, 1, 11)] * 3)
    assert all(np.array_equal(rep[0][i], op[6, 1, 11]) for i in range(3))


def test_picked_shard_states_against_numpy_definition():
    # not only against the oracle's other entry point: a few triples written out with NumPy from the
    # definition (scores through the table, clamped range, softmax, weighted mean of the value rows)
    w = _pick_workload()
    sh = shape_of(w)
    pick = [(0, 2, 5), (2, 0, 0), (3, 3, 11), (6, 0, 9), (2, 1, 4), (5, 3, 2)]
    o, m, l = orc.decode_partial_pick(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh, pick)
    G = w.group
    for i, (b, s, h) in enumerate(pick):
        L = int(w.seq_lens[b])
        lo, hi = (int(x) for x in w.shard_ranges[b, s])
        lo, hi = max(lo, 0), min(hi, L)
        K = token_rows(w, w.k_cache, b, h // G)[lo:hi]
        V = token_rows(w, w.v_cache, b, h // G)[lo:hi]
        sc = K @ wl.bf16_bits_to_f64(w.q[b, h]) / math.sqrt(128.0)
        assert len(sc) > 0
        p = np.exp(sc - sc.max())
        assert m[i] == pytest.approx(sc.max(), rel=1e-14)
        assert l[i] == pytest.approx(sc.max() + math.log(p.sum()), rel=1e-13)
        assert np.allclose(o[i], (p[:, None] * V).sum(0) / p.sum(), rtol=1e-12, atol=1e-14)


def test_picked_unsharded_results_equal_the_rows_of_the_full_set():
    w = _pick_workload()
    sh = shape_of(w)
    out, lse = full(w)
    rng = np.random.default_rng(6)
    B, H = w.batch, w.num_q_heads
    every = [(b, h) for b in range(B) for h in range(H)]
    pick = [every[i] for i in rng.permutation(len(every))] + [every[i] for i in rng.integers(len(every), size=25)]
    o, l = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh, pick=pick)
    pk = np.asarray(pick)
    assert np.array_equal(o, out[pk[:, 0], pk[:, 1]])
    assert np.array_equal(l, lse[pk[:, 0], pk[:, 1]])
    assert np.isneginf(l[pk[:, 0] == 1]).all() and (o[pk[:, 0] == 1] == 0).all()     # the empty request
    one_o, one_l = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh, pick=[(6, 10)])
    assert np.array_equal(one_o[0], out[6, 10]) and one_l[0] == lse[6, 10]
