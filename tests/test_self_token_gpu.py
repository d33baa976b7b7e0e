"""GPU parity of the decode step's finish (Section 2): the current token folded into the swept
state (qf_combine_self) and the cache write (qf_append_kv), against the fp64 CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import qf_oracle as orc
from paper_2608_15473_b200 import binding as qf
from paper_2608_15473_b200 import build as qf_build
from paper_2608_15473_b200 import workloads as wl
from paper_2608_15473_b200.runtime import DeviceWorkload

import qf_testlib as T

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    qf_build.build()


def new_token(w, seed, k_scale=1.0):
    rng = np.random.default_rng(seed)
    k = wl.f32_to_bf16_bits((rng.standard_normal((w.batch, w.num_kv_heads, 128)) * k_scale).astype(np.float32))
    v = wl.f32_to_bf16_bits(rng.standard_normal((w.batch, w.num_kv_heads, 128)).astype(np.float32))
    return k, v


def dev_bf16(a):
    return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda()


@pytest.mark.parametrize("G,Hkv", [(2, 8), (4, 8), (1, 2), (8, 2)])
def test_fold_matches_oracle_and_full_attention(G, Hkv):
    lens = [0, 1, 15, 16, 17, 700, 2500]
    ranges = [wl.fixed_shards(L, 600) if L else [(0, 0)] for L in lens]
    w = wl.make_workload("self", lens, ranges, Hkv * G, Hkv, seed=61 + G, max_pages_per_req=200)
    k_new, v_new = new_token(w, 7)
    dw = DeviceWorkload(w)
    dw.sweep()
    out = torch.full_like(dw.out, float("nan"))
    lse = torch.full_like(dw.lse, float("nan"))
    qf.combine_self(dw.o_part, dw.lse_part, dw.shard_counts, dw.q, dev_bf16(k_new), dev_bf16(v_new), out, lse,
                    dw.params)
    torch.cuda.synchronize()
    sh = T.oracle_shape(w)
    o_prev, lse_prev = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
    ref_out, ref_lse, _ = orc.self_fold(o_prev, lse_prev, w.q, k_new, v_new, sh)
    assert T.out_err(out.cpu().numpy(), ref_out) <= T.ENG_OUT
    assert T.lse_err(lse.cpu().numpy(), ref_lse) <= T.ENG_LSE
    # empty cache: the step returns the new value row and its own score
    got = out.cpu().numpy()
    v0 = wl.bf16_bits_to_f64(v_new[0]).repeat(G, axis=0)
    assert np.array_equal(got[0].astype(np.float64), v0)


def test_fold_sign_cases_and_large_magnitudes():
    # new scores far above and far below the cached log-sum-exp, and both near 100
    w = wl.make_workload("sign", [1, 1, 64], [[(0, 1)], [(0, 1)], [(0, 64)]], 8, 8, seed=67)
    for b in range(3):
        w.q[b, :] = w.q[b, 0]
    qv = wl.bf16_bits_to_f32(w.q[:, 0])                       # [3, 128]
    k_new = np.zeros((3, 8, 128), np.uint16)
    k_new[0] = wl.f32_to_bf16_bits(qv[0])                     # s_jj = |q|^2/sqrt(d): far above lse of one token
    k_new[1] = wl.f32_to_bf16_bits(-qv[1])                    # far below
    scale = 100.0 * np.sqrt(128.0) / float(qv[2].astype(np.float64) @ qv[2].astype(np.float64))
    k_new[2] = wl.f32_to_bf16_bits((qv[2] * np.float32(scale)))   # s_jj near 100
    for i in range(64):                                       # and every cached key near 100 too
        w.k_cache[w.block_table[2, i // 16], :, i % 16] = k_new[2, 0]
    v_new = wl.f32_to_bf16_bits(np.full((3, 8, 128), 3.0, np.float32))
    dw = DeviceWorkload(w)
    dw.sweep()
    out = torch.empty_like(dw.out)
    lse = torch.empty_like(dw.lse)
    qf.combine_self(dw.o_part, dw.lse_part, dw.shard_counts, dw.q, dev_bf16(k_new), dev_bf16(v_new), out, lse,
                    dw.params)
    torch.cuda.synchronize()
    sh = T.oracle_shape(w)
    o_prev, lse_prev = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
    ref_out, ref_lse, s_self = orc.self_fold(o_prev, lse_prev, w.q, k_new, v_new, sh)
    assert (s_self[0] - lse_prev[0] > 5).all() and (s_self[1] - lse_prev[1] < -5).all()
    assert (np.abs(s_self[2] - 100) < 1).all() and (lse_prev[2] > 100).all()
    assert T.out_err(out.cpu().numpy(), ref_out) <= T.ENG_OUT
    assert T.lse_err(lse.cpu().numpy(), ref_lse) <= T.ENG_LSE


def test_append_then_sweep_equals_fold():
    # writing the token into the cache and sweeping L+1 positions gives what the fold gave
    lens = [0, 15, 16, 300]
    w = wl.make_workload("app", lens, [[(0, L + 1)] for L in lens], 16, 8, seed=71, max_pages_per_req=24,
                         pool_factor=2.0)
    # give every request the page its next position needs
    free = [p for p in range(w.num_pages) if p not in set(w.block_table[w.block_table >= 0].tolist())]
    for b, L in enumerate(lens):
        if w.block_table[b, L // 16] < 0:
            w.block_table[b, L // 16] = free.pop()
    k_new, v_new = new_token(w, 9)
    dw = DeviceWorkload(w)
    k_before = dw.k_cache.clone()
    qf.append_kv(dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, dev_bf16(k_new), dev_bf16(v_new), dw.params)
    torch.cuda.synchronize()
    # bit-exact placement, nothing else touched
    kc = dw.k_cache.view(torch.int16).cpu().numpy().view(np.uint16)
    vc = dw.v_cache.view(torch.int16).cpu().numpy().view(np.uint16)
    exp_k, exp_v = w.k_cache.copy(), w.v_cache.copy()
    for b, L in enumerate(lens):
        exp_k[w.block_table[b, L // 16], :, L % 16] = k_new[b]
        exp_v[w.block_table[b, L // 16], :, L % 16] = v_new[b]
    assert np.array_equal(kc, exp_k) and np.array_equal(vc, exp_v)
    assert int((k_before.view(torch.int16) != dw.k_cache.view(torch.int16)).sum()) <= len(lens) * 8 * 128
    # sweep over L+1 positions (host advances seq_lens) vs fold over L positions
    dw.seq_lens += 1
    dw.step()
    torch.cuda.synchronize()
    sh = T.oracle_shape(w)
    o_prev, lse_prev = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
    ref_out, ref_lse, _ = orc.self_fold(o_prev, lse_prev, w.q, k_new, v_new, sh)
    assert T.out_err(dw.out.cpu().numpy(), ref_out) <= T.ENG_OUT
    assert T.lse_err(dw.lse.cpu().numpy(), ref_lse) <= T.ENG_LSE


def test_append_skips_requests_without_a_page():
    w = wl.make_workload("nopage", [16, 5], [[(0, 16)], [(0, 5)]], 2, 1, seed=73, max_pages_per_req=1)
    k_new, v_new = new_token(w, 11)
    dw = DeviceWorkload(w)
    before_k = dw.k_cache.clone()
    qf.append_kv(dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, dev_bf16(k_new), dev_bf16(v_new), dw.params)
    torch.cuda.synchronize()
    diff = (before_k.view(torch.int16) != dw.k_cache.view(torch.int16))
    # request 0 is full (position 16 needs a second page that does not exist): untouched; request 1 got its row
    p1 = int(w.block_table[1, 0])
    assert int(diff.sum()) == int(diff[p1, :, 5].sum()) and int(diff[p1, :, 5].sum()) > 0


@pytest.mark.parametrize("layout", [0, qf.QF_FLAG_KV_NHD])
@pytest.mark.parametrize("advance", [True, False])
def test_fold_append_in_one_launch_equals_the_two_calls(advance, layout):
    # request 1 is full (its next position needs a page its table row does not have): nothing stored, length kept
    lens = [0, 16, 15, 16, 17, 700, 2500]
    cap = [16, 16, 15, 32, 17, 700, 2500]       # tokens each request has pages for
    w = wl.make_workload("fa", cap, [wl.fixed_shards(c, 600) for c in cap], 32, 8, seed=89, max_pages_per_req=200)
    w.seq_lens = np.asarray(lens, np.int32)
    k_new, v_new = new_token(w, 13)
    dk, dv = dev_bf16(k_new), dev_bf16(v_new)
    a, f = DeviceWorkload(w, flags=layout), DeviceWorkload(w, flags=layout)
    for dw in (a, f):
        dw.seq_lens.copy_(torch.from_numpy(w.seq_lens).cuda())
        dw.sweep()
    qf.combine_self(a.o_part, a.lse_part, a.shard_counts, a.q, dk, dv, a.out, a.lse, a.params)
    qf.append_kv(a.k_cache, a.v_cache, a.block_table, a.seq_lens, dk, dv, a.params)
    qf.fold_append(f.o_part, f.lse_part, f.shard_counts, f.q, dk, dv, f.out, f.lse, f.k_cache, f.v_cache,
                   f.block_table, f.seq_lens, f.params, advance_lengths=advance)
    assert qf.last_launch_count() == 1
    torch.cuda.synchronize()
    for x, y in ((a.out, f.out), (a.lse, f.lse)):
        assert torch.equal(x.view(torch.int32), y.view(torch.int32))
    for x, y in ((a.k_cache, f.k_cache), (a.v_cache, f.v_cache)):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))
    stored = np.array([L // 16 < (c + 15) // 16 for L, c in zip(lens, cap)])
    assert stored.tolist() == [True, False, True, True, True, True, True]
    want = np.asarray(lens) + (stored if advance else 0)
    assert np.array_equal(f.seq_lens.cpu().numpy(), want)
    # and the stored rows are the token's, where they belong
    kc = f.cache_head_major("k")
    for b in np.nonzero(stored)[0]:
        assert np.array_equal(kc[w.block_table[b, lens[b] // 16], :, lens[b] % 16], k_new[b])


@pytest.mark.parametrize("layout", [0, qf.QF_FLAG_KV_NHD])
def test_decode_loop_is_a_fold_over_steps(layout):
    # Twenty decode steps: sweep the cache, fold the current token in, append it, advance.  After every step
    # the result must equal attention over all positions so far plus the current one (the appendix's fold).
    lens0 = [0, 14, 250, 1000]
    steps = 20
    Hq, Hkv = 16, 8
    cap = [L + steps for L in lens0]
    # pages for the final lengths are allocated up front; the sweep only ever sees seq_lens positions
    w = wl.make_workload("loop", cap, [wl.fixed_shards(c, 512) for c in cap], Hq, Hkv, seed=97)
    w.seq_lens = np.asarray(lens0, np.int32)
    rng = np.random.default_rng(97)
    dw = DeviceWorkload(w, flags=layout)
    dw.seq_lens.copy_(torch.from_numpy(w.seq_lens).cuda())
    sh = T.oracle_shape(w)
    out = torch.empty_like(dw.out)
    lse = torch.empty_like(dw.lse)
    for j in range(steps):
        qj = wl.f32_to_bf16_bits(rng.standard_normal(w.q.shape).astype(np.float32))
        kj = wl.f32_to_bf16_bits(rng.standard_normal((w.batch, Hkv, 128)).astype(np.float32))
        vj = wl.f32_to_bf16_bits(rng.standard_normal((w.batch, Hkv, 128)).astype(np.float32))
        dw.q.copy_(dev_bf16(qj))
        dk, dv = dev_bf16(kj), dev_bf16(vj)
        dw.sweep()
        qf.combine_self(dw.o_part, dw.lse_part, dw.shard_counts, dw.q, dk, dv, out, lse, dw.params)
        qf.append_kv(dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, dk, dv, dw.params)
        dw.seq_lens += 1
        torch.cuda.synchronize()
        # host mirror of the cache, then the oracle over the positions including the current one
        for b in range(w.batch):
            L = int(w.seq_lens[b])
            w.k_cache[w.block_table[b, L // 16], :, L % 16] = kj[b]
            w.v_cache[w.block_table[b, L // 16], :, L % 16] = vj[b]
        w.seq_lens = w.seq_lens + 1
        w.q = qj
        ref_out, ref_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
        assert T.out_err(out.cpu().numpy(), ref_out) <= T.ENG_OUT, j
        assert T.lse_err(lse.cpu().numpy(), ref_lse) <= T.ENG_LSE, j
    # the device cache equals the host mirror bit for bit
    assert np.array_equal(dw.cache_head_major("k"), w.k_cache)
    assert np.array_equal(dw.cache_head_major("v"), w.v_cache)


def test_decode_loop_replayed_from_one_cuda_graph():
    # One decode step (sweep, fold of the current token, cache write, length advance) captured ONCE and replayed:
    # the lengths live on the device and grow between replays, so every replay plans a different sweep inside the
    # kernel; the result of every step must equal attention over all positions so far plus the current one.
    lens0 = [3, 500, 4090, 12_000]
    steps = 12
    Hq, Hkv = 32, 8
    cap = [L + steps for L in lens0]
    w = wl.make_workload("gloop", cap, [wl.fixed_shards(c, 4096) for c in cap], Hq, Hkv, seed=131)
    w.seq_lens = np.asarray(lens0, np.int32)
    rng = np.random.default_rng(131)
    dw = DeviceWorkload(w)
    dw.seq_lens.copy_(torch.from_numpy(w.seq_lens).cuda())
    sh = T.oracle_shape(w)
    out = torch.empty_like(dw.out)
    lse = torch.empty_like(dw.lse)
    k_in = torch.empty((w.batch, Hkv, 128), dtype=torch.bfloat16, device="cuda")
    v_in = torch.empty_like(k_in)

    def one_step(stream):
        dw.sweep(stream)
        qf.combine_self(dw.o_part, dw.lse_part, dw.shard_counts, dw.q, k_in, v_in, out, lse, dw.params, stream)
        qf.append_kv(dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, k_in, v_in, dw.params, stream)
        dw.seq_lens.add_(1)

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        # one un-captured step first (one-time set-up), on throw-away inputs, then restore the state it changed
        k_before, v_before = dw.k_cache.clone(), dw.v_cache.clone()
        k_in.zero_(); v_in.zero_()
        one_step(s)
        torch.cuda.synchronize()
        dw.k_cache.copy_(k_before); dw.v_cache.copy_(v_before)
        dw.seq_lens.copy_(torch.from_numpy(w.seq_lens).cuda())
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            one_step(s)
    # the capture did not run anything: lengths are still the initial ones
    assert np.array_equal(dw.seq_lens.cpu().numpy(), w.seq_lens)
    for j in range(steps):
        qj = wl.f32_to_bf16_bits(rng.standard_normal(w.q.shape).astype(np.float32))
        kj = wl.f32_to_bf16_bits(rng.standard_normal((w.batch, Hkv, 128)).astype(np.float32))
        vj = wl.f32_to_bf16_bits(rng.standard_normal((w.batch, Hkv, 128)).astype(np.float32))
        dw.q.copy_(dev_bf16(qj)); k_in.copy_(dev_bf16(kj)); v_in.copy_(dev_bf16(vj))
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        for b in range(w.batch):
            L = int(w.seq_lens[b])
            w.k_cache[w.block_table[b, L // 16], :, L % 16] = kj[b]
            w.v_cache[w.block_table[b, L // 16], :, L % 16] = vj[b]
        w.seq_lens = w.seq_lens + 1
        w.q = qj
        assert np.array_equal(dw.seq_lens.cpu().numpy(), w.seq_lens)
        ref_out, ref_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
        assert T.out_err(out.cpu().numpy(), ref_out) <= T.ENG_OUT, j
        assert T.lse_err(lse.cpu().numpy(), ref_lse) <= T.ENG_LSE, j
        assert dw.status() == 0
