"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle, element by
element on the same seeded inputs.  Tolerances: max-abs 2e-3 on outputs, 1e-5 relative on
log-sum-exp (the contract), plus a much tighter engineering gate (see qf_testlib)."""
import numpy as np
import pytest
import torch

from oracle import qf_oracle as orc
from paper_2608_15473_b200 import binding as qf
from paper_2608_15473_b200 import build as qf_build
from paper_2608_15473_b200 import workloads as wl
from paper_2608_15473_b200.runtime import DeviceWorkload, HostPipeline, HostStepper

import qf_testlib as T

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    qf_build.build()
    assert qf.version() == 100


def run(w, flags=0, null_table=False, two_calls=False):
    dw = DeviceWorkload(w, flags=flags, identity_table_as_null=null_table)
    dw.poison_outputs()
    if two_calls:
        dw.step_two_calls()
    else:
        dw.step()
    return dw


# (flags, number of KV heads): the default kernel with 8 and 2 KV heads; the plain-load kernel is the validation aid
# "draw": the unit kernel with its drawn-chunk tail forced on (by default only long sweeps use it)
KERNELS = [pytest.param((0, 16), id="unit16"), pytest.param((0, 8), id="unit8"),
           pytest.param((0, 2), id="unit2"), pytest.param((qf.QF_FLAG_SIMPLE_KERNEL, 2), id="simple"),
           pytest.param((qf.QF_FLAG_DRAW_ALWAYS, 8), id="draw8"), pytest.param((qf.QF_FLAG_DRAW_ALWAYS, 2), id="draw2"),
           # token-major pages (the device copy is rearranged by DeviceWorkload; the oracle sees the same values)
           pytest.param((qf.QF_FLAG_KV_NHD, 8), id="nhd8"), pytest.param((qf.QF_FLAG_KV_NHD, 2), id="nhd2"),
           pytest.param((qf.QF_FLAG_KV_NHD | qf.QF_FLAG_SIMPLE_KERNEL, 2), id="simple-nhd"),
           pytest.param((qf.QF_FLAG_KV_NHD | qf.QF_FLAG_DRAW_ALWAYS, 8), id="draw8-nhd"),
           # a whole step over a small sweep merges with one kernel by default; these keep the finish and merge kernels
           pytest.param((qf.QF_FLAG_NO_SMALL_MERGE, 8), id="nosmall8"), pytest.param((qf.QF_FLAG_NO_SMALL_MERGE, 2), id="nosmall2"),
           pytest.param((qf.QF_FLAG_NO_SMALL_MERGE | qf.QF_FLAG_DRAW_ALWAYS, 8), id="nosmall-draw8")]


# T1: every short length, both group sizes, shuffled table: tail-page masking, first-tile guard
@pytest.mark.parametrize("flags", KERNELS)
@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 6, 7, 8])
def test_every_short_length(G, flags):
    flags, Hkv = flags
    lens = list(range(1, 49))
    w = wl.make_workload("t1", lens, [[(0, L)] for L in lens], Hkv * G, Hkv, seed=G, poison_tails=True,
                         pool_factor=1.3, poison_unused=True)
    dw = run(w, flags)
    T.compare_all(dw, w, tag=f"G={G}")
    assert dw.status() == 0


# T2: degenerate and unaligned shard ranges, clamping, L = 0, shard_counts < S
@pytest.mark.parametrize("flags", KERNELS)
def test_degenerate_shard_ranges(flags):
    flags, Hkv = flags
    lens = [100, 0, 37, 300, 16, 1]
    ranges = [
        [(0, 7), (7, 7), (7, 33), (33, 100)],
        [(0, 0), (0, 5), (3, 2), (0, 0)],              # empty request: every shard empty
        [(0, 500), (-5, 10), (36, 37), (40, 50)],      # clamped at both ends, one fully outside
        [(0, 128), (128, 129), (129, 257), (257, 300)],
        [(0, 16), (16, 16), (0, 0), (0, 0)],
        [(0, 1), (1, 1), (0, 0), (0, 0)],
    ]
    counts = [4, 4, 4, 4, 2, 1]
    w = wl.make_workload("t2", lens, ranges, 4 * Hkv, Hkv, seed=5, poison_tails=True, shard_counts=counts,
                         max_pages_per_req=40)
    dw = run(w, flags)
    T.compare_all(dw, w)
    got_op, got_mp, got_lp, got_out, got_lse = dw.results()
    assert (got_out[1] == 0).all() and np.isneginf(got_lse[1]).all()     # L = 0
    assert np.isneginf(got_lp[0, 1]).all() and (got_op[0, 1] == 0).all()  # [7,7)
    assert np.isneginf(got_lp[2, 3]).all()                                # range past the end


# T3: a dominant token (logit ~ +22 over the rest) planted at structure boundaries
@pytest.mark.parametrize("flags", KERNELS)
@pytest.mark.parametrize("G", [2, 4])
def test_planted_dominant_token(G, flags):
    flags, Hkv = flags
    L = 1500
    shards = [(0, 130), (130, 641), (641, 1024), (1024, 1500)]
    spots = [0, L - 1, 15, 16, 17, 127, 128, 129, 130, 255, 256, 640, 641, 1023, 1024, 1039, 1040, 1279, 1280, 1499 - 16]
    B = len(spots)
    w = wl.make_workload("t3", [L] * B, [shards] * B, Hkv * G, Hkv, seed=11 + G)
    for b, pos in enumerate(spots):
        for c in range(Hkv):
            w.q[b, c * G:(c + 1) * G] = w.q[b, c * G]      # one query per group, so one key dominates all its heads
            qrow = wl.bf16_bits_to_f32(w.q[b, c * G])
            w.k_cache[w.block_table[b, pos // 16], c, pos % 16] = wl.f32_to_bf16_bits(2.0 * qrow)
    dw = run(w, flags)
    T.compare_all(dw, w, tag=f"G={G}")
    # the planted token really dominates: out ~ its value row
    _, _, _, got_out, _ = dw.results()
    for b, pos in enumerate(spots):
        v = wl.bf16_bits_to_f64(w.v_cache[w.block_table[b, pos // 16], 0, pos % 16])
        assert np.abs(got_out[b, 0] - v).max() < 0.05, (b, pos)


# T4: NaN poison everywhere the path must not read
@pytest.mark.parametrize("flags", KERNELS)
def test_nan_poison_is_never_read(flags):
    flags, Hkv = flags
    lens = [70, 333, 18]
    ranges = [[(5, 40), (40, 70)], [(3, 200), (200, 321)], [(1, 2), (2, 17)]]
    w = wl.make_workload("t4", lens, ranges, 4 * Hkv, Hkv, seed=13, pool_factor=2.0, poison_unused=True,
                         poison_tails=True)
    nan = np.uint16(0x7FC0)
    for b, rr in enumerate(ranges):  # poison the tokens outside every shard range too
        covered = np.zeros(lens[b], bool)
        for lo, hi in rr:
            covered[lo:hi] = True
        for i in np.nonzero(~covered)[0]:
            w.k_cache[w.block_table[b, i // 16], :, i % 16] = nan
            w.v_cache[w.block_table[b, i // 16], :, i % 16] = nan
    dw = run(w, flags)
    errs = T.compare_all(dw, w)
    assert errs["out"] < T.ENG_OUT
    # empty shards' vectors are never read by the combine
    w2 = wl.make_workload("t4b", [64], [[(0, 30), (30, 30), (30, 64)]], 2 * Hkv, Hkv, seed=14)
    dw2 = DeviceWorkload(w2, flags=flags)
    dw2.sweep()
    dw2.o_part[0, 1].fill_(float("nan"))
    dw2.merge()
    got = dw2.results()
    ref = T.oracle_all(w2)
    assert T.out_err(got[3], ref[3]) < T.ENG_OUT and T.lse_err(got[4], ref[4]) < T.ENG_LSE


# T5: the same logical data under two page permutations gives bit-identical results
def test_paging_invariance_bitwise():
    lens = [257, 1000, 31]
    ranges = [wl.even_shards(L, 3) for L in lens]
    a = wl.make_workload("t5", lens, ranges, 8, 2, seed=17, table="identity")
    rng = np.random.default_rng(3)
    P = 200
    perm = rng.permutation(P)
    npg = [(L + 15) // 16 for L in lens]
    bt = np.full((3, a.max_pages_per_req), -1, np.int32)
    kc = np.full((P, 2, 16, 128), 0x7FC0, np.uint16)
    vc = np.full((P, 2, 16, 128), 0x7FC0, np.uint16)
    pos = 0
    for b in range(3):
        for p in range(npg[b]):
            bt[b, p] = perm[pos]
            kc[perm[pos]] = a.k_cache[a.block_table[b, p]]
            vc[perm[pos]] = a.v_cache[a.block_table[b, p]]
            pos += 1
    b_ = wl.Workload("t5b", a.batch, a.num_q_heads, a.num_kv_heads, a.max_pages_per_req, a.max_shards, P,
                     a.q, kc, vc, bt, a.seq_lens, a.shard_ranges, a.shard_counts)
    ra = run(a).results()
    rb = run(b_).results()
    rc = run(a, null_table=True).results()   # NULL block table = identity
    for x, y, z in zip(ra, rb, rc):
        assert np.array_equal(x, y) and np.array_equal(x, z)
    T.compare_all(run(a), a)


# T6: extremes: logits near +85, near -85, mixed across shards
@pytest.mark.parametrize("flags", KERNELS)
def test_extreme_logits(flags):
    flags, Hkv = flags
    L = 2048
    w = wl.make_workload("t6", [L] * 3, [wl.even_shards(L, 4)] * 3, 2 * Hkv, Hkv, seed=19, table="shuffled")
    G = 2
    for c in range(Hkv):
        for b in range(3):
            w.q[b, c * G:(c + 1) * G] = w.q[b, c * G]
    def set_logit(b, toks, target):
        for c in range(Hkv):
            qv = wl.bf16_bits_to_f64(w.q[b, c * G])
            k = qv * (target * np.sqrt(128.0) / (qv @ qv))
            for i in toks:
                w.k_cache[w.block_table[b, i // 16], c, i % 16] = wl.f32_to_bf16_bits(k.astype(np.float32))
    set_logit(0, range(L), 85.0)                    # everything near +85: naive sum of e^s overflows fp32
    set_logit(1, range(L), -85.0)                   # everything near -85: naive sum underflows to 0
    set_logit(2, range(0, 512), 85.0)               # shard 0 at +85, shard 3 at -85
    set_logit(2, range(1536, L), -85.0)
    dw = run(w, flags)
    T.compare_all(dw, w)
    _, _, got_lp, _, got_lse = dw.results()
    assert abs(got_lse[0, 0] - (85 + np.log(L))) < 0.5 and abs(got_lse[1, 0] - (-85 + np.log(L))) < 0.5
    assert got_lp[2, 0, 0] > 80 and got_lp[2, 3, 0] < -70


# T7: the combine alone on hand-made shard states
def test_combine_on_handmade_states():
    rng = np.random.default_rng(23)
    cases = [(100.0, 100.0), (85.0, 91.0), (90.0, -90.0), (-90.0, 90.0), (3.0, -np.inf), (-np.inf, 3.0),
             (-np.inf, -np.inf), (0.0, 0.0), (-0.5, 0.25), (88.0, 89.5)]
    B, S, Hq, D = len(cases), 2, 4, 128
    o = rng.standard_normal((B, S, Hq, D)).astype(np.float32)
    l = np.zeros((B, S, Hq), np.float32)
    for b, (a, c) in enumerate(cases):
        l[b, 0], l[b, 1] = a, c
    o[np.isneginf(l)] = np.nan   # empty shards hold garbage that must not be read
    sh = orc.Shape(batch=B, num_q_heads=Hq, num_kv_heads=2, max_shards=S)
    p = qf.params(B, Hq, 2, 4, S, 4)
    for order in ([0, 1], [1, 0]):
        oo, ll = o[:, order].copy(), l[:, order].copy()
        ref_out, ref_lse = orc.combine(oo.astype(np.float64), ll.astype(np.float64), None, sh)
        fold_out, fold_lse = orc.combine_fold(oo.astype(np.float64), ll.astype(np.float64), None, sh)
        d_o, d_l = torch.from_numpy(oo).cuda(), torch.from_numpy(ll).cuda()
        out = torch.full((B, Hq, D), float("nan"), device="cuda")
        lse = torch.full((B, Hq), float("nan"), device="cuda")
        qf.combine(d_o, d_l, None, out, lse, p)
        torch.cuda.synchronize()
        assert T.out_err(out.cpu().numpy(), ref_out) < 1e-6
        assert T.lse_err(lse.cpu().numpy(), ref_lse) < 1e-6
        assert T.out_err(out.cpu().numpy(), fold_out) < 1e-6 and T.lse_err(lse.cpu().numpy(), fold_lse) < 1e-6
    # shard_counts: slots past the count are ignored even if finite
    cnt = torch.ones(B, dtype=torch.int32, device="cuda")
    d_o, d_l = torch.from_numpy(o).cuda(), torch.from_numpy(l).cuda()
    out = torch.empty((B, Hq, D), device="cuda")
    lse = torch.empty((B, Hq), device="cuda")
    qf.combine(d_o, d_l, cnt, out, lse, p)
    ref_out, ref_lse = orc.combine(o.astype(np.float64), l.astype(np.float64), np.ones(B, np.int32), sh)
    assert T.out_err(out.cpu().numpy(), ref_out) < 1e-6 and T.lse_err(lse.cpu().numpy(), ref_lse) < 1e-6


# medium cases that span many stages, several CTA slices and ragged tails
@pytest.mark.parametrize("flags", KERNELS)
@pytest.mark.parametrize("G,seed", [(2, 0), (4, 1), (8, 2), (1, 3), (3, 4), (5, 5), (6, 6), (7, 7)])
def test_medium_ragged_batch(G, seed, flags):
    flags, Hkv = flags
    rng = np.random.default_rng(seed)
    lens = rng.integers(1, 6000, size=12).tolist() + [4096, 129, 127]
    ranges = [wl.fixed_shards(L, 1000) for L in lens]
    w = wl.make_workload("med", lens, ranges, Hkv * G, Hkv, seed=seed, pool_factor=1.2, poison_unused=True,
                         poison_tails=True)
    dw = run(w, flags)
    T.compare_all(dw, w, tag=f"G={G}")
    assert dw.status() == 0


@pytest.mark.parametrize("Hkv,flags", [(2, 0), (8, 0), (16, 0), (2, qf.QF_FLAG_DRAW_ALWAYS), (8, qf.QF_FLAG_DRAW_ALWAYS)])
def test_long_single_request_many_segments(Hkv, flags):
    # one request whose single shard is split over every SM by the balanced schedule
    L = 150_001 if Hkv <= 8 else 40_001
    w = wl.make_workload("long", [L], [[(0, L)]], 2 * Hkv, Hkv, seed=29)
    dw = run(w, flags)
    T.compare_all(dw, w)


def test_small_configs_elementwise():
    for w in (wl.config1(seed=0), wl.config2(seed=1, batch=6), wl.config3(seed=2, batch=4, hi=9000),
              wl.config4(seed=0, ctx=1 << 15, n_shards=16, n_plant=400),
              wl.config4(seed=1, ctx=1 << 15, n_shards=16, n_plant=400, table="shuffled"),
              wl.config5(seed=0, batch=12, hi=8192)):
        dw = run(w)
        T.compare_all(dw, w, tag=w.name)
        dws = run(w, qf.QF_FLAG_SIMPLE_KERNEL)
        T.compare_all(dws, w, tag=w.name + "/simple")
        dwd = run(w, qf.QF_FLAG_DRAW_ALWAYS)
        T.compare_all(dwd, w, tag=w.name + "/draw")


# The schedule of the unit kernel: equal static slices, then chunks of halving size drawn from a counter;
# units cut by piece boundaries are merged by the finish kernel.  Totals from just above the smallest
# sweep that draws (two stage units per SM) up to the size at which drawing is on by default, with units
# much shorter than a chunk, about a chunk, and much longer; the result must not depend on the flag
# beyond fp32 summation order, and both must match the oracle element by element.
@pytest.mark.parametrize("B,L,shard,Hkv,G", [
    (3, 2100, 2100, 8, 4),        # ~400 stage units: a few per SM
    (40, 700, 130, 8, 2),         # units of one or two stages: most chunks hold several whole units
    (6, 9000, 1024, 8, 4),        # units of 8 stages
    (2, 60_000, 60_000, 8, 2),    # two very long units per KV head: every unit cut many times
    (22, 20_000, 4096, 8, 4),     # ~21,000 stage units: drawing is on by default (from 112 per SM)
    (5, 33_000, 7000, 2, 8),      # G = 8 (two epilogue rounds), few KV heads
    (4, 40_000, 5000, 8, 5),      # G = 5 (Qwen3-14B's 40 / 8 heads): a second round of one head
    (3, 30_000, 30_000, 4, 7),    # G = 7, long units cut many times
])
def test_drawn_chunk_schedule(B, L, shard, Hkv, G):
    rng = np.random.default_rng(B * 1000 + L)
    lens = [int(x) for x in rng.integers(L // 2, L + 1, size=B)]
    w = wl.make_workload("draw", lens, [wl.fixed_shards(x, shard) for x in lens], Hkv * G, Hkv, seed=L + G,
                         pool_factor=1.3, poison_unused=True, poison_tails=True)
    res = {}
    for flags in (0, qf.QF_FLAG_DRAW_ALWAYS):
        dw = run(w, flags)
        T.compare_all(dw, w, tag=f"flags={flags}")
        assert dw.status() == 0
        res[flags] = [r.copy() for r in dw.results()]
        # replays of the same launch give the same bits (who draws which chunk varies, the result must not)
        for _ in range(3):
            dw.poison_outputs()
            dw.step()
            for x, y in zip(res[flags], dw.results()):
                assert np.array_equal(x, y)
    for x, y in zip(res[0], res[qf.QF_FLAG_DRAW_ALWAYS]):
        assert np.allclose(x, y, rtol=0, atol=T.ENG_OUT, equal_nan=True)


# T9: run-to-run determinism and canaries around the outputs
@pytest.mark.parametrize("flags", [0, qf.QF_FLAG_DRAW_ALWAYS])
def test_determinism_and_no_stray_writes(flags):
    w = wl.config3(seed=5, batch=6, hi=12000)
    dw = DeviceWorkload(w, flags=flags)
    canary = 1234.5
    bufs = {}
    # the workspace too: exactly qf_workspace_bytes, with guard bytes on both sides (the segment slots of
    # cut units and the piece records live at its end)
    ws_big = torch.full((dw.ws_bytes + 2 * 4096,), 0x5A, dtype=torch.uint8, device="cuda")
    off = (-ws_big.data_ptr()) % 256 + 2048
    dw.workspace = ws_big[off:off + dw.ws_bytes]
    assert dw.workspace.data_ptr() % 256 == 0
    for name in ("o_part", "m_part", "lse_part", "out", "lse"):
        t = getattr(dw, name)
        big = torch.full((t.numel() + 512,), canary, dtype=torch.float32, device="cuda")
        setattr(dw, name, big[256:256 + t.numel()].view(t.shape))
        bufs[name] = big
    runs = []
    for _ in range(3):
        dw.poison_outputs()
        dw.step()
        runs.append([r.copy() for r in dw.results()])
    for r in runs[1:]:
        for x, y in zip(runs[0], r):
            assert np.array_equal(x, y)
    for name, big in bufs.items():
        assert (big[:256] == canary).all() and (big[-256:] == canary).all(), name
    assert (ws_big[:off] == 0x5A).all() and (ws_big[off + dw.ws_bytes:] == 0x5A).all(), "write outside the workspace"
    T.compare_all(dw, w)


# debug flag: an out-of-range page index is skipped and reported, never a fault
@pytest.mark.parametrize("flags", KERNELS)
def test_bad_page_index_is_reported_not_followed(flags):
    flags, Hkv = flags
    L = 400
    w = wl.make_workload("bad", [L, L], [[(0, L)], [(0, L)]], 2 * Hkv, Hkv, seed=31)
    good_entry = int(w.block_table[1, 3])
    w.block_table[1, 3] = w.num_pages + 7
    dw = run(w, flags | qf.QF_FLAG_CHECK_BOUNDS)
    assert dw.status() & qf.QF_STATUS_BAD_PAGE
    # request 0 is untouched; request 1 equals the sweep with page 3's tokens left out
    w.block_table[1, 3] = good_entry
    w2 = wl.make_workload("bad", [L, L], [[(0, L)], [(0, 48), (64, L)]], 2 * Hkv, Hkv, seed=31)
    ref = T.oracle_all(w2)
    got = dw.results()
    assert T.out_err(got[3][0], ref[3][0]) < T.ENG_OUT
    assert T.out_err(got[3][1], ref[3][1]) < T.ENG_OUT and T.lse_err(got[4][1], ref[4][1]) < T.ENG_LSE


@pytest.mark.parametrize("pinned", [True, False])
def test_host_step_matches_device_path(pinned):
    # pinned host buffers are read and written by the kernels themselves (one staging launch more, no copy
    # operations); pageable ones go through copies: the same bits either way
    w = wl.config3(seed=7, batch=5, hi=6000)
    dw = run(w)
    device_launches = dw.step()
    hs = HostStepper(dw, pinned=pinned)
    hs.out_host.fill_(float("nan"))
    hs.lse_host.fill_(float("nan"))
    hs.step()
    assert qf.last_launch_count() == device_launches + (1 if pinned else 0)
    _, _, _, out, lse = dw.results()
    assert np.array_equal(hs.out_host.numpy().astype(np.float64), out)
    assert np.array_equal(hs.lse_host.numpy().astype(np.float64), lse)
    assert hs.h2d_bytes > 0 and hs.d2h_bytes == out.size * 4 + lse.size * 4
    # a second step with a new query through the same buffers
    rng = np.random.default_rng(5)
    w.q = wl.f32_to_bf16_bits(rng.standard_normal(w.q.shape).astype(np.float32))
    hs.q_host.copy_(torch.from_numpy(w.q.view(np.int16)))
    hs.step()
    dw.q.copy_(torch.from_numpy(w.q.view(np.int16)).view(torch.bfloat16).cuda())
    dw.step()
    _, _, _, out, lse = dw.results()
    assert np.array_equal(hs.out_host.numpy().astype(np.float64), out)
    assert np.array_equal(hs.lse_host.numpy().astype(np.float64), lse)


# T8: the five benchmark configurations x seeds 0-2 at full size, in the launch configuration the benchmark
# times, EVERY element of every output: shard states against the oracle's shard states, merged results against
# the oracle's unsharded sweep.  (The oracle finishes the largest of them in seconds on the host cores.)
@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_full_size_configs_every_element(cfg, seed):
    w = wl.CONFIGS[cfg](seed=seed)
    assert T.covers_context(w)
    dw = run(w)
    errs = T.compare_all(dw, w, tag=w.name)
    print(w.name, seed, errs)
    assert dw.status() == 0
    # unused shard slots follow the empty convention
    got_op, got_mp, got_lp, _, _ = dw.results()
    for b in range(w.batch):
        n = int(w.shard_counts[b])
        assert np.isneginf(got_lp[b, n:]).all() and np.isneginf(got_mp[b, n:]).all() and (got_op[b, n:] == 0).all()


# the same at full size for the variants off the headline: the one-million-token request behind a shuffled
# table, and token-major pages; every element again
@pytest.mark.parametrize("cfg,kwargs,flags", [(4, dict(table="shuffled"), 0), (3, {}, qf.QF_FLAG_KV_NHD),
                                              (2, {}, qf.QF_FLAG_KV_NHD), (4, {}, qf.QF_FLAG_KV_NHD)])
def test_full_size_variants_every_element(cfg, kwargs, flags):
    w = wl.CONFIGS[cfg](seed=0, **kwargs)
    dw = run(w, flags)
    T.compare_all(dw, w, tag=f"{w.name} {kwargs} flags={flags}")
    assert dw.status() == 0


# sampled outputs, computed one by one by the oracle's pick entry points (pinned on the CPU against the full
# set): the fast form of the check above, kept for the largest configuration under a second seed family
def test_full_size_config_sampled():
    w = wl.config5(seed=7)
    dw = run(w)
    errs = T.compare_sampled(dw, w, seed=57, tag=w.name)
    print(w.name, errs)
    assert dw.status() == 0


# A cached length beyond what the request's block-table row can address (a caller error) is treated as the row's
# limit: the sweep never indexes past the row (the entries after it belong to the next request).  With the
# bounds flag it is also reported.
@pytest.mark.parametrize("flags", KERNELS)
def test_length_beyond_the_table_row_is_clamped_and_reported(flags):
    flags, Hkv = flags
    mp = 8                                   # 128 tokens per row
    lens = [128, 100, 64]
    w = wl.make_workload("overlong", lens, [[(0, 500), (60, 2000)], [(0, 100), (0, 0)], [(0, 64), (10, 20)]],
                         2 * Hkv, Hkv, seed=37, max_pages_per_req=mp, poison_tails=True)
    for chk in (0, qf.QF_FLAG_CHECK_BOUNDS):
        dw = DeviceWorkload(w, flags=flags | chk)
        dw.seq_lens.copy_(torch.tensor([200, 100, 64], dtype=torch.int32))   # request 0 claims 200 > 8 * 16
        dw.poison_outputs()
        dw.step()
        T.compare_all(dw, w, tag=f"check={chk}")          # the oracle sees the honest length, 128
        assert dw.status() == (qf.QF_STATUS_BAD_PAGE if chk else 0)


@pytest.mark.parametrize("Hkv,flags", [(2, 0), (8, 0), (8, qf.QF_FLAG_DRAW_ALWAYS)])
def test_many_entries_plan_in_scratch(Hkv, flags):
    # more (request, shard) pairs than the in-kernel plan holds: the separate plan kernel path
    rng = np.random.default_rng(41)
    B = 700
    lens = rng.integers(0, 300, size=B).tolist()
    ranges = [wl.even_shards(L, 3) + [(0, 0)] for L in lens]   # S = 4 -> 2,800 entries
    w = wl.make_workload("many", lens, ranges, 2 * Hkv, Hkv, seed=41, poison_tails=True)
    assert w.batch * w.max_shards > 2048
    dw = run(w, flags)
    T.compare_all(dw, w)
    assert dw.status() == 0


def test_a_wait_that_cannot_be_satisfied_times_out_and_leaves_the_context_usable():
    w = wl.config3(seed=9, batch=3, hi=3000)
    dw = DeviceWorkload(w)
    qf.selftest_bounded_wait(dw.workspace)
    assert dw.status() == qf.QF_STATUS_TIMEOUT
    # the same workspace and context go on working, and the stale status does not leak into the next launch
    dw.poison_outputs()
    dw.step()
    assert dw.status() == 0
    T.compare_all(dw, w)


@pytest.mark.parametrize("flags", [0, qf.QF_FLAG_DRAW_ALWAYS])
def test_cuda_graph_replay_with_new_queries(flags):
    # a captured decode step replayed with fresh queries: every replay must behave like a fresh launch
    # (the scratch words that must "start at zero" are tagged per launch, also under replay)
    lens = [40_000, 9_000, 123, 17_000]
    w = wl.make_workload("graph", lens, [wl.fixed_shards(L, 8192) for L in lens], 16, 8, seed=83)
    dw = DeviceWorkload(w, flags=flags)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        dw.step(s)                      # first call outside capture (one-time set-up), as documented
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            dw.step(s)
    rng = np.random.default_rng(83)
    for it in range(3):
        w.q = wl.f32_to_bf16_bits(rng.standard_normal(w.q.shape).astype(np.float32))
        dw.q.copy_(torch.from_numpy(w.q.view(np.int16)).view(torch.bfloat16).cuda())
        dw.poison_outputs()
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        T.compare_all(dw, w, tag=f"replay {it}")
        assert dw.status() == 0


@pytest.mark.parametrize("seed", list(range(32)))
def test_randomized_shapes_and_ranges(seed):
    # random batch, head counts, group size, lengths, unaligned / overlapping / empty shard ranges, pool slack
    rng = np.random.default_rng(1000 + seed)
    Hkv = int(rng.choice([1, 2, 3, 4, 8, 16]))
    G = int(rng.integers(1, 9))
    B = int(rng.integers(1, 9))
    S = int(rng.integers(1, 7))
    lens = [int(x) for x in rng.choice([0, 1, 15, 16, 17, 127, 128, 129, 500, 3000, 20000], size=B)]
    ranges = []
    for L in lens:
        rr = []
        for _ in range(S):
            kind = rng.integers(4)
            if kind == 0 or L == 0:
                rr.append((0, 0))
            elif kind == 1:
                rr.append((0, L))
            else:
                a, b = sorted(int(x) for x in rng.integers(-3, L + 5, size=2))
                rr.append((a, b))
        ranges.append(rr)
    flags = int(rng.choice([0, qf.QF_FLAG_DRAW_ALWAYS, qf.QF_FLAG_CHECK_BOUNDS,
                            qf.QF_FLAG_DRAW_ALWAYS | qf.QF_FLAG_CHECK_BOUNDS]))
    w = wl.make_workload("fuzz", lens, ranges, Hkv * G, Hkv, seed=seed, pool_factor=float(rng.choice([1.0, 1.5])),
                         poison_unused=True, poison_tails=True, max_pages_per_req=max(1, (max(lens) + 15) // 16 + 2))
    dw = run(w, flags)
    T.compare_all(dw, w, tag=f"seed={seed} Hkv={Hkv} G={G} B={B} S={S} flags={flags}")
    assert dw.status() == 0


# Section 5, one request's cache split over devices, without a gather: every (virtual) rank sweeps the shard slots
# it holds and writes them straight into the merging device's shard-state arrays (out_shards / out_shard_offset);
# the merging device combines.  The ranks here are successive calls on one GPU, each with its own workspace, as
# they would be separate GPUs writing through peer-mapped pointers.
@pytest.mark.parametrize("world", [2, 3, 4])
@pytest.mark.parametrize("flags", [0, qf.QF_FLAG_DRAW_ALWAYS, qf.QF_FLAG_SIMPLE_KERNEL])
def test_split_request_written_in_place_by_virtual_ranks(world, flags):
    from paper_2608_15473_b200 import multi
    lens = [40_000, 7_000, 0, 129]
    S = 9
    w = wl.make_workload("split", lens, [wl.even_shards(L, S) for L in lens], 16, 8, seed=43 + world)
    base = DeviceWorkload(w, flags=flags)
    per = -(-S // world)
    St = per * world
    B, Hq = w.batch, w.num_q_heads
    canary = 777.0
    o_all = torch.full((B, St, Hq, 128), canary, dtype=torch.float32, device="cuda")
    m_all = torch.full((B, St, Hq), canary, dtype=torch.float32, device="cuda")
    l_all = torch.full((B, St, Hq), canary, dtype=torch.float32, device="cuda")
    for rank in range(world):
        p = multi.rank_sweep_params(base.params, world, rank)
        ranges = multi.local_shard_ranges(base.shard_ranges, S, world, rank).contiguous()
        ws = torch.empty(qf.workspace_bytes(p), dtype=torch.uint8, device="cuda")
        # before the call the rank's slots still hold the canary; after it, only they have changed
        before = o_all.clone()
        qf.decode_partial(base.q, base.k_cache, base.v_cache, base.block_table, base.seq_lens, ranges, o_all, m_all,
                          l_all, p, ws, ws.numel())
        torch.cuda.synchronize()
        lo, hi = rank * per, (rank + 1) * per
        assert (o_all[:, lo:hi] != canary).any() and not (l_all[:, lo:hi] == canary).any()
        untouched = torch.ones(St, dtype=torch.bool, device="cuda")
        untouched[lo:hi] = False
        assert torch.equal(o_all[:, untouched], before[:, untouched])
    # the merging device: n-way combine over the padded shard table
    out = torch.empty((B, Hq, 128), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
    pc = qf.params(batch=B, num_q_heads=Hq, num_kv_heads=w.num_kv_heads, max_pages_per_req=w.max_pages_per_req,
                   max_shards=St, num_pages=w.num_pages)
    qf.combine(o_all, l_all, None, out, lse, pc)
    torch.cuda.synchronize()
    sh = T.oracle_shape(w)
    ref_out, ref_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
    assert T.out_err(out.cpu().numpy(), ref_out) <= T.ENG_OUT
    assert T.lse_err(lse.cpu().numpy(), ref_lse) <= T.ENG_LSE
    # and every real slot equals the oracle's shard state; padded slots are empty
    ref_o, ref_m, ref_l = orc.decode_partial(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh)
    got_o, got_l = o_all.cpu().numpy().astype(np.float64), l_all.cpu().numpy().astype(np.float64)
    for rank in range(world):
        sl = multi.shard_slice(S, world, rank)
        dst = slice(rank * per, rank * per + len(sl))
        assert T.out_err(got_o[:, dst], ref_o[:, sl.start:sl.stop]) <= T.ENG_OUT
        assert T.lse_err(got_l[:, dst], ref_l[:, sl.start:sl.stop]) <= T.ENG_LSE
        assert np.isneginf(got_l[:, rank * per + len(sl):(rank + 1) * per]).all()


# A whole step over a SMALL sweep (qf_decode_step): the pieces of cut units and the request's shards are merged by
# one kernel that plans while the sweep runs.  Against the oracle, against the three-kernel path, and bit for bit
# against itself over repeated launches.
@pytest.mark.parametrize("Hkv,G", [(8, 2), (8, 4), (2, 8), (1, 1), (4, 7), (16, 2), (8, 5)])
def test_small_sweeps_merge_with_one_kernel(Hkv, G):
    rng = np.random.default_rng(Hkv * 10 + G)
    cases = [
        ([4096], [[(0, 4096)]]),                                     # one request, one shard: every unit cut ~16 times
        ([3000, 0, 17, 1200], [wl.even_shards(L, 3) for L in (3000, 0, 17, 1200)]),
        ([900] * 6, [[(0, 100), (100, 100), (100, 900), (950, 2000)]] * 6),   # empty and out-of-range shards
        ([int(x) for x in rng.integers(1, 2000, size=9)], None),
        ([5000, 64], [wl.even_shards(L, 20) for L in (5000, 64)]),   # more uncut shards than one batch holds
    ]
    for lens, ranges in cases:
        if ranges is None:
            ranges = [wl.fixed_shards(L, 512) for L in lens]
        w = wl.make_workload("small", lens, ranges, Hkv * G, Hkv, seed=G + len(lens), poison_tails=True,
                             pool_factor=1.25, poison_unused=True)
        dw = run(w)
        small = w.batch * w.max_shards * Hkv * (-(-w.max_pages_per_req // 8)) <= 16 * 148 and w.max_shards <= 32
        assert qf.last_launch_count() == (2 if small else 3)
        T.compare_all(dw, w, tag=f"Hkv={Hkv} G={G} lens={lens[:4]}")
        assert dw.status() == 0
        first = [r.copy() for r in dw.results()]
        for _ in range(3):
            dw.poison_outputs()
            dw.step()
            for x, y in zip(first, dw.results()):
                assert np.array_equal(x, y)
        # the same as two calls, and as one call with the small path switched off: three kernels, same results
        # within fp32 summation order
        for dw3 in (run(w, two_calls=True), run(w, qf.QF_FLAG_NO_SMALL_MERGE)):
            assert qf.last_launch_count() in (1, 3)      # the merge alone, or sweep + finish + merge
            T.compare_all(dw3, w)
            for x, y in zip(dw.results(), dw3.results()):
                assert np.allclose(x, y, rtol=0, atol=T.ENG_OUT, equal_nan=True)


def test_small_sweep_honours_shard_counts_and_the_length_bound():
    # shards past shard_counts[b] are swept but not merged; a max_seq_len bound makes a wide table small
    lens = [700, 300, 64]
    ranges = [[(0, 200), (200, 500), (500, 700)], [(0, 300), (0, 150), (150, 300)], [(0, 64), (0, 0), (0, 64)]]
    w = wl.make_workload("fuse-counts", lens, ranges, 8, 2, seed=3, shard_counts=[3, 1, 1], max_pages_per_req=4000)
    dw = run(w)
    assert qf.last_launch_count() == 3            # the table rows are wide: nothing says the sweep is small
    T.compare_all(dw, w)
    dw.params.max_seq_len = 1024
    dw.poison_outputs()
    dw.step()
    assert qf.last_launch_count() == 2
    T.compare_all(dw, w)
    # a bound below a request's real length clamps it, like a short table row
    dw.params.max_seq_len = 256
    dw.poison_outputs()
    dw.step()
    w2 = wl.make_workload("fuse-counts", lens, ranges, 8, 2, seed=3, shard_counts=[3, 1, 1], max_pages_per_req=4000)
    w2.seq_lens = np.minimum(w2.seq_lens, 256).astype(np.int32)
    T.compare_all(dw, w2)


@pytest.mark.parametrize("depth", [1, 2, 3])
def test_pipelined_host_steps_match_the_device_path(depth):
    # steps in flight with different queries: every ticket's result equals the device-resident step on that query,
    # bit for bit, whatever overlaps with whatever; host buffers rotate with the pipe's slots
    w = wl.config3(seed=11, batch=5, hi=7000)
    dw = DeviceWorkload(w)
    pipe = HostPipeline(dw, depth=depth)
    rng = np.random.default_rng(depth)
    queries = [wl.f32_to_bf16_bits(rng.standard_normal(w.q.shape).astype(np.float32)) for _ in range(7)]
    want = []
    for qb in queries:
        dw.q.copy_(torch.from_numpy(qb.view(np.int16)).view(torch.bfloat16).cuda())
        dw.poison_outputs()
        dw.step()
        _, _, _, out, lse = dw.results()
        want.append((out, lse))
    tickets = []
    got = {}
    for i, qb in enumerate(queries):
        tickets.append(pipe.submit(qb))
        if i >= depth - 1:                      # keep `depth` steps in flight, collect the oldest
            t = tickets[i - (depth - 1)]
            out, lse = pipe.wait(t)
            got[t] = (out.numpy().astype(np.float64).copy(), lse.numpy().astype(np.float64).copy())
    for t in tickets:
        if t not in got:
            out, lse = pipe.wait(t)
            got[t] = (out.numpy().astype(np.float64).copy(), lse.numpy().astype(np.float64).copy())
    for t, (out, lse) in zip(tickets, want):
        assert np.array_equal(got[t][0], out) and np.array_equal(got[t][1], lse), t
    # against the oracle for the last query
    w.q = queries[-1]
    ref = T.oracle_all(w)
    assert T.out_err(got[tickets[-1]][0], ref[3]) <= T.ENG_OUT and T.lse_err(got[tickets[-1]][1], ref[4]) <= T.ENG_LSE
    pipe.close()


@pytest.mark.parametrize("seed", list(range(24)))
def test_randomized_small_steps(seed):
    # whole steps over small random problems: up to 32 shard slots, random shard counts (0 included), random ranges,
    # every group size and layout flag; most of them take the one-kernel merge after the sweep
    rng = np.random.default_rng(5000 + seed)
    Hkv = int(rng.choice([1, 2, 4, 8, 16]))
    G = int(rng.integers(1, 9))
    B = int(rng.integers(1, 13))
    S = int(rng.choice([1, 2, 3, 5, 8, 13, 32]))
    maxlen = int(rng.choice([40, 300, 1500, 5000]))
    lens = [int(x) for x in rng.integers(0, maxlen + 1, size=B)]
    ranges = []
    for L in lens:
        kind = rng.integers(3)
        if kind == 0:
            rr = wl.even_shards(L, S)
        elif kind == 1:
            rr = wl.fixed_shards(L, max(1, int(rng.integers(1, maxlen + 2))))[:S]
        else:
            rr = [tuple(sorted(int(x) for x in rng.integers(-3, L + 5, size=2))) for _ in range(S)]
        rr = list(rr) + [(0, 0)] * (S - len(rr))
        ranges.append(rr[:S])
    counts = [int(rng.integers(0, S + 1)) for _ in lens] if rng.integers(2) else None
    flags = int(rng.choice([0, qf.QF_FLAG_DRAW_ALWAYS, qf.QF_FLAG_CHECK_BOUNDS, qf.QF_FLAG_KV_NHD]))
    w = wl.make_workload("small-fuzz", lens, ranges, Hkv * G, Hkv, seed=seed, pool_factor=float(rng.choice([1.0, 1.4])),
                         poison_unused=True, poison_tails=True, shard_counts=counts,
                         max_pages_per_req=max(1, (max(lens) + 15) // 16 + int(rng.integers(0, 3))))
    dw = run(w, flags)
    T.compare_all(dw, w, tag=f"seed={seed} Hkv={Hkv} G={G} B={B} S={S} flags={flags} launches={qf.last_launch_count()}")
    assert dw.status() == 0
