"""GPU parity of the cache side's projection pair (u' = z + W_o a, q = W_q N_1(u')) against the fp64 oracle.

Tolerance.  Both sides round value -> binary32 -> bf16 at the same three points, so most outputs are the same
bits.  The kernel's sums carry fp32 accumulation error, a few 1e-7 of the row's scale, which shows in two
ways: (1) now and then it carries a value across a bf16 rounding boundary, and the output differs by one
bf16 unit in the last place of the value; (2) where the sum nearly cancels, the value is so small that the
same absolute error is several of ITS units in the last place.  A u' element that flipped (one part in 2^8
of it; about one element in 4,000 does) changes that request's normalised operand x_k by the same share, and
through it every q of the request by |W_q[o,k]| 2^-8 |x_k|: with |W_q| up to about 4/sqrt(d_model) and |x_k|
up to about 4 that is up to 1e-3 of the row's scale, and a row may hold two flips.  So an element passes if
    |got - ref| <= ulp_bf16(max(|got|, |ref|)) + abs_tol * rms(row),   abs_tol = 1e-5 for u', 2.5e-3 for q
(for q that is two thirds of a bf16 unit in the last place of a typical element), and the share of elements
that differ at all is bounded (1 % for u', 5 % for q; measured 0.03 % and 0.2-1.6 %)."""
import numpy as np
import pytest
import torch

from oracle import qf_oracle as orc
from paper_2608_15473_b200 import binding as qf
from paper_2608_15473_b200 import build as qf_build
from paper_2608_15473_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    qf_build.build()


def bits_to_f64(b):
    return (np.asarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def host_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def make_inputs(batch, d_model, n_q, seed):
    rng = np.random.default_rng(seed)
    sc_o, sc_q = 1.0 / np.sqrt(n_q), 1.0 / np.sqrt(d_model)
    w_o = wl.f32_to_bf16_bits((rng.standard_normal((d_model, n_q)) * sc_o).astype(np.float32))
    w_q = wl.f32_to_bf16_bits((rng.standard_normal((n_q, d_model)) * sc_q).astype(np.float32))
    g = wl.f32_to_bf16_bits((1.0 + 0.1 * rng.standard_normal(d_model)).astype(np.float32))
    a = rng.standard_normal((batch, n_q)).astype(np.float32)
    z = wl.f32_to_bf16_bits((rng.standard_normal((batch, d_model)) * 2.0).astype(np.float32))
    return a, z, w_o, g, w_q


def run_gpu(a, z, w_o, g, w_q, eps):
    batch, n_q = a.shape
    d_model = z.shape[1]
    need = qf.project_workspace_bytes(batch, d_model, n_q)
    assert need > 0
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    u = torch.full((batch, d_model), float("nan"), dtype=torch.bfloat16, device="cuda")
    q = torch.full((batch, n_q), float("nan"), dtype=torch.bfloat16, device="cuda")
    args = (torch.from_numpy(a).cuda(), dev_bf16(z), dev_bf16(w_o), dev_bf16(g), dev_bf16(w_q), u, q, eps, ws)
    qf.project_pair(*args)
    torch.cuda.synchronize()
    assert qf.project_status(ws) == 0
    assert qf.last_launch_count() == 2
    return host_bits(u), host_bits(q), args


def ulp_bf16(x):
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(x), 2.0 ** -120))) - 7)


def check(u, q, ref_u, ref_q, tag):
    for name, got, ref, abs_tol, share in (("u'", u, ref_u, 1e-5, 0.01), ("q", q, ref_q, 2.5e-3, 0.05)):
        x, r = bits_to_f64(got), bits_to_f64(ref)
        assert np.isfinite(x).all(), (tag, name)
        rms = np.sqrt((r ** 2).mean(axis=1, keepdims=True))
        d = np.abs(x - r)
        lim = ulp_bf16(np.maximum(np.abs(r), np.abs(x))) + abs_tol * rms
        worst = np.unravel_index(np.argmax(d - lim), d.shape)
        assert (d <= lim).all(), (tag, name, "at", worst, "got", x[worst], "ref", r[worst], "limit", lim[worst])
        assert (d > 0).mean() < share, (tag, name, "share of elements that differ", (d > 0).mean())


@pytest.mark.parametrize("batch,d_model,n_q", [
    (8, 1024, 2048),      # Qwen3-0.6B shape, the paper's batch of eight
    (1, 1024, 2048),      # served alone: the matrix-vector case
    (17, 1024, 2048),     # a batch that is not a multiple of the tile's 16 columns
    (8, 2560, 4096),      # Qwen3-4B shape
    (33, 2560, 4096),     # 48 padded columns
    (64, 2560, 4096),     # the largest batch one call takes
    (32, 5120, 5120),     # the largest K (ten boxes per CTA)
    (64, 5120, 5120),     # and with the largest batch: a two-slot ring
    (32, 512, 1024),      # the smallest shapes: one and two boxes per CTA
    (64, 512, 1024),      # ... with the widest batch: the receive area is larger than the one-box ring
])
def test_matches_the_oracle(batch, d_model, n_q):
    a, z, w_o, g, w_q = make_inputs(batch, d_model, n_q, seed=batch * 7 + d_model)
    eps = 1e-6
    u, q, _ = run_gpu(a, z, w_o, g, w_q, eps)
    ref_u, ref_q = orc.project_pair(a, z, w_o, g, w_q, eps=eps)
    check(u, q, ref_u, ref_q, f"batch={batch} d_model={d_model} n_q={n_q}")


def test_structured_inputs_are_exact_and_runs_repeat_bit_for_bit():
    batch, d_model, n_q = 8, 1024, 2048
    a, z, w_o, g, w_q = make_inputs(batch, d_model, n_q, seed=3)
    # one-hot attention outputs read out single columns of W_o: no rounding anywhere, so bit-exact
    a1 = np.zeros_like(a)
    cols = [0, 63, 64, 1023, 1024, 2047, 511, 1500]
    for m, j in enumerate(cols):
        a1[m, j] = 1.0
    z0 = np.zeros_like(z)
    u, q, args = run_gpu(a1, z0, w_o, g, w_q, 1e-6)
    for m, j in enumerate(cols):
        assert np.array_equal(u[m], w_o[:, j]), (m, j)
    ref_u, ref_q = orc.project_pair(a1, z0, w_o, g, w_q, eps=1e-6)
    check(u, q, ref_u, ref_q, "one-hot")
    # determinism: the split-K sum runs in rank order, so repeated launches give the same bits
    first = None
    for _ in range(4):
        qf.project_pair(*args)
        torch.cuda.synchronize()
        bits = (host_bits(args[5]).copy(), host_bits(args[6]).copy())
        if first is None:
            first = bits
        assert np.array_equal(first[0], bits[0]) and np.array_equal(first[1], bits[1])


def test_feeds_the_sweep():
    # q of the pair has the layout the sweep consumes.  No oracle here (its inputs never come from the GPU):
    # the sweep run directly on the projection's output tensor must give the same bits as the sweep run on a
    # fresh upload of those bits, and the oracle's own chain (projection, then sweep with ITS q) must agree
    # with the GPU's chain to within what a few flipped bf16 units of q can move the attention output.
    from paper_2608_15473_b200.runtime import DeviceWorkload
    Hq, Hkv, D = 16, 8, 128
    lens = [300, 4000, 17, 2048, 999, 64, 1, 1500]
    w = wl.make_workload("proj", lens, [wl.fixed_shards(L, 1024) for L in lens], Hq, Hkv, seed=5)
    a, z, w_o, g, w_q = make_inputs(len(lens), 1024, Hq * D, seed=11)
    _, q_bits, args = run_gpu(a, z, w_o, g, w_q, 1e-6)
    dw = DeviceWorkload(w)
    dw.q = args[6].view(len(lens), Hq, D)              # the projection's output tensor, in place
    dw.step()
    in_place = [r.copy() for r in dw.results()]
    dw2 = DeviceWorkload(w)
    dw2.q.copy_(dev_bf16(q_bits).view(len(lens), Hq, D))
    dw2.step()
    for x, y in zip(in_place, dw2.results()):
        assert np.array_equal(x, y, equal_nan=True)
    # the oracle's chain, from its own q
    _, ref_q = orc.project_pair(a, z, w_o, g, w_q, eps=1e-6)
    sh = orc.Shape(batch=w.batch, num_q_heads=Hq, num_kv_heads=Hkv, max_pages_per_req=w.max_pages_per_req,
                   max_shards=w.max_shards)
    ref_out, ref_lse = orc.decode_full(ref_q.reshape(len(lens), Hq, D), w.k_cache, w.v_cache, w.block_table,
                                       w.seq_lens, sh)
    out, lse = in_place[3], in_place[4]
    # one flipped unit of one q element moves a score by |q_k| 2^-8 |k_ik| / sqrt(D), about 4e-4: an order of
    # magnitude inside these bounds, far outside the 5e-5 / 1e-6 a correct sweep has on identical inputs
    assert np.abs(out - ref_out).max() <= 5e-3
    fin = np.isfinite(ref_lse)
    assert np.array_equal(np.isfinite(lse), fin) and np.abs(lse[fin] - ref_lse[fin]).max() <= 5e-3


def test_unsupported_shapes_and_bad_arguments_are_rejected():
    assert qf.project_workspace_bytes(8, 1000, 2048) == 0        # not a multiple of 512
    assert qf.project_workspace_bytes(65, 1024, 2048) == 0       # batch above 64
    assert qf.project_workspace_bytes(8, 1024, 6144) == 0        # K above 5,120
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    t = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    L = qf.lib()
    p = lambda x: qf._ptr(x)
    assert L.qf_project_pair(p(t), p(t), p(t), p(t), p(t), p(t), p(t), 8, 1000, 2048, 1e-6, p(ws), 4096, None) == qf.QF_ERR_UNSUPPORTED
    assert L.qf_project_pair(None, p(t), p(t), p(t), p(t), p(t), p(t), 8, 1024, 2048, 1e-6, p(ws), 4096, None) == qf.QF_ERR_NULL
    assert L.qf_project_pair(p(t), p(t), p(t), p(t), p(t), p(t), p(t), 8, 1024, 2048, 1e-6, p(ws), 16, None) == qf.QF_ERR_WORKSPACE
    assert L.qf_project_pair(p(t), p(t), p(t) + 64, p(t), p(t), p(t), p(t), 8, 1024, 2048, 1e-6, p(ws), 4096, None) == qf.QF_ERR_BAD_SHAPE


def test_graph_replay_with_new_inputs():
    # the pair captured in a CUDA graph and replayed with new attention outputs: every replay is a fresh call
    batch, d_model, n_q = 8, 1024, 2048
    a, z, w_o, g, w_q = make_inputs(batch, d_model, n_q, seed=21)
    _, _, args = run_gpu(a, z, w_o, g, w_q, 1e-6)           # first call outside capture
    a_dev, u_dev, q_dev = args[0], args[5], args[6]
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            qf.project_pair(*args, stream=s)
    rng = np.random.default_rng(22)
    for it in range(3):
        a2 = rng.standard_normal(a.shape).astype(np.float32)
        a_dev.copy_(torch.from_numpy(a2).cuda())
        u_dev.fill_(float("nan"))
        q_dev.fill_(float("nan"))
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        ref_u, ref_q = orc.project_pair(a2, z, w_o, g, w_q, eps=1e-6)
        check(host_bits(u_dev), host_bits(q_dev), ref_u, ref_q, f"replay {it}")
        assert qf.project_status(args[8]) == 0


def test_no_stray_writes():
    # outputs and workspace sit inside guard regions; nothing outside them may change
    batch, d_model, n_q = 17, 1024, 2048
    a, z, w_o, g, w_q = make_inputs(batch, d_model, n_q, seed=31)
    need = qf.project_workspace_bytes(batch, d_model, n_q)
    guard = 4096
    ws_big = torch.full((need + 2 * guard + 256,), 0x5A, dtype=torch.uint8, device="cuda")
    off = (-ws_big.data_ptr()) % 256 + guard
    ws = ws_big[off:off + need]
    u_big = torch.full((batch * d_model + 1024,), 7.0, dtype=torch.bfloat16, device="cuda")
    q_big = torch.full((batch * n_q + 1024,), 7.0, dtype=torch.bfloat16, device="cuda")
    u = u_big[512:512 + batch * d_model].view(batch, d_model)
    q = q_big[512:512 + batch * n_q].view(batch, n_q)
    qf.project_pair(torch.from_numpy(a).cuda(), dev_bf16(z), dev_bf16(w_o), dev_bf16(g), dev_bf16(w_q), u, q, 1e-6, ws)
    torch.cuda.synchronize()
    assert qf.project_status(ws) == 0
    assert (ws_big[:off] == 0x5A).all() and (ws_big[off + need:] == 0x5A).all()
    for big, n in ((u_big, batch * d_model), (q_big, batch * n_q)):
        assert (big[:512] == 7.0).all() and (big[512 + n:] == 7.0).all()
    ref_u, ref_q = orc.project_pair(a, z, w_o, g, w_q, eps=1e-6)
    check(host_bits(u.contiguous()), host_bits(q.contiguous()), ref_u, ref_q, "guarded")


@pytest.mark.parametrize("seed", list(range(12)))
def test_random_shapes(seed):
    # every supported K (multiples of 512 up to 5,120) picks its own ring of weight requests: 1 to 10 boxes per
    # CTA, one to four requests; batches straddle the 16-column padding steps
    rng = np.random.default_rng(500 + seed)
    dims = [512 * k for k in range(1, 11)]
    for _ in range(50):
        batch = int(rng.integers(1, 65))
        d_model, n_q = int(rng.choice(dims)), int(rng.choice(dims))
        if qf.project_workspace_bytes(batch, d_model, n_q) > 0:
            break
    else:
        pytest.skip("no supported shape drawn")
    a, z, w_o, g, w_q = make_inputs(batch, d_model, n_q, seed=seed)
    u, q, _ = run_gpu(a, z, w_o, g, w_q, 1e-6)
    ref_u, ref_q = orc.project_pair(a, z, w_o, g, w_q, eps=1e-6)
    check(u, q, ref_u, ref_q, f"seed={seed} batch={batch} d_model={d_model} n_q={n_q}")


@pytest.mark.parametrize("batch,d_model,n_q", [(8, 1024, 2048), (8, 2560, 4096), (40, 2560, 4096)])
def test_against_the_values_before_the_last_rounding(batch, d_model, n_q):
    # Not through shared rounding points: the oracle also returns u' and q BEFORE their last rounding
    # (fp64 sums of exact products).  A correctly rounded result lies within half a bf16 unit of that value;
    # the kernel's fp32 accumulation adds a few 1e-7 of the row's scale on top (K terms of relative error
    # 2^-24 each, random signs: sqrt(K) 2^-24 of the terms' scale, taken as 4e-6 of the row's rms here).
    # For q the exact value is a function of the oracle's OWN rounded stream, and a flipped u' element on the
    # GPU side moves a whole row of q by up to 1e-3 of its scale (see the module docstring): that term stays.
    a, z, w_o, g, w_q = make_inputs(batch, d_model, n_q, seed=batch + 3 * d_model)
    u, q, _ = run_gpu(a, z, w_o, g, w_q, 1e-6)
    _, _, u_exact, q_exact = orc.project_pair(a, z, w_o, g, w_q, eps=1e-6, exact=True)
    for name, got, exact, abs_tol in (("u'", u, u_exact, 4e-6), ("q", q, q_exact, 2.5e-3)):
        x = bits_to_f64(got)
        rms = np.sqrt((exact ** 2).mean(axis=1, keepdims=True))
        d = np.abs(x - exact)
        lim = 0.5 * ulp_bf16(np.maximum(np.abs(exact), np.abs(x))) + abs_tol * rms
        worst = np.unravel_index(np.argmax(d - lim), d.shape)
        assert (d <= lim).all(), (name, "at", worst, "got", x[worst], "exact", exact[worst], "limit", lim[worst])


def test_against_the_chain_without_any_intermediate_rounding():
    # The definition itself, with NumPy in fp64 and NO rounding of a, u', N_1(u') or q: what the pair computes
    # up to the bf16 roundings the stream's dtype forces.  Each rounding is a relative error of at most 2^-9 per
    # element with random sign, so a row of q is off by well under one percent of its scale in the mean, and no
    # element by more than a few percent; a misplaced or missing step (gain, residual, normalisation, eps, a
    # transposed weight) would be off by tens of percent.
    batch, d_model, n_q = 8, 2560, 4096
    a, z, w_o, g, w_q = make_inputs(batch, d_model, n_q, seed=123)
    eps = 1e-6
    u, q, _ = run_gpu(a, z, w_o, g, w_q, eps)
    Wo, Wq, gg, zz = bits_to_f64(w_o), bits_to_f64(w_q), bits_to_f64(g), bits_to_f64(z)
    u_true = zz + a.astype(np.float64) @ Wo.T
    x_true = gg * u_true / np.sqrt((u_true ** 2).mean(axis=1, keepdims=True) + eps)
    q_true = x_true @ Wq.T
    for name, got, true, mean_tol, max_tol in (("u'", u, u_true, 3e-3, 2e-2), ("q", q, q_true, 6e-3, 4e-2)):
        x = bits_to_f64(got)
        rms = np.sqrt((true ** 2).mean(axis=1, keepdims=True))
        rel = np.abs(x - true) / rms
        assert np.sqrt((rel ** 2).mean()) < mean_tol and rel.max() < max_tol, (name, np.sqrt((rel ** 2).mean()), rel.max())


def test_status_word_is_sticky_until_it_is_read():
    # a timeout raised by one layer's pair must survive the pairs of the layers after it (they share the
    # workspace) until the host reads it; reading clears it.  The failure is made on the host: the test hook
    # ORs the bit in exactly as a kernel whose bounded wait ran out would; no kernel waits on anything.
    batch, d_model, n_q = 8, 1024, 2048
    a, z, w_o, g, w_q = make_inputs(batch, d_model, n_q, seed=9)
    u, q, args = run_gpu(a, z, w_o, g, w_q, 1e-6)
    ws = args[-1]
    assert qf.project_status(ws) == 0
    qf.project_status_inject(ws, qf.QF_STATUS_TIMEOUT)
    for _ in range(5):                      # "layers 1 to L-1"
        qf.project_pair(*args)
    assert qf.project_status(ws) == qf.QF_STATUS_TIMEOUT
    assert qf.project_status(ws) == 0       # read once, then clean
    qf.project_pair(*args)
    torch.cuda.synchronize()
    assert qf.project_status(ws) == 0
    assert np.array_equal(host_bits(args[5]), u) and np.array_equal(host_bits(args[6]), q)
    # an uninitialised workspace (any bit pattern without the tag) reads as clean
    ws.fill_(0xA5)
    assert qf.project_status(ws) == 0
