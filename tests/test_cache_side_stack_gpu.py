"""GPU parity of the cache side's whole per-token job over a stack of layers (Section 4): per layer sweep with the
query it holds, fold of the current token, cache write, u' = z + W_o a and the next layer's q = W_q N_1(u') —
driven by runtime.CacheSideStack, eagerly and replayed from one CUDA graph, against the fp64 CPU oracle's own chain
(the oracle never sees a value the GPU computed)."""
import numpy as np
import pytest
import torch

from oracle import qf_oracle as orc
from paper_2608_15473_b200 import build as qf_build
from paper_2608_15473_b200 import workloads as wl
from paper_2608_15473_b200.runtime import CacheSideStack, DeviceWorkload

import qf_testlib as T

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    qf_build.build()


def bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, np.float32))


def dev_bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).cuda()


def f64(b):
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def host_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def close_bf16(got_bits, want_bits, abs_tol):
    """One bf16 unit in the last place of the value plus abs_tol of the row's scale (the projection tests' bar)."""
    got, want = f64(got_bits), f64(want_bits)
    rms = np.sqrt((want ** 2).mean(axis=-1, keepdims=True))
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.maximum(np.abs(got), np.abs(want)), 2.0 ** -120))) - 7)
    return float((np.abs(got - want) - (ulp + abs_tol * rms)).max())


def test_tokens_through_a_stack_of_layers():
    n_layers, tokens = 3, 4
    Hq, Hkv, D, d_model = 16, 8, 128, 1024
    n_q = Hq * D
    lens0 = [5, 300, 2000]
    B = len(lens0)
    cap = [L + tokens for L in lens0]
    rng = np.random.default_rng(211)
    ws = []
    for l in range(n_layers):
        w = wl.make_workload(f"stack{l}", cap, [wl.fixed_shards(c, 512) for c in cap], Hq, Hkv, seed=300 + l)
        w.seq_lens = np.asarray(lens0, np.int32)
        ws.append(w)
    w_o = bits(rng.standard_normal((n_layers, d_model, n_q)) / n_q ** 0.5)
    w_q = bits(rng.standard_normal((n_layers, n_q, d_model)) / d_model ** 0.5)
    gain = bits(1.0 + 0.1 * rng.standard_normal((n_layers, d_model)))
    dws = []
    for w in ws:
        dw = DeviceWorkload(w)
        dw.seq_lens.copy_(torch.from_numpy(w.seq_lens).cuda())
        dws.append(dw)
    stack = CacheSideStack(dws, dev_bf16(w_o), dev_bf16(w_q), dev_bf16(gain), eps=1e-6)
    z = torch.empty((n_layers, B, d_model), dtype=torch.bfloat16, device="cuda")
    k_new = torch.empty((n_layers, B, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_new = torch.empty_like(k_new)
    u_out = torch.zeros((n_layers, B, d_model), dtype=torch.bfloat16, device="cuda")
    sh = T.oracle_shape(ws[0])
    q_ref = ws[0].q.copy()          # the oracle's own query for the next stage, starting from layer 0's given one
    stream = torch.cuda.Stream()
    graph = None
    worst_u = worst_q = -1.0
    for t in range(tokens):
        z_h = bits(2.0 * rng.standard_normal((n_layers, B, d_model)))
        k_h = bits(rng.standard_normal((n_layers, B, Hkv, D)))
        v_h = bits(rng.standard_normal((n_layers, B, Hkv, D)))
        z.copy_(dev_bf16(z_h)); k_new.copy_(dev_bf16(k_h)); v_new.copy_(dev_bf16(v_h))
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            if t == 0:
                n = stack.token(z, k_new, v_new, u_out, stream)          # eager: also the one-time set-up
                assert n == n_layers * 5     # sweep and its finish, fold with cache write and length advance, two products
            else:
                if graph is None:
                    graph = stack.capture(z, k_new, v_new, u_out, stream)
                    # the capture ran nothing: lengths are where token t - 1 left them
                    assert np.array_equal(dws[0].seq_lens.cpu().numpy(), ws[0].seq_lens)
                graph.replay()
        torch.cuda.synchronize()
        assert stack.status() == 0
        for l in range(n_layers):
            w = ws[l]
            for b in range(B):
                L = int(w.seq_lens[b])
                w.k_cache[w.block_table[b, L // 16], :, L % 16] = k_h[l, b]
                w.v_cache[w.block_table[b, L // 16], :, L % 16] = v_h[l, b]
            w.seq_lens = w.seq_lens + 1
            a_ref, _ = orc.decode_full(q_ref, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
            u_ref, q_next = orc.project_pair(a_ref.reshape(B, n_q).astype(np.float32), z_h[l], w_o[l], gain[l],
                                             w_q[l], eps=1e-6)
            # a unit flipped in a query moves that request's attention output by up to a few 1e-3 and everything
            # after it by as much of the row's scale: one percent is an order of magnitude inside a wrong wiring
            worst_u = max(worst_u, close_bf16(host_bits(u_out[l]), u_ref, 1e-2))
            got_q = host_bits(dws[(l + 1) % n_layers].q).reshape(B, n_q)
            worst_q = max(worst_q, close_bf16(got_q, q_next, 1e-2))
            assert np.array_equal(dws[l].seq_lens.cpu().numpy(), w.seq_lens)
            q_ref = q_next.reshape(B, Hq, D)
        assert worst_u <= 0 and worst_q <= 0, (t, worst_u, worst_q)
    for l in range(n_layers):        # every layer's cache equals its host mirror bit for bit
        assert np.array_equal(host_bits(dws[l].k_cache), ws[l].k_cache)
        assert np.array_equal(host_bits(dws[l].v_cache), ws[l].v_cache)

