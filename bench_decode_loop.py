#!/usr/bin/env python
"""Benchmark of the cache side's whole per-token job (Section 4) on one B200: for every layer of a stack, sweep the
layer's KV cache with the query the cache side already holds, fold in the current token, write it into the cache,
close the layer with u' = z + W_o a and open the next with q = W_q N_1(u').

Not the headline benchmark (that is bench.py: the sweep and the merge alone).  A step is one decoded token for the
whole batch through every layer, replayed from ONE CUDA graph; the lengths live on the device and grow by one per
replay, so every replay plans its sweeps anew inside the kernels.  Every layer has its own KV pool and weights
(Qwen3-4B shape: 32 requests with ragged contexts U[1,024, 36,480] -> about 2.4 GB of KV per layer, 42 MB of
weights), so nothing is served from L2.  What the pool would send (z, and the token's k and v per layer) is
synthetic and already on the device: the wire is not part of this measurement.

  python bench_decode_loop.py [--layers 12] [--steps 10] [--warmup 3] [--batch 32]
"""
from __future__ import annotations

import argparse
import json
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

FALLBACK_HBM_GBS = 6650.0
MODEL_LAYERS = 36      # Qwen3-4B: what a whole token costs is reported for this many layers


def hbm_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=12)
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)

    import torch
    from paper_2608_15473_b200 import build as qf_build
    from paper_2608_15473_b200 import workloads as wl
    from paper_2608_15473_b200.runtime import CacheSideStack, DeviceWorkload
    if not torch.cuda.is_available():
        raise SystemExit("bench_decode_loop.py needs a CUDA device: there is no CPU path")
    qf_build.build()
    dev = torch.device("cuda", 0)
    Hq, Hkv, D, d_model = 32, 8, 128, 2560
    n_q = Hq * D
    L, B = args.layers, args.batch
    grow = args.warmup + args.steps + 2                    # tokens appended over the run: pages exist for them
    rng = np.random.Generator(np.random.SFC64(np.random.SeedSequence([args.seed, 0xD1])))
    lens = rng.integers(1024, 36480 + 1, size=B)
    cap = [int(x) + grow for x in lens]
    w = wl.make_workload("cache_side_stack", cap, [wl.fixed_shards(c, 4096) for c in cap], Hq, Hkv, seed=args.seed,
                         table="shuffled")
    w.seq_lens = np.asarray(lens, np.int32)
    layers = []
    for _ in range(L):                                     # the same contents in L separate pools
        dw = DeviceWorkload(w, device=dev)
        dw.seq_lens.copy_(torch.from_numpy(w.seq_lens).to(dev))
        layers.append(dw)
    gen = torch.Generator(device=dev).manual_seed(args.seed)
    w_o = (torch.randn((L, d_model, n_q), device=dev, generator=gen) / n_q ** 0.5).to(torch.bfloat16)
    w_q = (torch.randn((L, n_q, d_model), device=dev, generator=gen) / d_model ** 0.5).to(torch.bfloat16)
    gain = (1.0 + 0.1 * torch.randn((L, d_model), device=dev, generator=gen)).to(torch.bfloat16)
    z = (2.0 * torch.randn((L, B, d_model), device=dev, generator=gen)).to(torch.bfloat16)
    k_new = torch.randn((L, B, Hkv, D), device=dev, generator=gen).to(torch.bfloat16)
    v_new = torch.randn((L, B, Hkv, D), device=dev, generator=gen).to(torch.bfloat16)
    u_out = torch.empty((L, B, d_model), device=dev, dtype=torch.bfloat16)
    stack = CacheSideStack(layers, w_o, w_q, gain, eps=1e-6)
    torch.cuda.synchronize()

    st = torch.cuda.Stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(st):
        launches = stack.token(z, k_new, v_new, u_out, st)          # one-time set-up; also the first warm-up token
        torch.cuda.synchronize()
        graph = stack.capture(z, k_new, v_new, u_out, st)
        for _ in range(args.warmup - 1):
            graph.replay()
        torch.cuda.synchronize()
        e0.record(st)
        for _ in range(args.steps):
            graph.replay()
        e1.record(st)
        torch.cuda.synchronize()
    ms_per_token = e0.elapsed_time(e1) / args.steps
    assert stack.status() == 0 and bool(torch.isfinite(u_out.float()).all())
    lens_now = layers[0].seq_lens.cpu().numpy()
    assert np.array_equal(lens_now, w.seq_lens + args.warmup + args.steps)

    us_per_stage = ms_per_token * 1e3 / L
    mid = w.seq_lens.astype(np.int64) + args.warmup + args.steps // 2     # lengths halfway through the timed region
    kv_bytes = int(mid.sum()) * Hkv * D * 2 * 2
    io_bytes = B * Hq * D * (2 + 4) + B * (w.max_shards * Hq * (D + 2) * 4)        # q in, out, shard states once
    pair_bytes = 2 * d_model * n_q * 2 + B * (n_q * 4 + 3 * d_model * 2 + n_q * 2)
    stage_bytes = kv_bytes + io_bytes + pair_bytes
    peak, peak_kind = hbm_peak()
    achieved = stage_bytes / (us_per_stage * 1e-6) / 1e9
    line = {
        "metric": "cache-side decode: microseconds per layer stage (sweep, fold, cache write, projection pair)",
        "value": us_per_stage, "unit": "us", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_token, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"Qwen3-4B-shaped cache side, {L} layers with their own KV pools and weights, {B} "
                               f"requests, ragged contexts U[1,024, 36,480], 4,096-token shards",
                   "cached_tokens_per_layer": int(mid.sum()), "kv_bytes_per_layer": kv_bytes, "seed": args.seed,
                   "l2": "every layer's KV (GBs) and weights (42 MB) are its own: far larger than L2, no flush needed"},
        "gpu_launches": launches * args.steps,
        "launches_per_stage": launches // L,
        "tokens_per_s_at_36_layers": B / (us_per_stage * 1e-6 * MODEL_LAYERS),
        "ms_per_token_at_36_layers": us_per_stage * MODEL_LAYERS * 1e-3,
        "roofline": {"bound": "hbm", "kernel": "a whole stage (sweep, finish, fold, cache write, two products)",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "bytes_per_stage": stage_bytes, "traffic": None},
    }
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
