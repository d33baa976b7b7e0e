#!/usr/bin/env python
"""Benchmark of the cache side's projection pair (u' = z + W_o a, q = W_q N_1(u')) on one B200.

Not the headline benchmark (that is bench.py): this measures the one dense contraction the cache side owns.
A step is one pass over every layer's pair of a Qwen3-shaped stack, each layer with its own weights (1.5 GB
at the 4B shape: far more than L2, so every weight byte comes from HBM), for one batch of co-resident
requests.  Prints one JSON line: weight GB/s of the pass, the HBM roofline fraction (algorithmic bytes of a
pair / its average time, against the measured copy peak), the same pass with host buffers (attention output
and stream copied in, stream and query copied back, per layer), and the CPU oracle on a sample.

  python bench_projections.py [--shape 4b|0.6b] [--batch 8] [--steps 20] [--warmup 3]
"""
from __future__ import annotations

import argparse
import json
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

SHAPES = {"4b": (2560, 4096, 36), "0.6b": (1024, 2048, 28)}   # d_model, n_q = Hq * 128, layers
FALLBACK_HBM_GBS = 6650.0


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
    ap.add_argument("--shape", default="4b", choices=sorted(SHAPES))
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)

    import torch
    from paper_2608_15473_b200 import binding as qf
    from paper_2608_15473_b200 import build as qf_build
    if not torch.cuda.is_available():
        raise SystemExit("bench_projections.py needs a CUDA device: there is no CPU path")
    qf_build.build()
    d_model, n_q, layers = SHAPES[args.shape]
    batch = args.batch
    dev = torch.device("cuda", 0)
    gen = torch.Generator(device=dev).manual_seed(args.seed)
    w_o = (torch.randn((layers, d_model, n_q), device=dev, generator=gen) / n_q ** 0.5).to(torch.bfloat16)
    w_q = (torch.randn((layers, n_q, d_model), device=dev, generator=gen) / d_model ** 0.5).to(torch.bfloat16)
    gain = (1.0 + 0.1 * torch.randn((layers, d_model), device=dev, generator=gen)).to(torch.bfloat16)
    a = torch.randn((batch, n_q), device=dev, generator=gen)
    z = (2.0 * torch.randn((batch, d_model), device=dev, generator=gen)).to(torch.bfloat16)
    u = torch.empty((batch, d_model), device=dev, dtype=torch.bfloat16)
    q = torch.empty((batch, n_q), device=dev, dtype=torch.bfloat16)
    ws = torch.empty(qf.project_workspace_bytes(batch, d_model, n_q), dtype=torch.uint8, device=dev)
    eps = 1e-6

    def one_pass():
        for l in range(layers):
            qf.project_pair(a, z, w_o[l], gain[l], w_q[l], u, q, eps, ws)

    one_pass()
    torch.cuda.synchronize()
    assert qf.project_status(ws) == 0 and bool(torch.isfinite(q.float()).all())
    # A pass is 2 x layers short dependent launches: it is replayed from a CUDA graph, as a decode loop would
    # run it (launched one by one from Python the host, not the GPU, sets the pace: reported as "eager").
    st = torch.cuda.Stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(st):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            for l in range(layers):
                qf.project_pair(a, z, w_o[l], gain[l], w_q[l], u, q, eps, ws, stream=st)
        for _ in range(args.warmup):
            graph.replay()
        torch.cuda.synchronize()
        e0.record(st)
        for _ in range(args.steps):
            graph.replay()
        e1.record(st)
        torch.cuda.synchronize()
    ms_per_step = e0.elapsed_time(e1) / args.steps
    us_per_pair = ms_per_step * 1e3 / layers
    assert qf.project_status(ws) == 0
    e0.record()
    for _ in range(args.steps):
        one_pass()
    e1.record()
    torch.cuda.synchronize()
    eager_us_per_pair = e0.elapsed_time(e1) / args.steps * 1e3 / layers

    # the same pass from pinned host buffers: a and z in, u' and q back, per layer
    a_h, z_h = a.cpu().pin_memory(), z.cpu().pin_memory()
    u_h, q_h = torch.empty_like(u, device="cpu").pin_memory(), torch.empty_like(q, device="cpu").pin_memory()

    def host_pass():
        for l in range(layers):
            a.copy_(a_h, non_blocking=True)
            z.copy_(z_h, non_blocking=True)
            qf.project_pair(a, z, w_o[l], gain[l], w_q[l], u, q, eps, ws)
            u_h.copy_(u, non_blocking=True)
            q_h.copy_(q, non_blocking=True)
        torch.cuda.synchronize()

    host_pass()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        host_pass()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / args.steps

    weight_bytes = 2 * d_model * n_q * 2
    act_bytes = batch * (n_q * 4 + d_model * 2 + d_model * 2 + d_model * 2 + n_q * 2)   # a, z in; u' out and in again; q out
    pair_bytes = weight_bytes + act_bytes
    peak, peak_kind = hbm_peak()
    achieved = pair_bytes / (us_per_pair * 1e-6) / 1e9
    line = {
        "metric": "projection-pair weight and activation GB/s (cache-side W_o/W_q at a layer boundary)",
        "value": pair_bytes * layers / (ms_per_step * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "us_per_pair": us_per_pair,
        "us_per_pair_eager_launches": eager_us_per_pair, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"Qwen3-{args.shape.upper()}-shaped projection pair, {layers} layers with their own "
                               f"weights, batch {batch}", "d_model": d_model, "n_q": n_q, "seed": args.seed,
                   "l2": "weights of a pass (layers x pair) are far larger than L2, no flush needed"},
        "e2e": {"value": pair_bytes * layers / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": layers * batch * (n_q * 4 + d_model * 2),
                "d2h_bytes_per_step": layers * batch * (d_model * 2 + n_q * 2)},
        "gpu_launches": 2 * layers * args.steps,
        "roofline": {"bound": "hbm", "kernel": "proj_kernel (both stages of a pair)", "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "bytes_per_pair": pair_bytes, "traffic": None,
                     "note": "a pair is two dependent kernels; each waits for its weight stream (21 MB at the 4B shape: "
                             "3 us at peak, 4 to 7 us as a CTA's 64-80 KB requests land) and then spends about 2 us in "
                             "products, split-K exchange and epilogue, so the pair is bound by latency, not by HBM"},
    }
    if not args.no_cpu_baseline:
        from oracle import qf_oracle as orc
        orc.build()
        n_sample = min(layers, 2)
        a_n = a.cpu().numpy()
        z_n = z.view(torch.int16).cpu().numpy().view(np.uint16)
        t0 = time.perf_counter()
        for l in range(n_sample):
            orc.project_pair(a_n, z_n, w_o[l].view(torch.int16).cpu().numpy().view(np.uint16),
                             gain[l].view(torch.int16).cpu().numpy().view(np.uint16),
                             w_q[l].view(torch.int16).cpu().numpy().view(np.uint16), eps=eps)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": pair_bytes * n_sample / dt / 1e9, "unit": "GB/s", "cores": orc.num_threads(),
                                "kind": "oracle", "seconds": dt, "sample": f"{n_sample} of {layers} layer pairs"}
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
