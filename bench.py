#!/usr/bin/env python
"""Benchmark of the Q-First cache-side decode path on B200.

A step is one pass of the whole hot path over one batch of synthetic input:
the sweep kernel (plan, stream, warp merge: shard states or segments of them), the finish kernel
(merges the shards that the schedule cut into segments) and the combine kernel.  The default
workload is the Qwen3-4B-shaped batched decode (32 requests, 32 q / 8 kv heads,
ragged contexts in [1,024, 36,480], 16-token pages in a shuffled block table,
4,096-token shards), the configuration the headline metric is quoted on.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 3] [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run)
every rank sweeps its own batch of requests; requests are independent, so there
is no data-path collective and scaling is weak.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "decode-attention KV GB/s and % of B200 HBM peak (Qwen3-4B shape, batched)"
# dram__bytes_read.sum + dram__bytes_write.sum of one sweep-kernel launch, from the committed ncu summaries of
# the Qwen3-4B-shaped and one-million-token workloads (seed 0)
NCU_TRAFFIC_BYTES = {3: 2013151000 + 5875456, 4: 4295394816 + 605952}
FALLBACK_HBM_GBS = 6650.0
DATASHEET_HBM_GBS = 8000.0


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def workload_name(idx: int) -> str:
    return {1: "cfg1 Qwen3-0.6B-shaped single request, 4,096 tokens, 1 shard",
            2: "cfg2 Qwen3-0.6B-shaped batch 64 x 4,608 tokens, 4 shards, shuffled pages",
            3: "cfg3 Qwen3-4B-shaped batch 32, ragged 1,024-36,480 tokens, 4,096-token shards, shuffled pages",
            4: "cfg4 one-million-token split-KV, 16 shards of 65,536, planted logits near 85",
            5: "cfg5 Qwen3-4B-shaped mixed batch 256, log-uniform 512-32,768 tokens, 1-8 shards, fragmented pool"}[idx]


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.rows = []
        self._stop = threading.Event()
        self._thread = None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.gpu_index)], capture_output=True, text=True, timeout=5).stdout
                for line in out.strip().splitlines():
                    self.rows.append([x.strip() for x in line.split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thread.join(timeout=6)

    def summary(self):
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def sweep_kernel_bytes(w) -> int:
    """Algorithmic bytes of ONE sweep-kernel launch: K and V of every swept token, the block-table
    entries of its pages, q, and the shard states it writes ((D+2) fp32 per shard and query head)."""
    D = w.head_dim
    tok = w.swept_tokens()
    n_sh = int(w.shard_counts.astype(np.int64).sum())
    return (tok * 2 * w.num_kv_heads * D * 2 + 4 * ((tok + w.page_size - 1) // w.page_size) +
            w.batch * w.num_q_heads * D * 2 + n_sh * w.num_q_heads * (D + 2) * 4)


def oracle_pass(w, orc, sample_requests=None, results=None):
    """The CPU oracle over (a sample of) the workload: shard states, then the merge.  `results`, a list, receives
    the merged (out, lse) of a whole-workload pass."""
    sh = orc.Shape(batch=w.batch, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads,
                   max_pages_per_req=w.max_pages_per_req, max_shards=w.max_shards)
    if sample_requests is None:
        t0 = time.perf_counter()
        op, mp, lp = orc.decode_partial(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh)
        merged = orc.combine(op, lp, w.shard_counts, sh)
        dt = time.perf_counter() - t0
        if results is not None:
            results.extend(merged[:2])
        return dt, w.algorithmic_bytes(), w.swept_tokens()
    # bounded sample: the first n requests (all their shards and heads)
    n = sample_requests
    sh.batch = n
    t0 = time.perf_counter()
    op, mp, lp = orc.decode_partial(w.q[:n], w.k_cache, w.v_cache, w.block_table[:n], w.seq_lens[:n],
                                    w.shard_ranges[:n], sh)
    orc.combine(op, lp, w.shard_counts[:n], sh)
    dt = time.perf_counter() - t0
    frac = float(w.seq_lens[:n].astype(np.int64).sum()) / max(1, w.total_tokens)
    return dt, int(w.algorithmic_bytes() * frac), int(w.seq_lens[:n].astype(np.int64).sum())


def run_reference(args):
    """--impl reference: the fp64 CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import qf_oracle as orc
    from paper_2608_15473_b200 import workloads as wl
    orc.build()
    w = wl.CONFIGS[args.workload](seed=args.seed)
    cores = orc.num_threads()
    # size the per-step sample so the whole run stays within a few minutes
    t_probe, _, tok_probe = oracle_pass(w, orc, sample_requests=1)
    per_tok = t_probe / max(1, tok_probe)
    budget_s = 120.0 / max(1, args.steps + args.warmup)
    n_req = w.batch
    cum = np.cumsum(w.seq_lens.astype(np.int64))
    while n_req > 1 and cum[n_req - 1] * per_tok > budget_s:
        n_req -= 1
    for _ in range(args.warmup):
        oracle_pass(w, orc, sample_requests=n_req)
    times, nbytes, ntok = [], 0, 0
    for _ in range(args.steps):
        dt, nbytes, ntok = oracle_pass(w, orc, sample_requests=n_req)
        times.append(dt)
    total = float(sum(times))
    value = nbytes * args.steps / total / 1e9
    sample = f"first {n_req} of {w.batch} requests ({ntok} cached tokens), all shards and heads, partials + combine"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args.workload), "seed": args.seed, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "kv_tokens_per_s": ntok * args.steps / total,
    }
    print(json.dumps(line), flush=True)


def run_cuda(args):
    import torch
    from paper_2608_15473_b200 import binding as qf
    from paper_2608_15473_b200 import build as qf_build
    from paper_2608_15473_b200 import workloads as wl
    from paper_2608_15473_b200.runtime import DeviceWorkload, HostStepper

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path (use --impl reference for the oracle)")
    if rank == 0:
        qf_build.build()
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)

    # every rank owns its own batch of requests (weak scaling): seed + rank
    w = wl.CONFIGS[args.workload](seed=args.seed + rank)
    dw = DeviceWorkload(w, device=device, flags=qf.QF_FLAG_KV_NHD if args.kv_layout == "nhd" else 0)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- correctness guard (cheap): the timed configuration produces finite results, clean status
    launches_per_step = dw.step()
    torch.cuda.synchronize()
    assert dw.status() == 0 and bool(torch.isfinite(dw.out).all())

    for _ in range(max(0, args.warmup - 1)):
        dw.step()
    barrier()

    # ---- device-resident timing: K steps, CUDA events on the launching stream, nothing else in the region
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    gpu_id = vis.split(",")[local_rank].strip() if vis and local_rank < len(vis.split(",")) else str(local_rank)
    barrier()
    with ClockSampler(gpu_id) as clocks:
        t_start.record(stream)
        for _ in range(args.steps):
            dw.step()
        t_stop.record(stream)
        barrier()
        if not args.profile_mode and t_start.elapsed_time(t_stop) < 300.0:   # a few sampler readings under the same load
            t_end = time.perf_counter() + 0.5
            while time.perf_counter() < t_end:
                dw.step()
            torch.cuda.synchronize()
    elapsed_ms = t_start.elapsed_time(t_stop)

    # ---- the dominant kernel alone: K more steps with an event pair recorded by the library right around
    # each sweep-kernel launch (kept out of the region above: two event records per step cost ~10 us)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in ev:  # create the underlying handles so the library can re-record them
        a.record(stream)
        b.record(stream)
    barrier()
    for a, b in ev:
        qf.set_profile_events(a.cuda_event, b.cuda_event)
        dw.step()
    qf.set_profile_events(None, None)
    barrier()
    sweep_ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))

    # ---- end to end through the host-buffer entry point: q + metadata in, out + lse back
    hs = HostStepper(dw)
    e2e_steps = 1 if args.profile_mode else args.steps
    for _ in range(0 if args.profile_mode else 3):
        hs.step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        hs.step()       # synchronises the stream before returning
    e2e_s = (time.perf_counter() - t0) * args.steps / e2e_steps

    from paper_2608_15473_b200.multi import reduce_timings, whole_job_throughput
    times, counts = reduce_timings({"elapsed": elapsed_ms, "e2e": e2e_s * 1e3, "sweep": sweep_ms},
                                   {"bytes": float(w.algorithmic_bytes()), "tokens": float(w.swept_tokens())},
                                   dist, device)
    elapsed_ms, e2e_ms = times["elapsed"], times["e2e"]
    tot_bytes, tot_tokens = counts["bytes"], counts["tokens"]

    if rank == 0:
        peak, peak_kind = measured_peaks()
        ms_per_step = elapsed_ms / args.steps
        value = whole_job_throughput(tot_bytes, ms_per_step)
        kbytes = sweep_kernel_bytes(w)
        achieved = kbytes / (sweep_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(args.workload), "seed": args.seed, "requests_per_gpu": w.batch,
                       "cached_tokens_per_gpu": w.total_tokens, "num_pages": w.num_pages,
                       "l2": "inputs larger than L2 (KV bytes per step >> 126 MB), no flush needed",
                       "parallelism": f"requests sharded over {world} GPU(s), no collective",
                       "kv_layout": "[page, Hkv, 16, D]" if args.kv_layout == "hnd" else "[page, 16, Hkv, D]"},
            "clocks": clocks.summary(),
            "e2e": {"value": whole_job_throughput(tot_bytes, e2e_ms / args.steps), "unit": "GB/s",
                    "h2d_bytes_per_step": hs.h2d_bytes, "d2h_bytes_per_step": hs.d2h_bytes,
                    "ms_per_step": e2e_ms / args.steps,
                    "note": "qf_decode_step_host with pinned host buffers: a staging kernel reads q and the step "
                            "metadata from host memory and the merge kernel writes out and lse to host memory "
                            "(no copy-engine operations); the KV cache stays resident (only the query travels)"},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": {"bound": "hbm", "kernel": "sweep_kernel", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "frac_of_datasheet_8TBs": achieved / DATASHEET_HBM_GBS,
                         "ms_per_launch": sweep_ms, "bytes_per_launch": kbytes,
                         "traffic": args.ncu_traffic if args.ncu_traffic is not None else
                         (NCU_TRAFFIC_BYTES.get(args.workload) if args.seed == 0 else None),
                         "note": "kernel timed by an event pair around each launch in a second K-step region"},
            "kv_tokens_per_s": tot_tokens / (ms_per_step * 1e-3),
            "pct_of_hbm_peak": 100.0 * value / (peak * world),
        }
        if not args.no_cpu_baseline and not args.profile_mode and world == 1:
            from oracle import qf_oracle as orc
            orc.build()
            merged = []
            dt, nb, ntok = oracle_pass(w, orc, results=merged)
            # the oracle's pass is here anyway: what the timed configuration computed, against it
            ref_out, ref_lse = merged
            got_out, got_lse = dw.out.cpu().numpy().astype(np.float64), dw.lse.cpu().numpy().astype(np.float64)
            fin = np.isfinite(ref_lse)
            line["parity"] = {"max_abs_out": float(np.abs(got_out - ref_out).max()),
                              "max_rel_lse": float((np.abs(got_lse[fin] - ref_lse[fin]) /
                                                    np.maximum(1.0, np.abs(ref_lse[fin]))).max()) if fin.any() else 0.0,
                              "inf_pattern_matches": bool(np.array_equal(np.isfinite(got_lse), fin)),
                              "tolerance": {"out_max_abs": 2e-3, "lse_rel": 1e-5},
                              "against": "the CPU oracle's merged result over the whole workload (every request and head)"}
            line["cpu_baseline"] = {"value": nb / dt / 1e9, "unit": "GB/s", "cores": orc.num_threads(),
                                    "kind": "oracle", "seconds": dt,
                                    "sample": f"the whole workload once: {w.batch} requests, {ntok} cached tokens, "
                                              "partials + combine"}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", type=int, default=3, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--kv-layout", default="hnd", choices=["hnd", "nhd"],
                    help="page layout of the KV pools: head-major (default, the headline) or token-major")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-mode", action="store_true",
                    help="for runs under a profiler: no padding loop, one end-to-end step, no CPU baseline")
    ap.add_argument("--ncu-traffic", type=float, default=None,
                    help="DRAM bytes per sweep launch from an ncu capture (recorded in the roofline object)")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
