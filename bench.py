#!/usr/bin/env python
"""Benchmark of the Q-First cache-side decode path on B200.

A step is one pass of the whole hot path over one batch of synthetic input:
the sweep kernel (plan, stream, warp merge: shard states or segments of them), the finish kernel
(merges the shards that the schedule cut into segments) and the combine kernel.  The default
workload is the Qwen3-4B-shaped batched decode (32 requests, 32 q / 8 kv heads,
ragged contexts in [1,024, 36,480], 16-token pages in a shuffled block table,
4,096-token shards), the configuration the headline metric is quoted on.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 3] [--impl reference]
                  [--split-request] [--no-also]

Prints ONE JSON line (rank 0).  The K steps are timed R >= 7 times (enough repeats for about 0.4 s of
load); `ms_per_step` is the median repeat, and the line carries the spread and every repeat's median SM
clock, so that a reader can tell the kernel from the clock.  At N = 1 the line also carries, under
`also`, the other configurations (the one-million-token split-KV workload with its identity table and
with a shuffled one, the two other batched workloads, the single short request cold and warm), each
with its own roofline, clocks and whole-workload parity against the CPU oracle.

With N > 1 (launched by torch.distributed.run) every rank sweeps its own batch of requests; requests are
independent, so there is no data-path collective and scaling is weak.  With --split-request the N ranks
instead hold slices of ONE request's cache (the one-million-token workload): only the query is
broadcast, every rank sweeps its own shards straight into the owner's shard-state arrays through
peer-mapped memory, and the owner merges (strong scaling).
"""
from __future__ import annotations

import argparse
import json
import math
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
# dram__bytes_read.sum + dram__bytes_write.sum of one sweep-kernel launch, from the committed ncu summaries
# (seed 0; see profiles/)
NCU_TRAFFIC_BYTES = {3: 2013157000 + 5919744, 4: 4295357184 + 508416, 2: 1208430080 + 2514688, 5: 8382518784 + 7926272}
FALLBACK_HBM_GBS = 6650.0
DATASHEET_HBM_GBS = 8000.0
TARGET_LOAD_MS = 400.0       # the timed region of a workload lasts about this long (R repeats of K steps)
MIN_REPEATS, MAX_REPEATS = 7, 200


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


def config_record(args, w, world):
    """The `config` object of the JSON line: the same for the CUDA arm and the reference arm."""
    return {"workload": workload_name(args.workload), "seed": args.seed, "requests_per_gpu": w.batch,
            "cached_tokens_per_gpu": w.total_tokens, "num_pages": w.num_pages,
            "l2": "inputs larger than L2 (KV bytes per step >> 126 MB), no flush needed",
            "parallelism": f"requests sharded over {world} GPU(s), no collective",
            "kv_layout": "[page, Hkv, 16, D]" if args.kv_layout == "hnd" else "[page, 16, Hkv, D]"}


class ClockSampler:
    """Samples the SM clock and the clock-event reasons while the timed regions run: through NVML every
    couple of milliseconds when the binding is there (reads only), else through nvidia-smi every 100 ms."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index, uuid=None):
        self.gpu_index = gpu_index
        self.samples = []            # (host time, SM MHz)
        self.reasons = set()
        self.max_mhz = None
        self.power_w = []
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None
        self._handle = None
        try:
            import pynvml
            pynvml.nvmlInit()
            h = None
            if uuid:
                for u in (f"GPU-{uuid}", str(uuid)):
                    try:
                        h = pynvml.nvmlDeviceGetHandleByUUID(u.encode() if isinstance(u, str) else u)
                        break
                    except Exception:
                        h = None
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(int(gpu_index))
            self._nvml, self._handle = pynvml, h
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nvml = None

    def _run_nvml(self):
        nv, h = self._nvml, self._handle
        names = (("hw_slowdown", nv.nvmlClocksThrottleReasonHwSlowdown),
                 ("hw_thermal_slowdown", nv.nvmlClocksThrottleReasonHwThermalSlowdown),
                 ("sw_thermal_slowdown", nv.nvmlClocksThrottleReasonSwThermalSlowdown),
                 ("sw_power_cap", nv.nvmlClocksThrottleReasonSwPowerCap),
                 ("hw_power_brake_slowdown", nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown))
        k = 0
        while not self._stop.is_set():
            try:
                self.samples.append((time.perf_counter(), float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))))
                if k % 8 == 0:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                    for name, bit in names:
                        if r & bit:
                            self.reasons.add(name)
                    self.power_w.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
            except Exception:
                pass
            k += 1
            self._stop.wait(0.002)

    def _run_smi(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.gpu_index)], capture_output=True, text=True, timeout=5).stdout
                for line in out.strip().splitlines():
                    r = [x.strip() for x in line.split(",")]
                    self.samples.append((time.perf_counter(), float(r[1])))
                    self.max_mhz = max(self.max_mhz or 0.0, float(r[2]))
                    self.power_w.append(float(r[3]))
                    for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                        if v.lower().startswith("active"):
                            self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._thread = threading.Thread(target=self._run_nvml if self._nvml else self._run_smi, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thread.join(timeout=6)

    def window(self, t0, t1):
        """Median SM MHz of the samples taken in [t0, t1] (the nearest sample if none fell inside)."""
        inside = [m for t, m in self.samples if t0 <= t <= t1]
        if inside:
            return float(np.median(inside))
        if not self.samples:
            return None
        mid = 0.5 * (t0 + t1)
        return float(min(self.samples, key=lambda s: abs(s[0] - mid))[1])

    def summary(self, windows):
        """Clock record over the given host-time windows (the timed regions)."""
        mhz = [m for t, m in self.samples if any(a <= t <= b for a, b in windows)]
        if not mhz:
            mhz = [m for _, m in self.samples]
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(mhz),
                "power_w_max": max(self.power_w) if self.power_w else None,
                "source": "nvml" if self._nvml else "nvidia-smi"}


def sweep_kernel_bytes(w) -> int:
    """Algorithmic bytes of ONE sweep-kernel launch: K and V of every swept token, the block-table
    entries of its pages, q, and the shard states it writes ((D+2) fp32 per shard and query head)."""
    D = w.head_dim
    tok = w.swept_tokens()
    n_sh = int(w.shard_counts.astype(np.int64).sum())
    return (tok * 2 * w.num_kv_heads * D * 2 + 4 * ((tok + w.page_size - 1) // w.page_size) +
            w.batch * w.num_q_heads * D * 2 + n_sh * w.num_q_heads * (D + 2) * 4)


def oracle_pass(w, orc, sample_requests=None, results=None):
    """The CPU oracle over (a sample of) the workload: shard states, then the merge.  `results`, a dict, receives
    the shard states and the merged result of a whole-workload pass."""
    sh = orc.Shape(batch=w.batch, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads,
                   max_pages_per_req=w.max_pages_per_req, max_shards=w.max_shards)
    if sample_requests is None:
        t0 = time.perf_counter()
        op, mp, lp = orc.decode_partial(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh)
        merged = orc.combine(op, lp, w.shard_counts, sh)
        dt = time.perf_counter() - t0
        if results is not None:
            results.update(o_part=op, m_part=mp, lse_part=lp, out=merged[0], lse=merged[1])
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
        "config": config_record(args, w, args.gpus),
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "kv_tokens_per_s": ntok * args.steps / total,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- timing
def n_repeats(est_ms_per_step: float, steps: int) -> int:
    return int(min(MAX_REPEATS, max(MIN_REPEATS, math.ceil(TARGET_LOAD_MS / max(1e-3, est_ms_per_step * steps)))))


def time_repeats(step_fn, steps: int, repeats: int, stream, barrier, clocks):
    """R repeats of K steps, each bracketed by a CUDA-event pair on the launching stream and a synchronise on
    both sides.  Returns per-repeat ms per step, per-repeat median SM MHz and the host-time windows."""
    import torch
    ms, windows = [], []
    for _ in range(repeats):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.perf_counter()
        a.record(stream)
        for _ in range(steps):
            step_fn()
        b.record(stream)
        barrier()
        t1 = time.perf_counter()
        ms.append(a.elapsed_time(b) / steps)
        windows.append((t0, t1))
    mhz = [clocks.window(t0, t1) for t0, t1 in windows] if clocks is not None else [None] * repeats
    return ms, mhz, windows


def spread(ms, mhz):
    """Median, extremes and the per-repeat record of a list of per-step times."""
    order = np.argsort(ms)
    med = float(np.median(ms))
    rec = {"what": "per-step time of each repeat of the K steps (CUDA events; max over ranks for the median)",
           "median_ms": med, "min_ms": float(np.min(ms)), "max_ms": float(np.max(ms)),
           "p10_ms": float(np.percentile(ms, 10)), "p90_ms": float(np.percentile(ms, 90)), "repeats": len(ms),
           "per_repeat_ms": [round(float(x), 5) for x in ms],
           "per_repeat_sm_mhz": [None if x is None else round(float(x), 1) for x in mhz]}
    good = [(t, c) for t, c in zip(ms, mhz) if c]
    if len(good) >= 3:
        # time x clock of a repeat: flat if the spread is the clock's, varying if it is the kernel's
        tc = [t * c for t, c in good]
        rec["ms_x_mhz_median"] = float(np.median(tc))
        rec["ms_x_mhz_rel_spread"] = float((np.max(tc) - np.min(tc)) / np.median(tc))
        if np.std([c for _, c in good]) > 0:
            rec["corr_ms_vs_mhz"] = float(np.corrcoef([t for t, _ in good], [c for _, c in good])[0, 1])
    rec["fastest_repeat_sm_mhz"] = rec["per_repeat_sm_mhz"][int(order[0])]
    rec["slowest_repeat_sm_mhz"] = rec["per_repeat_sm_mhz"][int(order[-1])]
    return rec


def parity_against_oracle(dw, ref):
    """Every element of every output of the timed configuration against the oracle's whole-workload pass."""
    import torch
    torch.cuda.synchronize()
    out = {}
    for name in ("o_part", "m_part", "lse_part", "out", "lse"):
        got = getattr(dw, name).detach().cpu().numpy().astype(np.float64)
        want = ref[name]
        if name in ("o_part", "out"):
            out["max_abs_" + name] = float(np.abs(got - want).max())
        else:
            fin = np.isfinite(want)
            out["max_rel_" + name] = (float((np.abs(got[fin] - want[fin]) / np.maximum(1.0, np.abs(want[fin]))).max())
                                      if fin.any() else 0.0)
            out["inf_pattern_" + name] = bool(np.array_equal(np.isfinite(got), fin))
    out["tolerance"] = {"out_max_abs": 2e-3, "lse_rel": 1e-5}
    out["ok"] = bool(out["max_abs_o_part"] <= 2e-3 and out["max_abs_out"] <= 2e-3 and out["max_rel_m_part"] <= 1e-5 and
                     out["max_rel_lse_part"] <= 1e-5 and out["max_rel_lse"] <= 1e-5 and out["inf_pattern_lse"] and
                     out["inf_pattern_lse_part"] and out["inf_pattern_m_part"])
    out["against"] = "the CPU oracle over the whole workload: every shard state and every merged output"
    return out


def measure_workload(w, dw, steps, warmup, stream, barrier, clocks, qf, reduce=None, profile_mode=False):
    """Device-resident timing of one workload: R repeats of K whole passes, then the sweep kernel alone."""
    import torch
    for _ in range(max(3, warmup)):
        dw.step()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    a.record(stream)
    for _ in range(3):
        dw.step()
    b.record(stream)
    barrier()
    est = a.elapsed_time(b) / 3
    if reduce is not None:
        est = reduce({"est": est})["est"]
    repeats = 1 if profile_mode else n_repeats(est, steps)
    ms, mhz, windows = time_repeats(dw.step, steps, repeats, stream, barrier, clocks)
    # the dominant kernel alone: K more steps with an event pair recorded by the library right around each
    # sweep-kernel launch (kept out of the regions above: two event records per step cost ~10 us)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for x, y in ev:  # create the underlying handles so the library can re-record them
        x.record(stream)
        y.record(stream)
    barrier()
    t0 = time.perf_counter()
    for x, y in ev:
        qf.set_profile_events(x.cuda_event, y.cuda_event)
        dw.step()
    qf.set_profile_events(None, None)
    barrier()
    windows.append((t0, time.perf_counter()))
    sweep = [x.elapsed_time(y) for x, y in ev]
    return ms, mhz, windows, float(np.median(sweep)), float(np.min(sweep))


def roofline_record(w, sweep_ms, peak, peak_kind, traffic):
    kbytes = sweep_kernel_bytes(w)
    achieved = kbytes / (sweep_ms * 1e-3) / 1e9
    return {"bound": "hbm", "kernel": "sweep_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
            "frac_of_datasheet_8TBs": achieved / DATASHEET_HBM_GBS,
            "ms_per_launch": sweep_ms, "bytes_per_launch": kbytes, "traffic": traffic,
            "note": "kernel timed by an event pair around each launch (median over K launches) in a separate K-step region"}


def also_entry(idx, w, dw, label, plain, args, stream, barrier, gpu_id, uuid, qf, orc, peak, peak_kind):
    """One more configuration in the same run: timing, roofline, clocks, whole-workload parity.  `plain`: the
    configuration as the benchmark spec states it (the committed ncu traffic figure belongs to that form only)."""
    launches = dw.step()
    with ClockSampler(gpu_id, uuid) as clocks:
        ms, mhz, windows, sweep_ms, _ = measure_workload(w, dw, args.steps, args.warmup, stream, barrier, clocks, qf)
    sp = spread(ms, mhz)
    nbytes = w.algorithmic_bytes()
    gbs = nbytes / (sp["median_ms"] * 1e-3) / 1e9
    rec = {"workload": label, "seed": args.seed, "ms_per_step": sp["median_ms"], "GB/s": gbs,
           "pct_of_hbm_peak": 100.0 * gbs / DATASHEET_HBM_GBS, "pct_of_measured_copy": 100.0 * gbs / peak,
           "kv_tokens_per_s": w.swept_tokens() / (sp["median_ms"] * 1e-3), "launches_per_step": launches,
           "timing": sp, "clocks": clocks.summary(windows),
           "roofline": roofline_record(w, sweep_ms, peak, peak_kind,
                                       NCU_TRAFFIC_BYTES.get(idx) if (args.seed == 0 and plain) else None)}
    if orc is not None:
        ref = {}
        dt, nb, ntok = oracle_pass(w, orc, results=ref)
        dw.poison_outputs()
        dw.step()
        rec["parity"] = parity_against_oracle(dw, ref)
        rec["cpu_baseline"] = {"value": nb / dt / 1e9, "unit": "GB/s", "cores": orc.num_threads(), "kind": "oracle",
                               "seconds": dt, "sample": f"the whole workload once: {w.batch} requests, {ntok} cached tokens"}
    return rec


def small_request_latency(args, qf, wl, DeviceWorkload, device, stream, barrier, orc):
    """cfg1 (one request of 4,096 tokens: 16.8 MB, 2.6 us at the copy rate, so launch-bound): latency per pass,
    warm (one pool, served from L2) and cold (nine distinct pools of 16.8 MB visited in turn, 151 MB > L2),
    launched one by one and replayed from a CUDA graph."""
    import torch
    n_pools = 9
    ws = [wl.config1(seed=args.seed + i) for i in range(n_pools)]
    dws = [DeviceWorkload(w, device=device) for w in ws]
    launches = dws[0].step()
    for d in dws:
        d.step()
    torch.cuda.synchronize()
    rec = {"workload": workload_name(1), "seed": args.seed, "launches_per_step": launches,
           "bytes_per_step": ws[0].algorithmic_bytes(),
           "note": "latency per pass; warm = one pool (L2-resident), cold = nine pools in turn (151 MB > L2); "
                   "eager = launched call by call, graph = nine passes captured once and replayed"}

    def timed(fn, calls_per_fn, reps=30):
        for _ in range(3):
            fn()
        out = []
        for _ in range(7):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            a.record(stream)
            for _ in range(reps):
                fn()
            b.record(stream)
            barrier()
            out.append(1e3 * a.elapsed_time(b) / (reps * calls_per_fn))
        return {"median_us": float(np.median(out)), "min_us": float(np.min(out)), "max_us": float(np.max(out))}

    def cold_eager():
        for d in dws:
            d.step()

    def warm_eager():
        for _ in range(n_pools):
            dws[0].step()

    rec["warm_eager"] = timed(warm_eager, n_pools)
    rec["cold_eager"] = timed(cold_eager, n_pools)
    side = torch.cuda.Stream(device=device)
    graphs = {}
    for name, fn in (("warm_graph", lambda s: [dws[0].step(s) for _ in range(n_pools)]),
                     ("cold_graph", lambda s: [d.step(s) for d in dws])):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                fn(side)
        graphs[name] = g
    torch.cuda.synchronize()
    for name, g in graphs.items():
        rec[name] = timed(g.replay, n_pools)
    med = rec["cold_graph"]["median_us"]
    rec["ms_per_step"] = med * 1e-3
    rec["GB/s"] = ws[0].algorithmic_bytes() / (med * 1e-6) / 1e9
    if orc is not None:
        ref = {}
        oracle_pass(ws[0], orc, results=ref)
        dws[0].poison_outputs()
        dws[0].step()
        rec["parity"] = parity_against_oracle(dws[0], ref)
    return rec


def run_split_request(args, dist, rank, world, local_rank, device):
    """--split-request: ONE request's cache (the one-million-token workload, 16 shards) split over the N ranks.
    Every rank draws the same seeded workload on its host and uploads only the pages of the shards it owns; a
    step is query broadcast -> every rank's sweep into the owner's shard-state arrays (peer-mapped, plain stores)
    -> stream barrier -> merge on the owner.  Total work is fixed as N grows: strong scaling."""
    import torch
    from paper_2608_15473_b200 import workloads as wl
    from paper_2608_15473_b200.multi import reduce_timings, whole_job_throughput
    from paper_2608_15473_b200.split_request import SplitPlan, cuda_runner

    w = wl.config4(seed=args.seed)
    plan = SplitPlan(world=world, rank=rank, max_shards=w.max_shards)
    runner, out, lse, dw = cuda_runner(w, plan, dist, device, transport=args.split_transport)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        runner.step()
    barrier()
    assert dw.status() == 0
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(3):
        runner.step()
    b.record(stream)
    barrier()
    est = reduce_timings({"est": a.elapsed_time(b) / 3}, {}, dist, device)[0]["est"]
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    gpu_id = vis.split(",")[local_rank].strip() if vis and local_rank < len(vis.split(",")) else str(local_rank)
    try:
        uuid = str(torch.cuda.get_device_properties(device).uuid)
    except Exception:
        uuid = None
    with ClockSampler(gpu_id, uuid) as clocks:
        ms, mhz, windows = time_repeats(runner.step, args.steps, n_repeats(est, args.steps), stream, barrier, clocks)
    timing = spread(ms, mhz)
    local_tokens = float(dw.w.swept_tokens())
    times, counts = reduce_timings({"step": timing["median_ms"]}, {"tokens": local_tokens}, dist, device)
    if rank == 0:
        peak, peak_kind = measured_peaks()
        ms_per_step = times["step"]
        total_bytes = float(w.algorithmic_bytes())
        value = whole_job_throughput(total_bytes, ms_per_step)
        B, Hq, D = w.batch, w.num_q_heads, w.head_dim
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(4) + f", the cache split over {world} GPU(s)", "seed": args.seed,
                       "shards_per_gpu": plan.per_rank, "cached_tokens_total": w.total_tokens,
                       "l2": "inputs larger than L2 (each rank's KV slice >> 126 MB), no flush needed",
                       "parallelism": f"one request's KV shards over {world} GPU(s); query broadcast, shard states "
                                      f"{'stored into the owner arrays through peer-mapped memory' if args.split_transport == 'parked' else 'all-gathered'}, "
                                      "merge on the owner",
                       "transport": args.split_transport},
            "timing": timing, "clocks": clocks.summary(windows),
            "gpu_launches": 4 * args.steps,
            "exchange": {"query_bytes_out_per_rank": B * Hq * D * 2,
                         "state_bytes_back_per_rank": B * plan.per_rank * Hq * (D + 2) * 4,
                         "kv_bytes_moved": 0},
            "kv_tokens_per_s": counts["tokens"] / (ms_per_step * 1e-3),
            "pct_of_hbm_peak": 100.0 * value / (DATASHEET_HBM_GBS * world),
            "pct_of_measured_copy": 100.0 * value / (peak * world),
        }
        if not args.no_cpu_baseline:
            from oracle import qf_oracle as orc
            orc.build()
            sh = orc.Shape(batch=w.batch, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads,
                           max_pages_per_req=w.max_pages_per_req, max_shards=w.max_shards)
            t0 = time.perf_counter()
            ref_out, ref_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
            dt = time.perf_counter() - t0
            got_out, got_lse = out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
            line["parity"] = {"max_abs_out": float(np.abs(got_out - ref_out).max()),
                              "max_rel_lse": float((np.abs(got_lse - ref_lse) / np.maximum(1.0, np.abs(ref_lse))).max()),
                              "tolerance": {"out_max_abs": 2e-3, "lse_rel": 1e-5},
                              "against": "the CPU oracle's unsharded sweep of the whole request"}
            line["cpu_baseline"] = {"value": total_bytes / dt / 1e9, "unit": "GB/s", "cores": orc.num_threads(),
                                    "kind": "oracle", "seconds": dt, "sample": "the whole request once, unsharded"}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_cuda(args):
    import torch
    from paper_2608_15473_b200 import binding as qf
    from paper_2608_15473_b200 import build as qf_build
    from paper_2608_15473_b200 import workloads as wl
    from paper_2608_15473_b200.multi import reduce_timings, whole_job_throughput
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
    if args.split_request:
        return run_split_request(args, dist, rank, world, local_rank, device)

    # every rank owns its own batch of requests (weak scaling): seed + rank
    w = wl.CONFIGS[args.workload](seed=args.seed + rank)
    dw = DeviceWorkload(w, device=device, flags=qf.QF_FLAG_KV_NHD if args.kv_layout == "nhd" else 0)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def reduce_max(d):
        return reduce_timings(d, {}, dist, device)[0]

    # ---- correctness guard (cheap): the timed configuration produces finite results, clean status
    launches_per_step = dw.step()
    torch.cuda.synchronize()
    assert dw.status() == 0 and bool(torch.isfinite(dw.out).all())

    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    gpu_id = vis.split(",")[local_rank].strip() if vis and local_rank < len(vis.split(",")) else str(local_rank)
    try:
        uuid = str(torch.cuda.get_device_properties(device).uuid)
    except Exception:
        uuid = None

    # ---- device-resident timing: R repeats of K steps, CUDA events on the launching stream
    with ClockSampler(gpu_id, uuid) as clocks:
        ms, mhz, windows, sweep_ms, sweep_min_ms = measure_workload(
            w, dw, args.steps, args.warmup, stream, barrier, clocks, qf, reduce=reduce_max if dist is not None else None,
            profile_mode=args.profile_mode)
    timing = spread(ms, mhz)

    # ---- end to end through the host-buffer entry point: q + metadata in, out + lse back
    hs = HostStepper(dw)
    for _ in range(0 if args.profile_mode else 3):
        hs.step()
    e2e = []
    for _ in range(1 if args.profile_mode else MIN_REPEATS):
        barrier()
        t0 = time.perf_counter()
        for _ in range(1 if args.profile_mode else args.steps):
            hs.step()       # synchronises the stream before returning
        e2e.append((time.perf_counter() - t0) * 1e3 / (1 if args.profile_mode else args.steps))
    e2e_sync_ms = float(np.median(e2e))
    # ... and pipelined (qf_host_pipe_*): two steps in flight, every step still brings its own query in from pinned
    # host memory and its result back; the transfers ride under the previous and the next sweep
    from paper_2608_15473_b200.runtime import HostPipeline
    pipe = HostPipeline(dw, depth=2)
    e2e_pipe = []
    for rep in range(1 if args.profile_mode else MIN_REPEATS + 1):
        n = 1 if args.profile_mode else args.steps
        barrier()
        t0 = time.perf_counter()
        tickets = [pipe.submit() for _ in range(n)]
        pipe.wait(tickets[-1])
        dt = (time.perf_counter() - t0) * 1e3 / n
        if rep > 0 or args.profile_mode:      # the first repeat warms the pipe up
            e2e_pipe.append(dt)
    pipe.close()
    e2e_ms_step = float(np.median(e2e_pipe))

    times, counts = reduce_timings({"step": timing["median_ms"], "e2e": e2e_ms_step, "sweep": sweep_ms},
                                   {"bytes": float(w.algorithmic_bytes()), "tokens": float(w.swept_tokens())},
                                   dist, device)
    ms_per_step, e2e_ms = times["step"], times["e2e"]
    tot_bytes, tot_tokens = counts["bytes"], counts["tokens"]

    if rank == 0:
        peak, peak_kind = measured_peaks()
        value = whole_job_throughput(tot_bytes, ms_per_step)
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_record(args, w, world),
            "timing": timing,
            "clocks": clocks.summary(windows),
            "e2e": {"value": whole_job_throughput(tot_bytes, e2e_ms), "unit": "GB/s",
                    "h2d_bytes_per_step": hs.h2d_bytes, "d2h_bytes_per_step": hs.d2h_bytes,
                    "ms_per_step": e2e_ms, "min_ms_per_step": float(np.min(e2e_pipe)), "max_ms_per_step": float(np.max(e2e_pipe)),
                    "synchronous_ms_per_step": e2e_sync_ms, "synchronous_min_ms": float(np.min(e2e)),
                    "note": "qf_host_pipe_* with pinned host buffers, two steps in flight: every step copies its query "
                            "and metadata host -> device and its out and lse device -> host inside the timed region; "
                            "the copies run on transfer streams under the neighbouring sweeps.  synchronous_ms_per_step "
                            "is qf_decode_step_host, one step at a time (submit, wait, next): the latency of a step.  "
                            "The KV cache stays resident (only the query travels)"},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline_record(w, sweep_ms, peak, peak_kind,
                                        args.ncu_traffic if args.ncu_traffic is not None else
                                        (NCU_TRAFFIC_BYTES.get(args.workload) if args.seed == 0 else None)),
            "kv_tokens_per_s": tot_tokens / (ms_per_step * 1e-3),
            # the benchmark spec's target is a share of the part's peak HBM bandwidth: the 8 TB/s datasheet figure;
            # the measured copy rate (read + write, 6.5 TB/s) is a rate this read-mostly sweep can exceed
            "pct_of_hbm_peak": 100.0 * value / (DATASHEET_HBM_GBS * world),
            "pct_of_measured_copy": 100.0 * value / (peak * world),
            "sweep_kernel_pct_of_hbm_peak": 100.0 * sweep_kernel_bytes(w) / (sweep_ms * 1e-3) / 1e9 / DATASHEET_HBM_GBS,
        }
        line["roofline"]["min_ms_per_launch"] = sweep_min_ms
        orc = None
        if not args.no_cpu_baseline and not args.profile_mode and world == 1:
            from oracle import qf_oracle as orc
            orc.build()
            ref = {}
            dt, nb, ntok = oracle_pass(w, orc, results=ref)
            # the oracle's pass is here anyway: what the timed configuration computed, against it
            dw.poison_outputs()
            dw.step()
            line["parity"] = parity_against_oracle(dw, ref)
            cores = orc.num_threads()
            line["cpu_baseline"] = {"value": nb / dt / 1e9, "unit": "GB/s", "cores": cores,
                                    "kind": "oracle", "seconds": dt,
                                    "sample": f"the whole workload once: {w.batch} requests, {ntok} cached tokens, "
                                              "partials + combine"}
            # and on one thread: the first requests of the workload, about ten seconds' worth
            orc.set_num_threads(1)
            try:
                cum = np.cumsum(w.seq_lens.astype(np.int64))
                per_tok = dt * cores / max(1, ntok)            # rough: perfect scaling assumed for sizing only
                n1 = int(max(1, np.searchsorted(cum, 10.0 / max(per_tok, 1e-12), side="right")))
                n1 = min(n1, w.batch)
                dt1, nb1, ntok1 = oracle_pass(w, orc, sample_requests=None if n1 == w.batch else n1)
            finally:
                orc.set_num_threads(cores)
            line["cpu_baseline"]["single_thread"] = {
                "value": nb1 / dt1 / 1e9, "unit": "GB/s", "cores": 1, "seconds": dt1,
                "sample": f"the first {n1} of {w.batch} requests ({ntok1} cached tokens), all shards and heads"}
        if not args.no_also and not args.profile_mode and world == 1 and args.workload == 3 and args.kv_layout == "hnd":
            del hs
            also = []
            plan = [(4, {}, workload_name(4), True), (4, {"table": "shuffled"}, workload_name(4) + " (shuffled table)", False),
                    (2, {}, workload_name(2), True), (5, {}, workload_name(5), True),
                    (3, {"flags": qf.QF_FLAG_KV_NHD}, workload_name(3) + " (token-major pages [page, 16, Hkv, D])", False)]
            dw = None
            torch.cuda.empty_cache()
            for idx, kw, label, plain in plan:
                try:
                    kw = dict(kw)
                    flags2 = kw.pop("flags", 0)
                    w2 = wl.CONFIGS[idx](seed=args.seed, **kw)
                    dw2 = DeviceWorkload(w2, device=device, flags=flags2)
                    also.append(also_entry(idx, w2, dw2, label, plain, args, stream, barrier, gpu_id, uuid, qf, orc, peak, peak_kind))
                except Exception as ex:  # one configuration failing must not take the headline line with it
                    also.append({"workload": label, "error": f"{type(ex).__name__}: {ex}"})
                dw2 = w2 = None
                torch.cuda.empty_cache()
            try:
                also.append(small_request_latency(args, qf, wl, DeviceWorkload, device, stream, barrier, orc))
            except Exception as ex:
                also.append({"workload": workload_name(1), "error": f"{type(ex).__name__}: {ex}"})
            line["also"] = also
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", type=int, default=3, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--kv-layout", default="hnd", choices=["hnd", "nhd"],
                    help="page layout of the KV pools: head-major (default, the headline) or token-major")
    ap.add_argument("--split-request", action="store_true",
                    help="N ranks hold slices of ONE request's cache (the one-million-token workload) and write "
                         "their shard states into the owner's arrays through peer-mapped memory (strong scaling)")
    ap.add_argument("--split-transport", default="parked", choices=["parked", "gather"],
                    help="with --split-request: shard states stored straight into the owner's arrays (default) or all-gathered")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="time the headline configuration only")
    ap.add_argument("--profile-mode", action="store_true",
                    help="for runs under a profiler: one repeat, one end-to-end step, no CPU baseline, no other configurations")
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
