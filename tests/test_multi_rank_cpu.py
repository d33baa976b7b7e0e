"""The N > 1 path on CPU: two gloo ranks.  Requests shard over ranks with no data-path collective;
the only communication is the max/sum reduction of the benchmark's timings and work counts."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_15473_b200 import workloads as wl
from paper_2608_15473_b200.multi import reduce_timings, whole_job_throughput


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank draws its own batch (seed + rank), as bench.py does
        w = wl.config3(seed=rank, batch=3, hi=3000)
        own = wl.split_requests(10, world, rank)
        times, counts = reduce_timings({"elapsed": 10.0 + 5.0 * rank, "e2e": 30.0 - rank},
                                       {"bytes": float(w.algorithmic_bytes()), "tokens": float(w.swept_tokens())},
                                       dist, "cpu")
        np.save(os.path.join(out_dir, f"r{rank}.npy"),
                np.array([times["elapsed"], times["e2e"], counts["bytes"], counts["tokens"],
                          float(w.algorithmic_bytes()), float(w.swept_tokens()), own.start, own.stop]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_reduce_timings_and_counts(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0 = np.load(tmp_path / "r0.npy")
    r1 = np.load(tmp_path / "r1.npy")
    # both ranks see the same reduced values: max of times, sum of counts
    assert np.array_equal(r0[:4], r1[:4])
    assert r0[0] == 15.0 and r0[1] == 30.0
    assert r0[2] == r0[4] + r1[4] and r0[3] == r0[5] + r1[5]
    assert r0[4] != r1[4]                      # the ranks really hold different batches
    # whole-job value: all ranks' bytes over the slowest rank's time
    assert whole_job_throughput(r0[2], 15.0) == pytest.approx(r0[2] / 15e-3 / 1e9)
    # the request split is a partition of 0..9
    assert (r0[6], r0[7], r1[6], r1[7]) == (0, 5, 5, 10)


def test_split_requests_is_a_partition():
    for n in (0, 1, 7, 32, 33):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                seen += list(wl.split_requests(n, world, r))
            assert seen == list(range(n))
            sizes = [len(wl.split_requests(n, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def test_single_process_reduction_is_identity():
    t, c = reduce_timings({"a": 1.5}, {"b": 2.0}, None)
    assert t == {"a": 1.5} and c == {"b": 2.0}
