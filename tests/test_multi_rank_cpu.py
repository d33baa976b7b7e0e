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
        # the bench's estimate reduction: times only, no counts (nothing to sum: no collective for it)
        est, none = reduce_timings({"est": 1.0 + rank}, {}, dist, "cpu")
        assert est == {"est": float(world)} and none == {}
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


# ---- one request's cache split over ranks (Section 5): plumbing of the shard-state exchange
def _sharded_rank(rank, world, port, out_dir):
    from oracle import qf_oracle as orc
    from paper_2608_15473_b200.multi import gather_shard_states, local_shard_ranges, shard_slice
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lens = [1000, 37, 0, 513]
        S = 5                                                    # not a multiple of the world size
        w = wl.make_workload("split", lens, [wl.even_shards(L, S) for L in lens], 4, 2, seed=91)
        q = torch.from_numpy(w.q.view(np.uint8).copy())         # raw bytes of the bf16 query
        if rank != 0:
            q.zero_()
        dist.broadcast(q, src=0)                                 # only the query travels
        local = local_shard_ranges(torch.from_numpy(w.shard_ranges), S, world, rank).numpy()
        sh = orc.Shape(batch=w.batch, num_q_heads=4, num_kv_heads=2, max_pages_per_req=w.max_pages_per_req,
                       max_shards=local.shape[1])
        # the device-side sweep of this rank's shards (the CPU oracle stands in for the GPU here)
        o_loc, _, l_loc = orc.decode_partial(q.numpy().view(np.uint16).reshape(w.q.shape), w.k_cache, w.v_cache, w.block_table,
                                             w.seq_lens, np.ascontiguousarray(local), sh)
        o, lse = gather_shard_states(torch.from_numpy(o_loc), torch.from_numpy(l_loc), S, dist)
        if rank == 0:                                            # the owner merges
            sh_all = orc.Shape(batch=w.batch, num_q_heads=4, num_kv_heads=2,
                               max_pages_per_req=w.max_pages_per_req, max_shards=S)
            out, lse_out = orc.combine(o.numpy(), lse.numpy(), None, sh_all)
            ref_out, ref_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh_all)
            np.save(os.path.join(out_dir, "err.npy"),
                    np.array([np.abs(out - ref_out).max(),
                              np.abs(np.where(np.isneginf(ref_lse), 0, lse_out - ref_lse)).max(),
                              float(np.array_equal(np.isneginf(lse_out), np.isneginf(ref_lse))),
                              float(list(shard_slice(S, world, 0)) == [0, 1, 2]),
                              float(list(shard_slice(S, world, 1)) == [3, 4])]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_request_split_over_two_ranks_merges_to_the_unsplit_result(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_sharded_rank, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    err = np.load(tmp_path / "err.npy")
    assert err[0] < 1e-13 and err[1] < 1e-12 and err[2] == 1.0 and err[3] == 1.0 and err[4] == 1.0


def test_rank_sweep_params_tile_the_owners_shard_table():
    from paper_2608_15473_b200 import binding as qf
    from paper_2608_15473_b200 import multi
    p = qf.params(batch=3, num_q_heads=16, num_kv_heads=8, max_pages_per_req=64, max_shards=9, num_pages=512)
    for world in (1, 2, 3, 4, 9, 16):
        per = -(-9 // world)
        covered = []
        for rank in range(world):
            q = multi.rank_sweep_params(p, world, rank)
            assert (q.max_shards, q.out_shards, q.out_shard_offset) == (per, per * world, rank * per)
            assert q.batch == p.batch and q.num_pages == p.num_pages and p.out_shards == 0   # the original is untouched
            covered += list(range(q.out_shard_offset, q.out_shard_offset + q.max_shards))
            assert len(multi.shard_slice(9, world, rank)) <= per
        assert covered == list(range(per * world))
