"""One request's cache split over ranks (Section 5), on the CPU: the slicing of a workload into per-rank pools and
tables, and the per-step control flow (query broadcast, every rank's sweep into its slots of the owner's arrays,
barrier, merge on the owner) over two gloo ranks, with the CPU checker standing in for the CUDA sweep and merge.
The owner's arrays are a shared-memory tensor here, as they are peer-mapped device memory on GPUs."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import qf_oracle as orc
from paper_2608_15473_b200 import workloads as wl
from paper_2608_15473_b200.split_request import SplitPlan, SplitRequestRunner, rank_workload


def _shape(w):
    return orc.Shape(batch=w.batch, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads,
                     max_pages_per_req=w.max_pages_per_req, max_shards=w.max_shards)


def _workload():
    # ragged requests, unaligned shard boundaries (boundary pages are held by two ranks), an empty request,
    # fewer shards than slots
    lens = [5000, 777, 0, 130, 2049]
    S = 5
    ranges = [wl.even_shards(L, S) for L in lens]
    ranges[1] = [(0, 100), (100, 777), (0, 0), (0, 0), (0, 0)]
    return wl.make_workload("split-cpu", lens, ranges, 8, 4, seed=61, pool_factor=1.3, poison_unused=True,
                            poison_tails=True, shard_counts=[5, 2, 5, 5, 5])


@pytest.mark.parametrize("world", [1, 2, 3, 4, 7])
def test_rank_workloads_hold_only_their_pages_and_reproduce_the_whole(world):
    w = _workload()
    ref_o, ref_m, ref_l = orc.decode_partial(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, _shape(w))
    ref_out, ref_lse = orc.combine(ref_o, ref_l, w.shard_counts, _shape(w))
    plan0 = SplitPlan(world, 0, w.max_shards)
    St = plan0.padded_shards
    o_all = np.full((w.batch, St, w.num_q_heads, 128), np.nan)
    l_all = np.full((w.batch, St, w.num_q_heads), np.nan)
    pages_held = 0
    for r in range(world):
        plan = SplitPlan(world, r, w.max_shards)
        wr = rank_workload(w, plan)
        pages_held += wr.num_pages
        assert wr.max_shards == plan.per_rank and wr.shard_ranges.shape == (w.batch, plan.per_rank, 2)
        # the table points only into the rank's own pool
        used = wr.block_table[wr.block_table >= 0]
        assert used.size == 0 or used.max() < wr.num_pages
        o, m, l = orc.decode_partial(wr.q, wr.k_cache, wr.v_cache, wr.block_table, wr.seq_lens, wr.shard_ranges, _shape(wr))
        sl = plan.slots()
        # bit for bit the whole workload's shard states: same tokens, same order of every sum
        assert np.array_equal(o[:, :len(sl)], ref_o[:, sl.start:sl.stop])
        assert np.array_equal(l[:, :len(sl)], ref_l[:, sl.start:sl.stop])
        assert np.isneginf(l[:, len(sl):]).all()
        o_all[:, plan.out_offset:plan.out_offset + plan.per_rank] = o
        l_all[:, plan.out_offset:plan.out_offset + plan.per_rank] = l
    sh = _shape(w)
    sh.max_shards = St
    out, lse = orc.combine(o_all, l_all, None, sh)
    full_out, full_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, _shape(w))
    # request 1 counts only two of its shards, and they tile it
    assert np.allclose(out, full_out, rtol=0, atol=1e-12) and np.allclose(lse[np.isfinite(full_lse)], full_lse[np.isfinite(full_lse)], rtol=1e-13)
    assert np.allclose(out, ref_out, rtol=0, atol=1e-12)
    # nobody holds the whole cache once it is split (boundary pages may be held twice)
    total_pages = int(((w.seq_lens.astype(np.int64) + 15) // 16).sum())
    if world > 1:
        assert max(rank_workload(w, SplitPlan(world, r, w.max_shards)).num_pages for r in range(world)) < total_pages
    assert pages_held <= total_pages + 2 * world * w.batch


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, transport, owner_arrays, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = _workload()
        plan = SplitPlan(world, rank, w.max_shards)
        wr = rank_workload(w, plan)
        St, per = plan.padded_shards, plan.per_rank
        # only the owner knows the query; the others start from zeros and must receive it
        q = torch.from_numpy(w.q.view(np.int16).copy())
        if rank != plan.owner:
            q.zero_()
        result = {}

        def sweep(qt, o, m, l):
            qbits = qt.numpy().view(np.uint16)
            po, pm, pl = orc.decode_partial(qbits, wr.k_cache, wr.v_cache, wr.block_table, wr.seq_lens, wr.shard_ranges,
                                            _shape(wr))
            if transport == "parked":   # this rank's slots of the owner's arrays, nothing else
                lo = plan.out_offset
                o[:, lo:lo + per] = torch.from_numpy(po)
                m[:, lo:lo + per] = torch.from_numpy(pm)
                l[:, lo:lo + per] = torch.from_numpy(pl)
            else:
                o.copy_(torch.from_numpy(po)); m.copy_(torch.from_numpy(pm)); l.copy_(torch.from_numpy(pl))

        def merge(o, l):
            sh = _shape(w)
            sh.max_shards = St
            result["out"], result["lse"] = orc.combine(o.numpy(), l.numpy(), None, sh)

        if transport == "parked":
            runner = SplitRequestRunner(plan, dist, q, sweep, merge, owner_arrays=owner_arrays, transport="parked")
        else:
            B, Hq = w.batch, w.num_q_heads
            local = [torch.zeros((B, per, Hq, 128), dtype=torch.float64), torch.zeros((B, per, Hq), dtype=torch.float64),
                     torch.zeros((B, per, Hq), dtype=torch.float64)]
            runner = SplitRequestRunner(plan, dist, q, sweep, merge, local_arrays=local, transport="gather")
        for _ in range(2):      # two steps: the second finds the first's states in the arrays
            runner.step()
        if rank == plan.owner:
            np.save(os.path.join(out_dir, "out.npy"), result["out"])
            np.save(os.path.join(out_dir, "lse.npy"), result["lse"])
        else:
            assert "out" not in result            # only the owner merges
            assert np.array_equal(q.numpy().view(np.uint16), w.q)     # the query did arrive
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("transport", ["parked", "gather"])
def test_two_ranks_step_and_the_owner_merges(tmp_path, transport):
    world, port = 2, _free_port()
    w = _workload()
    plan = SplitPlan(world, 0, w.max_shards)
    B, Hq, St = w.batch, w.num_q_heads, plan.padded_shards
    owner_arrays = [torch.full((B, St, Hq, 128), float("nan"), dtype=torch.float64).share_memory_(),
                    torch.full((B, St, Hq), float("nan"), dtype=torch.float64).share_memory_(),
                    torch.full((B, St, Hq), float("nan"), dtype=torch.float64).share_memory_()]
    mp.spawn(_rank_main, args=(world, port, transport, owner_arrays, str(tmp_path)), nprocs=world, join=True)
    out, lse = np.load(tmp_path / "out.npy"), np.load(tmp_path / "lse.npy")
    ref_o, ref_m, ref_l = orc.decode_partial(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, _shape(w))
    # every shard is merged here (the padded table has no per-request counts): compare with all five shards
    ref_out, ref_lse = orc.combine(ref_o, ref_l, None, _shape(w))
    assert np.allclose(out, ref_out, rtol=0, atol=1e-12)
    fin = np.isfinite(ref_lse)
    assert np.array_equal(np.isfinite(lse), fin) and np.allclose(lse[fin], ref_lse[fin], rtol=1e-13)
    if transport == "parked":
        # every slot of the owner's arrays was written by exactly the rank that owns it
        got_l = owner_arrays[2].numpy()
        for r in range(world):
            p = SplitPlan(world, r, w.max_shards)
            sl = p.slots()
            assert np.array_equal(got_l[:, p.out_offset:p.out_offset + len(sl)], ref_l[:, sl.start:sl.stop])
            assert np.isneginf(got_l[:, p.out_offset + len(sl):p.out_offset + p.per_rank]).all()
