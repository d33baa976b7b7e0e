"""One request's cache split over devices (Section 5) on GPUs: the sweep of every rank's own pages, written into
its slots of the merging device's arrays, and the merge there.  On one GPU the ranks of a split run one after
another in this process (same code, same parameters, no peer mapping); with two or more GPUs a second test runs
real ranks as child processes over NCCL with the owner's arrays opened through CUDA IPC."""
import os
import socket

import numpy as np
import pytest
import torch

from oracle import qf_oracle as orc
from paper_2608_15473_b200 import binding as qf
from paper_2608_15473_b200 import build as qf_build
from paper_2608_15473_b200 import workloads as wl
from paper_2608_15473_b200.split_request import SplitPlan, SplitRequestRunner, cuda_runner, rank_workload

import qf_testlib as T

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    qf_build.build()


def workloads():
    lens = [40_000, 777, 0, 130, 9001]
    S = 6
    ragged = wl.make_workload("split-gpu", lens, [wl.even_shards(L, S) for L in lens], 16, 8, seed=67,
                              pool_factor=1.2, poison_unused=True, poison_tails=True)
    return [ragged, wl.config4(seed=3, ctx=1 << 16, n_shards=16, n_plant=400)]


@pytest.mark.parametrize("transport", ["parked", "gather"])
def test_one_rank_runs_the_whole_step(transport):
    for w in workloads():
        plan = SplitPlan(world=1, rank=0, max_shards=w.max_shards)
        runner, out, lse, dw = cuda_runner(w, plan, None, torch.device("cuda", 0), transport=transport)
        for _ in range(2):
            out.fill_(float("nan"))
            runner.step()
        torch.cuda.synchronize()
        ref_out, ref_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, T.oracle_shape(w))
        assert T.out_err(out.cpu().numpy(), ref_out) <= T.ENG_OUT and T.lse_err(lse.cpu().numpy(), ref_lse) <= T.ENG_LSE
        assert dw.status() == 0


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class _OneProcess:
    """Stands in for the process group when the ranks of a split run one after another in one process."""
    def broadcast(self, t, src=0):
        pass

    def all_reduce(self, t):
        pass


@pytest.mark.parametrize("world", [2, 3, 5])
def test_ranks_run_in_turn_on_one_gpu_each_with_only_its_pages(world):
    # every rank has its own pool (only its pages), its own table and workspace, and stores into its slots of one
    # set of arrays, as separate GPUs would through peer mappings; the merge runs once every rank has swept
    import copy
    dev = torch.device("cuda", 0)
    for w in workloads():
        B, Hq = w.batch, w.num_q_heads
        St = SplitPlan(world, 0, w.max_shards).padded_shards
        arrays = [torch.full((B, St, Hq, 128), 777.0, device=dev), torch.full((B, St, Hq), 777.0, device=dev),
                  torch.full((B, St, Hq), 777.0, device=dev)]
        out = torch.full((B, Hq, 128), float("nan"), device=dev)
        lse = torch.full((B, Hq), float("nan"), device=dev)
        from paper_2608_15473_b200.runtime import DeviceWorkload
        for rank in range(world):
            plan = SplitPlan(world, rank, w.max_shards)
            dw = DeviceWorkload(rank_workload(w, plan), device=dev)
            sp = copy.copy(dw.params)
            sp.out_shards, sp.out_shard_offset = St, plan.out_offset

            def sweep(q, o, m, l, dw=dw, sp=sp):
                qf.decode_partial(q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, dw.shard_ranges, o, m, l, sp,
                                  dw.workspace, dw.ws_bytes)

            def merge(o, l):
                raise AssertionError("the merge belongs to the last step of this emulation, run below")

            r = SplitRequestRunner(SplitPlan(world, rank, w.max_shards, owner=-1), _OneProcess(), dw.q, sweep, merge,
                                   owner_arrays=arrays, transport="parked")
            r.step()
            torch.cuda.synchronize()
            assert dw.status() == 0
        assert not (arrays[2] == 777.0).any()          # every slot written, padded ones with -inf
        pc = qf.params(B, Hq, w.num_kv_heads, w.max_pages_per_req, St, w.num_pages)
        qf.combine(arrays[0], arrays[2], None, out, lse, pc)
        torch.cuda.synchronize()
        sh = T.oracle_shape(w)
        ref_out, ref_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
        assert T.out_err(out.cpu().numpy(), ref_out) <= T.ENG_OUT and T.lse_err(lse.cpu().numpy(), ref_lse) <= T.ENG_LSE
        ref_o, ref_m, ref_l = orc.decode_partial(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh)
        got_o, got_l = arrays[0].cpu().numpy().astype(np.float64), arrays[2].cpu().numpy().astype(np.float64)
        for rank in range(world):
            p = SplitPlan(world, rank, w.max_shards)
            sl = p.slots()
            dst = slice(p.out_offset, p.out_offset + len(sl))
            assert T.out_err(got_o[:, dst], ref_o[:, sl.start:sl.stop]) <= T.ENG_OUT
            assert T.lse_err(got_l[:, dst], ref_l[:, sl.start:sl.stop]) <= T.ENG_LSE


def test_peer_access_call_on_the_same_device_is_a_no_op():
    assert qf.enable_peer_access(torch.cuda.current_device()) == qf.QF_OK
    assert qf.enable_peer_access(-1, check=False) == qf.QF_ERR_BAD_SHAPE


# ---- two PROCESSES on one GPU: everything of the real multi-rank path except NCCL and the cross-device hop.  The
# owner's arrays travel as CUDA IPC handles over the process group (gloo here) and are opened by the other process,
# whose sweep stores its shard states into them; no kernel of one process waits for a kernel of the other (the ranks
# meet in host-side collectives only), so sharing the GPU between the two is safe.
def _shared_gpu_rank(rank, world, port, out_dir):
    import datetime
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    dist.init_process_group("gloo", rank=rank, world_size=world, timeout=datetime.timedelta(seconds=120))
    try:
        for i, w in enumerate(workloads()):
            plan = SplitPlan(world, rank, w.max_shards)
            runner, out, lse, dw = cuda_runner(w, plan, dist, dev, transport="parked")
            if rank != plan.owner:
                dw.q.zero_()                      # only the owner holds the query: it must arrive by broadcast
                assert runner.owner_arrays[0].data_ptr() != 0
            for _ in range(3):
                runner.step()
            torch.cuda.synchronize()
            dist.barrier()
            assert dw.status() == 0
            if rank == plan.owner:
                np.save(os.path.join(out_dir, f"out{i}.npy"), out.cpu().numpy())
                np.save(os.path.join(out_dir, f"lse{i}.npy"), lse.cpu().numpy())
                np.save(os.path.join(out_dir, f"lpart{i}.npy"), runner.owner_arrays[2].cpu().numpy())
            dist.barrier()
            del runner
    finally:
        dist.destroy_process_group()


def test_two_processes_share_one_gpu_and_the_owners_arrays(tmp_path):
    import torch.multiprocessing as mp
    world = 2
    mp.spawn(_shared_gpu_rank, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for i, w in enumerate(workloads()):
        sh = T.oracle_shape(w)
        ref_out, ref_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, sh)
        assert T.out_err(np.load(tmp_path / f"out{i}.npy"), ref_out) <= T.ENG_OUT
        assert T.lse_err(np.load(tmp_path / f"lse{i}.npy"), ref_lse) <= T.ENG_LSE
        # the other process's slots of the owner's arrays hold its shards' states
        ref_o, ref_m, ref_l = orc.decode_partial(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.shard_ranges, sh)
        got_l = np.load(tmp_path / f"lpart{i}.npy").astype(np.float64)
        for r in range(world):
            p = SplitPlan(world, r, w.max_shards)
            sl = p.slots()
            assert T.lse_err(got_l[:, p.out_offset:p.out_offset + len(sl)], ref_l[:, sl.start:sl.stop]) <= T.ENG_LSE


# ---- real ranks, one per GPU (needs at least two)

def _gpu_rank(rank, world, port, transport, out_dir):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    os.environ.setdefault("NCCL_NVLS_ENABLE", "0")      # plain peer stores and rings only
    torch.cuda.set_device(rank)
    dev = torch.device("cuda", rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    try:
        for i, w in enumerate(workloads()):
            plan = SplitPlan(world, rank, w.max_shards)
            runner, out, lse, dw = cuda_runner(w, plan, dist, dev, transport=transport)
            if rank != plan.owner:
                dw.q.zero_()                      # only the owner holds the query: it must arrive by broadcast
            for _ in range(3):
                runner.step()
            torch.cuda.synchronize()
            dist.barrier()
            assert dw.status() == 0
            if rank == plan.owner:
                np.save(os.path.join(out_dir, f"out{i}.npy"), out.cpu().numpy())
                np.save(os.path.join(out_dir, f"lse{i}.npy"), lse.cpu().numpy())
            del runner
            dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("transport", ["parked", "gather"])
def test_two_gpus_split_one_request(tmp_path, transport):
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs")
    import torch.multiprocessing as mp
    world = 2
    mp.spawn(_gpu_rank, args=(world, _free_port(), transport, str(tmp_path)), nprocs=world, join=True)
    for i, w in enumerate(workloads()):
        ref_out, ref_lse = orc.decode_full(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, T.oracle_shape(w))
        assert T.out_err(np.load(tmp_path / f"out{i}.npy"), ref_out) <= T.ENG_OUT
        assert T.lse_err(np.load(tmp_path / f"lse{i}.npy"), ref_lse) <= T.ENG_LSE
