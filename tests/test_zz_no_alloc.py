"""qf_decode_partial_static: the sweep for callers that cannot allocate device memory.

Some users of the library have no allocator on the decode path (a memory pool frozen at
start-up, an operator plugin that only sees its own tensors, a point in the step where
cudaMalloc must not be called because it can stall the whole device).  For them the
library carries a fixed 8 MiB scratch array of its own.  This test drives that entry point
through the C ABI and checks it against the ordinary qf_decode_partial, twice in a row:
the second call finds the first call's leftovers in the shared array and must not be
disturbed by them.

The file name makes pytest collect it last, so a run that stops at the first failure has
already been through every other test.
"""
import pytest
import torch

from paper_2608_15473_b200 import binding as qf
from paper_2608_15473_b200 import build as qf_build
from paper_2608_15473_b200 import workloads as wl
from paper_2608_15473_b200.runtime import DeviceWorkload

import qf_testlib as T

pytestmark = pytest.mark.gpu


def test_static_scratch_sweep_matches_the_ordinary_entry_point_twice():
    qf_build.build()
    # first workload: ragged, several shards, segments split across SMs
    w1 = wl.config3(seed=3, batch=6, hi=9000)
    # second workload: different shape and group size, so the array holds stale, differently laid out data
    w2 = wl.make_workload("na2", [5000, 77, 0, 1300], [wl.fixed_shards(L, 700) for L in (5000, 77, 0, 1300)],
                          4, 2, seed=9, poison_tails=True)
    for w in (w1, w2):
        dw = DeviceWorkload(w)
        assert qf.workspace_bytes(dw.params) <= qf.QF_STATIC_SCRATCH_BYTES
        dw.poison_outputs()
        dw.sweep()                                    # the existing entry point, caller-provided workspace
        ref = [t.clone() for t in (dw.o_part, dw.m_part, dw.lse_part)]
        for _ in range(2):                            # two calls in a row on the shared array
            dw.poison_outputs()
            qf.decode_partial_static(dw.q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                     dw.shard_ranges, dw.o_part, dw.m_part, dw.lse_part, dw.params)
            torch.cuda.synchronize()
            # the same kernels on the same inputs: the same bits (the tolerance of the other GPU tests, 2e-3 on
            # outputs and 1e-5 on log-sum-exp against the oracle, is checked right after)
            for got, want in zip((dw.o_part, dw.m_part, dw.lse_part), ref):
                assert torch.equal(got, want)
            assert qf.static_scratch_status() == 0
            # and the merged result agrees with the CPU oracle
            dw.merge()
            T.compare_all(dw, w)


def test_static_scratch_rejects_problems_beyond_its_size():
    qf_build.build()
    big = qf.params(batch=4096, num_q_heads=32, num_kv_heads=8, max_pages_per_req=64, max_shards=8, num_pages=1 << 18)
    assert qf.workspace_bytes(big) > qf.QF_STATIC_SCRATCH_BYTES
    a = 0x10000  # never dereferenced: the size check comes first
    rc = qf.decode_partial_static(a, a, a, None, a, a, a, a, a, big, stream=0, check=False)
    assert rc == qf.QF_ERR_STATIC_SCRATCH
    with pytest.raises(qf.QFError, match="needs .* bytes of scratch"):
        qf.decode_partial_static(a, a, a, None, a, a, a, a, a, big, stream=0)
    # invalid parameters get the ordinary entry point's own error code
    bad = qf.params(batch=2, num_q_heads=16, num_kv_heads=8, max_pages_per_req=8, max_shards=2, num_pages=16, head_dim=64)
    assert qf.decode_partial_static(a, a, a, None, a, a, a, a, a, bad, stream=0, check=False) == qf.QF_ERR_UNSUPPORTED
