"""The C-ABI library: it loads, exports every symbol the header declares, and rejects bad
arguments before touching a device.  CPU only (no compute calls)."""
import ctypes
import re
from pathlib import Path

import pytest

from paper_2608_15473_b200 import binding as qf
from paper_2608_15473_b200 import build as qf_build

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module", autouse=True)
def built():
    qf_build.build()


def declared_functions():
    text = "".join(h.read_text() for h in sorted((ROOT / "include").glob("*.h")))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qf_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert sorted(qf.EXPORTS) == names
    L = qf.lib()
    for n in names:
        assert hasattr(L, n), n


def test_version_and_strerror():
    assert qf.version() == 100
    assert qf.strerror(0) == "ok"
    for code in (-1, -2, -3, -4, -5, -6):
        assert qf.strerror(code) and qf.strerror(code) != "unknown status"
    assert qf.strerror(-99) == "unknown status"


def good():
    return qf.params(batch=2, num_q_heads=16, num_kv_heads=8, max_pages_per_req=8, max_shards=2, num_pages=16)


def test_struct_layout_matches_header():
    assert ctypes.sizeof(qf.QFParams) == 56
    assert qf.QFParams.num_pages.offset == 32 and qf.QFParams.sm_scale.offset == 40
    assert qf.QFParams.out_shards.offset == 44 and qf.QFParams.out_shard_offset.offset == 48


def test_workspace_bytes():
    p = good()
    n = qf.workspace_bytes(p)
    assert n > 0 and n % 256 == 0
    assert qf.step_scratch_bytes(p) > n
    p.head_dim = 64
    assert qf.workspace_bytes(p) == 0 and qf.step_scratch_bytes(p) == 0


@pytest.mark.parametrize("field,value,code", [
    ("batch", 0, qf.QF_ERR_BAD_SHAPE),
    ("num_q_heads", 12, qf.QF_ERR_BAD_SHAPE),      # not a multiple of 8 KV heads
    ("max_shards", 0, qf.QF_ERR_BAD_SHAPE),
    ("num_pages", 0, qf.QF_ERR_BAD_SHAPE),
    ("head_dim", 64, qf.QF_ERR_UNSUPPORTED),
    ("page_size", 32, qf.QF_ERR_UNSUPPORTED),
    ("num_q_heads", 72, qf.QF_ERR_UNSUPPORTED),    # group of 9
    ("out_shards", 1, qf.QF_ERR_BAD_SHAPE),        # output table smaller than this call's two shards
    ("out_shard_offset", 1, qf.QF_ERR_BAD_SHAPE),  # an offset without an output table
    ("out_shards", -1, qf.QF_ERR_BAD_SHAPE),
])
def test_bad_params_are_rejected_before_any_launch(field, value, code):
    p = good()
    setattr(p, field, value)
    fake = 0x1000  # never dereferenced: validation fails first
    rc = qf.decode_partial(fake, fake, fake, fake, fake, fake, fake, fake, fake, p, fake, 1 << 30,
                           stream=0, check=False)
    assert rc == code
    rc = qf.combine(fake, fake, None, fake, fake, p, stream=0, check=False)
    assert rc == code
    with pytest.raises(qf.QFError):
        qf.combine(fake, fake, None, fake, fake, p, stream=0)


def test_null_pointers_and_workspace_checks():
    p = good()
    a = 0x10000
    args = [a] * 9
    for i in (0, 1, 2, 4, 5, 6, 7, 8):  # block_table (index 3) may be NULL
        bad = list(args)
        bad[i] = None
        assert qf.decode_partial(*bad, p, a, 1 << 30, stream=0, check=False) == qf.QF_ERR_NULL
    need = qf.workspace_bytes(p)
    assert qf.decode_partial(*args, p, None, need, stream=0, check=False) == qf.QF_ERR_WORKSPACE
    assert qf.decode_partial(*args, p, a + 8, need, stream=0, check=False) == qf.QF_ERR_WORKSPACE
    assert qf.decode_partial(*args, p, a, need - 1, stream=0, check=False) == qf.QF_ERR_WORKSPACE
    assert qf.combine(None, a, None, a, a, p, stream=0, check=False) == qf.QF_ERR_NULL
    assert qf.decode_step_host(None, a, a, None, a, a, None, a, a, p, a, 1 << 30, stream=0,
                               check=False) == qf.QF_ERR_NULL
    assert qf.decode_step_host(a, a, a, None, a, a, None, a, a, p, a, 16, stream=0,
                               check=False) == qf.QF_ERR_WORKSPACE


def test_no_device_is_a_loud_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    p = good()
    a = 0x10000
    rc = qf.combine(a, a, None, a, a, p, stream=0, check=False)
    assert rc in (qf.QF_ERR_CUDA, qf.QF_ERR_DEVICE)
    with pytest.raises(RuntimeError):
        from paper_2608_15473_b200.runtime import DeviceWorkload
        from paper_2608_15473_b200 import workloads as wl
        DeviceWorkload(wl.make_workload("x", [16], [[(0, 16)]], 2, 1))


def test_static_scratch_entry_rejects_without_touching_a_device():
    # invalid parameters and over-large problems are turned away before any device call
    p = good()
    p.head_dim = 64
    a = 0x10000
    assert qf.decode_partial_static(a, a, a, None, a, a, a, a, a, p, stream=0, check=False) == qf.QF_ERR_UNSUPPORTED
    p = good()
    p.batch = 0
    assert qf.decode_partial_static(a, a, a, None, a, a, a, a, a, p, stream=0, check=False) == qf.QF_ERR_BAD_SHAPE
    big = qf.params(batch=4096, num_q_heads=32, num_kv_heads=8, max_pages_per_req=64, max_shards=8, num_pages=1 << 18)
    assert qf.decode_partial_static(a, a, a, None, a, a, a, a, a, big, stream=0, check=False) == qf.QF_ERR_STATIC_SCRATCH


def test_peer_access_call_needs_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    assert qf.enable_peer_access(0, check=False) in (qf.QF_ERR_CUDA, qf.QF_ERR_DEVICE)
    with pytest.raises(qf.QFError):
        qf.enable_peer_access(1)
