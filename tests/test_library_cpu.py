"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its
host-side validation answers without a device."""
from __future__ import annotations

import ctypes as C
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2607_10987_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "aaf_kv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aaf_kv_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 20
    lib = C.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/aaf_kv.h but not exported"
    assert sorted(binding.SYMBOLS) == names, "the Python binding must mirror the header one to one"


def test_descriptor_struct_sizes_match_header_layout():
    assert C.sizeof(binding.aaf_kv_pool_desc) == 104
    assert C.sizeof(binding.aaf_kv_xfer_desc) == 48
    assert C.sizeof(binding.aaf_kv_stats) == 48 + 32 + 8 + 32 + 32


def test_workspace_size_and_geometry_validation():
    d = binding.make_desc(32, 8, 128, 16, 2, 32768, 64, 4096)
    ws = binding.aaf_kv_pool_workspace_bytes(d)
    assert 1 << 20 < ws < 64 << 20
    bad = binding.make_desc(32, 8, 3, 16, 2, 32768, 64, 4096)  # row = 48 is fine; 8*3*1 = 24 is not
    assert binding.aaf_kv_pool_workspace_bytes(bad) > 0
    bad = binding.make_desc(32, 8, 3, 16, 1, 32768, 64, 4096)
    assert binding.aaf_kv_pool_workspace_bytes(bad) == 0
    bad = binding.make_desc(0, 8, 128, 16, 2, 32768, 64, 4096)
    assert binding.aaf_kv_pool_workspace_bytes(bad) == 0
    bad = binding.make_desc(32, 8, 128, 16, 2, 32768, 64, 4096)
    bad.abi_version = 99
    assert binding.aaf_kv_pool_workspace_bytes(bad) == 0


def test_create_rejects_bad_arguments_before_touching_a_device():
    d = binding.make_desc(2, 2, 64, 16, 2, 256, 16, 128)
    out = C.c_void_p()
    assert binding.aaf_kv_pool_create(d, out) == binding.AAF_ERR_INVALID_ARG  # null pool / workspace
    d.pool_base, d.layer_stride_bytes = 0x1000, 256 * 2 * 16 * 256
    d.workspace, d.workspace_bytes = 0x100000, 16  # too small
    assert binding.aaf_kv_pool_create(d, out) == binding.AAF_ERR_INVALID_ARG
    d.workspace_bytes = binding.aaf_kv_pool_workspace_bytes(d)
    d.pool_base = 0x1008  # misaligned
    assert binding.aaf_kv_pool_create(d, out) == binding.AAF_ERR_INVALID_ARG
    d.pool_base = 0x1000
    order = (C.c_int32 * 256)(*([0] * 256))  # not a permutation
    d.free_order = order
    assert binding.aaf_kv_pool_create(d, out) == binding.AAF_ERR_INVALID_ARG
    assert out.value is None


def test_strerror_names_every_status():
    seen = {binding.aaf_kv_strerror(s) for s in range(0, -13, -1)}
    assert len(seen) == 13 and "unknown status" not in seen
    assert binding.aaf_kv_strerror(-99) == "unknown status"


def test_null_pool_is_rejected():
    assert binding.aaf_kv_evict(None, 1, (C.c_int32 * 1)(0), None) == binding.AAF_ERR_INVALID_ARG
    assert binding.aaf_kv_sync_status(None) == binding.AAF_ERR_INVALID_ARG
    one = (C.c_int32 * 2)(0, 1)
    assert binding.aaf_kv_compose_batch(None, 1, one, one, 0, one, None) == binding.AAF_ERR_INVALID_ARG
    assert binding.aaf_kv_materialize_batch(None, 1, one, None, None, None, None, None, None) == \
        binding.AAF_ERR_INVALID_ARG
    assert binding.aaf_kv_import_batch(None, 1, None, None, one, None) == binding.AAF_ERR_INVALID_ARG
    assert binding.aaf_kv_append_host(None, 1, one, one, None, None, 0, None) == binding.AAF_ERR_INVALID_ARG
