"""The no-allocation gather entry point against the regular one (collected last on purpose).

aaf_kv_materialize_noalloc serves callers that may not call cudaMalloc (all device memory already
committed to their own pool, a path that cannot afford an allocation's synchronisation, code that
is only handed pointers).  Its scratch is a fixed array inside the library that every call on the
device shares and that keeps the previous call's contents, so the check runs different
requests back to back and compares each, byte for byte, with aaf_kv_materialize and with the CPU
oracle's materialize of the same context.
"""
from __future__ import annotations

import ctypes as C

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_noalloc_gather_matches_materialize_twice_in_a_row():
    import torch

    import __graft_entry__ as entry
    from paper_2607_10987_b200 import KVPool, binding
    from workloads import configs, fill

    from tests.helpers import OracleBackend

    entry.build()
    g = configs.Geometry(3, 8, 128, 16, 2, 512, 8, 128)
    seed = 424242
    pool = KVPool(g.n_layers, g.n_kv_heads, g.head_dim, g.block_size, g.elt_bytes, g.n_blocks, g.max_ctx,
                  g.max_blocks_per_ctx, free_order=configs.free_order(seed, g.n_blocks))
    cpu = OracleBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks))
    dev = pool.device
    fill.fill_torch(seed, 0, 0, g.pool_bytes // 2, dev, out=pool.pool.view(torch.int16))
    ctxs = []
    for stream_id, n in ((1, 1003), (2, 517)):
        buf = fill.fill_torch(seed, stream_id, 0, g.n_layers * 2 * n * g.row // 2, dev).view(torch.uint8)
        st, c = pool.imp(buf, n)
        assert st == 0
        assert cpu.imp(cpu.payload(seed, stream_id, n), n) == (0, c)
        ctxs.append((c, n))
    stream = C.c_void_p(torch.cuda.current_stream(dev).cuda_stream)

    def gather_noalloc(c, t0, t1):
        table = pool.table(c)  # host copy of the block table
        tab = (C.c_int32 * len(table))(*table.tolist())
        out = torch.full(((t1 - t0) * g.bpt,), 0xA5, dtype=torch.uint8, device=dev)
        st = binding.aaf_kv_materialize_noalloc(pool.pool.data_ptr(), g.layer_stride, g.n_layers, g.n_kv_heads,
                                                g.head_dim, g.block_size, g.elt_bytes, g.n_blocks, tab, len(table),
                                                t0, t1, out.data_ptr(), out.numel(), stream)
        return st, out

    # two calls in a row: a long range first, then a shorter, shifted one that must not see the
    # first call's leftovers in the shared scratch
    for c, t0, t1 in ((ctxs[0][0], 0, 1003), (ctxs[1][0], 21, 400), (ctxs[0][0], 999, 1003)):
        st, got = gather_noalloc(c, t0, t1)
        assert st == binding.AAF_OK
        st, want = pool.materialize(c, t0, t1)
        assert st == binding.AAF_OK
        torch.cuda.synchronize()
        assert torch.equal(got, want[: got.numel()]), (c, t0, t1)
        st, oracle_bytes = cpu.materialize(c, t0, t1)
        assert st == 0 and np.array_equal(got.cpu().numpy(), oracle_bytes), (c, t0, t1)

    # a pinned table is uploaded asynchronously: it may be overwritten only after the stream has run the call
    c, n = ctxs[1]
    table = pool.table(c)
    pinned = torch.from_numpy(table.copy()).pin_memory()
    out = torch.full((n * g.bpt,), 0x5A, dtype=torch.uint8, device=dev)
    st = binding.aaf_kv_materialize_noalloc(pool.pool.data_ptr(), g.layer_stride, g.n_layers, g.n_kv_heads,
                                            g.head_dim, g.block_size, g.elt_bytes, g.n_blocks,
                                            C.cast(pinned.data_ptr(), C.POINTER(C.c_int32)), len(table), 0, n,
                                            out.data_ptr(), out.numel(), stream)
    assert st == binding.AAF_OK
    torch.cuda.synchronize()
    pinned.fill_(-1)
    assert np.array_equal(out.cpu().numpy(), cpu.materialize(c, 0, n)[1])

    # beyond the built-in scratch: rejected with its own status, nothing launched
    big_blocks = binding.AAF_NOALLOC_MAX_BLOCKS + 1
    tab = (C.c_int32 * big_blocks)(*([0] * big_blocks))
    dst = torch.empty(16, dtype=torch.uint8, device=dev)
    st = binding.aaf_kv_materialize_noalloc(pool.pool.data_ptr(), g.layer_stride, g.n_layers, g.n_kv_heads,
                                            g.head_dim, g.block_size, g.elt_bytes, g.n_blocks, tab, big_blocks, 0,
                                            big_blocks * g.block_size, dst.data_ptr(), 1 << 62, stream)
    assert st == binding.AAF_ERR_SCRATCH_LIMIT
    assert "scratch" in binding.aaf_kv_strerror(st)
    # a table entry outside the pool is refused on the host
    bad = (C.c_int32 * 2)(0, g.n_blocks)
    st = binding.aaf_kv_materialize_noalloc(pool.pool.data_ptr(), g.layer_stride, g.n_layers, g.n_kv_heads,
                                            g.head_dim, g.block_size, g.elt_bytes, g.n_blocks, bad, 2, 0, 20,
                                            dst.data_ptr(), 1 << 62, stream)
    assert st == binding.AAF_ERR_INVALID_ARG
    assert pool.sync_status() == 0
