"""Churn workload (config 5): seeded operator stream under memory pressure with LRU eviction,
block size swept over 8 / 16 / 32 / 64, CUDA library against the CPU oracle.

Both sides are driven by the same policy code (workloads.churn.ChurnDriver) with the same seed;
the driver reacts only to status codes, so the two call logs must be identical call by call --
including every out-of-blocks answer, which the library decides from a lower bound of the free
count that it refreshes from the device only when needed.
"""
from __future__ import annotations

import numpy as np
import pytest

from tests.helpers import GpuBackend, OracleBackend, check_conservation
from workloads import churn, configs
from workloads.configs import Geometry

pytestmark = pytest.mark.gpu

SEED = configs.SEED_BASE + 5


def demand_blocks(make_geometry, cap_tokens, bs, n_ops, **driver_kw):
    """peak live blocks of the trace on a pool that never runs out (the oracle, metadata only matters)"""
    g = make_geometry(64 * cap_tokens // bs)
    be = OracleBackend(g, SEED, init_fill=False)
    d = churn.ChurnDriver(be, SEED, max_ctx_tokens=cap_tokens, **driver_kw).run(n_ops)
    assert all(st == 0 for _, _, st in d.log), "the demand pass must never run out of blocks"
    return be.o.stats()["peak_live_blocks"]


def lockstep_churn(g, cap_tokens, n_ops, layers=None, snap_every=250, pool_every=1000, buf_every=7, **driver_kw):
    order = configs.free_order(SEED, g.n_blocks)
    layers = list(range(g.n_layers)) if layers is None else layers
    gpu = GpuBackend(g, SEED, free_order=order, init_fill=True, staging_tokens=cap_tokens)
    cpu = OracleBackend(g, SEED, layers=layers, free_order=order, init_fill=True)
    dg = churn.ChurnDriver(gpu, SEED, max_ctx_tokens=cap_tokens, **driver_kw)
    dc = churn.ChurnDriver(cpu, SEED, max_ctx_tokens=cap_tokens, **driver_kw)
    # remember the last materialised buffer of each side
    last = {}
    for name, be in (("g", gpu), ("c", cpu)):
        orig = be.materialize

        def wrapped(c, a, b, _orig=orig, _name=name):
            st, buf = _orig(c, a, b)
            last[_name] = (buf, b - a)
            return st, buf

        be.materialize = wrapped
    n_bufs = 0
    for i in range(n_ops):
        k = len(dc.log)
        dc.step()
        dg.step()
        assert dg.log[k:] == dc.log[k:], (i, dg.log[k:], dc.log[k:])
        if any(c == "materialize" for c, _, _ in dc.log[k:]):
            n_bufs += 1
            if n_bufs % buf_every == 0:
                (bg, n), (bc, _) = last["g"], last["c"]
                assert np.array_equal(gpu.buf_layers(bg, n, layers).reshape(-1), bc), i
        if (i + 1) % snap_every == 0:
            snap = cpu.snapshot()
            assert gpu.snapshot() == snap, i
            check_conservation(snap, g.n_blocks, g.block_size)
        if (i + 1) % pool_every == 0:
            assert np.array_equal(gpu.pool_layers(layers), cpu.o.pool_view()), i
    assert gpu.snapshot() == cpu.snapshot()
    assert np.array_equal(gpu.pool_layers(layers), cpu.o.pool_view())
    assert gpu.o.sync_status() == 0
    assert [s[:2] if s else None for s in dg.slots] == [s[:2] if s else None for s in dc.slots]
    gs, cs = gpu.o.stats(), cpu.o.stats()
    for key in ("free_blocks", "peak_live_blocks", "cow_count", "live_ctx"):
        assert gs[key] == cs[key]
    return dc, gs


@pytest.mark.parametrize("bs", [8, 16, 32, 64])
def test_full_trace_10000_ops_small_rows(bs):
    """The whole 10,000-operator trace with the workload's real lengths (median 2048, contexts up to
    32768 tokens); rows are 16 bytes so that the oracle keeps up -- tables, reference counts, free
    list, statuses and all bytes are compared."""
    cap = 32768
    make = lambda nb: Geometry(1, 1, 8, bs, 2, nb, 80, cap // bs)
    demand = demand_blocks(make, cap, bs, 10000)
    nb = int(0.75 * demand)
    d, stats = lockstep_churn(make(nb), cap, 10000)
    failed = [c for c, _, st in d.log if st == churn.OOM_BLOCKS]
    assert len(failed) > 20, "the capped pool must actually run out of blocks"
    assert stats["peak_live_blocks"] <= nb
    assert {"append", "fork", "compose", "materialize", "import", "evict"} <= set(d.counts)


@pytest.mark.parametrize("bs,n_ops", [(8, 1500), (16, 2500), (32, 1500), (64, 1500)])
def test_scaled_trace_8b_rows(bs, n_ops):
    """Llama-3-8B-shaped rows (2 KiB) and runs (16 / 32 / 64 / 128 KiB); lengths scaled down 8x so that
    the oracle finishes in seconds; every byte of both layers compared."""
    cap = 4096
    kw = dict(median_tokens=256.0, max_seg_tokens=2048)
    make = lambda nb: Geometry(2, 8, 128, bs, 2, nb, 80, cap // bs)
    demand = demand_blocks(lambda nb: Geometry(1, 1, 8, bs, 2, nb, 80, cap // bs), cap, bs, n_ops, **kw)
    nb = int(0.75 * demand)
    d, stats = lockstep_churn(make(nb), cap, n_ops, snap_every=100, pool_every=500, buf_every=3, **kw)
    assert any(st == churn.OOM_BLOCKS for _, _, st in d.log)
