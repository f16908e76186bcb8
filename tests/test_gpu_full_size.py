"""Parity at the full sizes of the workloads, in the launch configuration the benchmark times.

The GPU library runs the whole geometry; the CPU oracle runs the same operator list on a sample of
the layers (layers are independent and share block ids), which gives the exact tables, reference
counts and free list of the full geometry and the exact bytes of the sampled layers: every
materialised buffer and the final pool image of those layers are compared byte for byte.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

from tests.helpers import GpuBackend, check_conservation
from tests.test_gpu_parity import lockstep
from tests.value_check import ShadowBackend
from workloads import configs
from workloads.configs import Geometry
from workloads.replay import replay

pytestmark = pytest.mark.gpu


def _fits(g: Geometry, extra_gib: float) -> bool:
    import gc

    gc.collect()
    torch.cuda.empty_cache()  # memory cached by earlier tests must not make this one skip
    free_b, _ = torch.cuda.mem_get_info()
    return free_b > g.pool_bytes + extra_gib * 2**30


@pytest.mark.parametrize("unaligned", [False, True])
def test_config2_llama8b_full_pool(unaligned):
    g, seed, ops = configs.config2(unaligned)
    if not _fits(g, 12):
        pytest.skip("not enough free device memory for the 64 GiB pool")
    # unaligned variant: seeded pool image, last layer compared; literal variant: zero image, a middle layer
    # (every layer is compared, convention-free, by the value-model tests below)
    gpu, cpu = (lockstep(g, seed, ops, layers=[g.n_layers - 1]) if unaligned else
                lockstep(g, seed, ops, layers=[g.n_layers // 2], init_fill="zero"))
    st = gpu.o.stats()
    assert st["cow_count"] == (16 if unaligned else 0)
    assert st["live_blocks"] == (512 + 512 + 16 * 32 + (16 if unaligned else 0))


def test_config2_single_appends_give_the_same_state():
    g, seed, ops_b = configs.config2(True)
    _, _, ops_s = configs.config2(True, batched_append=False)
    small = Geometry(g.n_layers, g.n_kv_heads, g.head_dim, g.block_size, g.elt_bytes, 4096, g.max_ctx,
                     g.max_blocks_per_ctx)
    ga, _ = lockstep(small, seed, ops_b, layers=[7])
    snap_a, img_a = ga.snapshot(), ga.pool_layers([7])
    del ga
    gb, _ = lockstep(small, seed, ops_s, layers=[7])
    assert gb.snapshot() == snap_a
    assert np.array_equal(gb.pool_layers([7]), img_a)


@pytest.mark.parametrize("copy_all", [False, True])
def test_config3_compose_levels_8b(copy_all):
    g, seed, ops, lens = configs.config3(configs.LLAMA8B, copy_all=copy_all)
    if not _fits(g, 16):
        pytest.skip("not enough free device memory for the 64 GiB pool")
    gpu, cpu = lockstep(g, seed, ops, layers=[30] if copy_all else [3], init_fill="zero")
    assert gpu.o.ctx_len(gpu.o.live_ctxs()[-1]) == sum(lens)


@pytest.mark.parametrize("unaligned", [False, True])
def test_config4_llama70b(unaligned):
    g, seed, ops = configs.config4(unaligned)
    if not _fits(g, 40):
        pytest.skip("not enough free device memory for the 40 GiB pool plus 10 GiB buffers")
    gpu, cpu = lockstep(g, seed, ops, layers=[79] if unaligned else [0])
    assert gpu.o.stats()["cow_count"] == (8 if unaligned else 0)


def test_cow_stress_1024_children_8b_rows():
    g = Geometry(32, 8, 128, 16, 2, 4096, 1100, 1024)
    ops = configs.cow_stress_ops(context_tokens=8187, n_children=1024)
    gpu, cpu = lockstep(g, configs.SEED_BASE + 6, ops, layers=[0, 31], max_batch=1024)
    st = gpu.o.stats()
    assert st["cow_count"] == 1024
    assert st["live_blocks"] == 512 + 1024
    # one batched evict of all 1024 children (525 K table entries on 1.5 K blocks): the large-batch path
    # (release over a grid, compaction afterwards) must free the same blocks in the same order
    kids = [c for c in cpu.o.live_ctxs() if c != 0]
    assert len(kids) == 1024
    assert gpu.evict(kids)[0] == 0 and cpu.evict(kids)[0] == 0
    assert gpu.snapshot() == cpu.snapshot()
    assert gpu.o.stats()["live_blocks"] == 512
    assert gpu.evict([0])[0] == 0 and cpu.evict([0])[0] == 0
    assert gpu.snapshot() == cpu.snapshot() and gpu.o.sync_status() == 0
    assert sorted(gpu.o.free_list().tolist()) == list(range(g.n_blocks))


# ---------------------------------------------------------------------------------------------------------------
# Convention-free checks at full size, ALL layers: the value model (contexts are token sequences; no blocks, no
# reference counts, no free list) runs beside the library; every materialised buffer and, at the end, every live
# context is compared in every (layer, K/V) plane with bytes regenerated on the device from the fill function.
# These tests do not use the paged oracle: they hold whatever block ids the library hands out.  Reference-count
# conservation (refcount = number of table entries naming the block, free ring = exactly the unreferenced blocks)
# is recounted from the library's own tables.


def value_model_run(g, seed, ops, max_batch=0, staging_tokens=0):
    gpu = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), init_fill=False, max_batch=max_batch,
                     staging_tokens=staging_tokens)
    sh = ShadowBackend(gpu)
    n_bufs = 0
    for i, op, st, res, _ in replay(ops, sh, seed):
        assert st == 0, (i, op, st)
        if op["op"] == "materialize":
            sh.check_buffer(seed, res)
            n_bufs += 1
    sh.check_all_live(seed)
    check_conservation(gpu.snapshot(), g.n_blocks, g.block_size)
    assert gpu.o.sync_status() == 0
    return sh, n_bufs


def test_config2_llama8b_value_model_all_layers():
    g, seed, ops = configs.config2(True)
    if not _fits(g, 12):
        pytest.skip("not enough free device memory for the 64 GiB pool")
    sh, n_bufs = value_model_run(g, seed, ops)
    assert n_bufs == 18 and len(sh.vm.ctx) == 18
    assert sh.planes_checked == 64 * (n_bufs + 18)


@pytest.mark.parametrize("copy_all", [False, True])
def test_config3_compose_levels_value_model_all_layers(copy_all):
    g, seed, ops, lens = configs.config3(configs.LLAMA8B, copy_all=copy_all)
    if not _fits(g, 16):
        pytest.skip("not enough free device memory for the 64 GiB pool")
    sh, n_bufs = value_model_run(g, seed, ops)
    assert n_bufs == 2 and len(sh.vm.ctx) == 16 + 8 + 4 + 2
    # the tree and the flat composition are the same sequence
    assert sh.vm.ctx[max(sh.vm.ctx)] == sh.vm.ctx[max(sh.vm.ctx) - 1] and len(sh.vm.ctx[max(sh.vm.ctx)]) == sum(lens)


@pytest.mark.parametrize("copy_all", [False, True])
def test_config3_levels_as_batches_8b(copy_all):
    """The composition workload with every level issued as ONE batched call (8 pairs, 4 quads): tables, reference
    counts, free list, catalog and the bytes of the sampled layer equal the oracle's loop of single merges."""
    from tests.helpers import OracleBackend

    g, seed, ops, lens = configs.config3(configs.LLAMA8B, copy_all=copy_all)
    if not _fits(g, 16):
        pytest.skip("not enough free device memory for the 64 GiB pool")
    layers = [11]
    order = configs.free_order(seed, g.n_blocks)
    gpu = GpuBackend(g, seed, free_order=order, init_fill="zero")
    cpu = OracleBackend(g, seed, layers=layers, free_order=order, init_fill="zero")
    names = {}
    for o in (o for o in ops if o["op"] == "import"):
        for be in (gpu, cpu):
            st, c = be.imp(be.payload(seed, o["stream"], o["n"]), o["n"])
            assert st == 0
        names[o["out"]] = c
    for level in ("pairs", "quads", "all16", "flat16"):
        batch = [o for o in ops if o["op"] == "compose" and o["level"] == level]
        st, outs = gpu.o.compose_batch([[names[x] for x in o["segs"]] for o in batch], batch[0]["flags"])
        assert st == 0
        for o, c in zip(batch, outs):
            assert cpu.compose([names[x] for x in o["segs"]], o["flags"]) == (0, c)
            names[o["out"]] = c
        assert gpu.snapshot() == cpu.snapshot(), level
        assert gpu.o.catalog() == cpu.o.catalog(), level
    assert gpu.o.stats()["copy_launches"]["compose"] == 4
    assert np.array_equal(gpu.pool_layers(layers), cpu.o.pool_view())
    n = sum(lens)
    for name in ("all_tree", "all_flat"):
        got = gpu.buf_layers(gpu.materialize(names[name], 0, n)[1], n, layers).reshape(-1)
        assert np.array_equal(got, cpu.materialize(names[name], 0, n)[1])
    assert gpu.o.sync_status() == 0


def test_config2_host_buffer_path_value_model_all_layers():
    """The end-to-end form of the 8B step, as the benchmark times it: every input arrives from pinned host memory
    through the library's host-buffer calls (chunked import, chunked materialize, append from host buffers), on
    the full 64 GiB pool.  The bytes that come back to the host and every live context (all layers) are compared
    with what the value model says they must be."""
    import torch

    from tests.value_check import Paired

    g, seed, _ = configs.config2(True)
    if not _fits(g, 12):
        pytest.skip("not enough free device memory for the 64 GiB pool")
    T, agents, n_new = 8187, 16, 512
    gpu = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), init_fill=False)
    sh = ShadowBackend(gpu)
    pool, dev = gpu.o, gpu.o.device
    root = sh.payload(seed, 1, T)
    conts = [sh.payload(seed, 2 + i, n_new) for i in range(agents)]
    h_root = torch.empty(T * g.bpt, dtype=torch.uint8).pin_memory()
    h_root.copy_(root.dev)
    h_conts = [torch.empty(n_new * g.bpt, dtype=torch.uint8).pin_memory() for _ in conts]
    for h, c in zip(h_conts, conts):
        h.copy_(c.dev)
    h_out = torch.zeros(T * g.bpt, dtype=torch.uint8).pin_memory()
    d_root = torch.empty(T * g.bpt, dtype=torch.uint8, device=dev)
    d_conts = torch.empty(agents * n_new * g.bpt, dtype=torch.uint8, device=dev)
    staging = torch.empty(T * g.bpt, dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()
    for rnd in range(2):  # twice: the second round reuses every staging buffer while the first is still in flight
        st, c_root = pool.import_host_chunked(h_root, T, d_root, 1024)
        assert st == 0 and sh.vm.imp(root.tokens) == c_root
        st, _ = pool.materialize_host_chunked(c_root, 0, T, h_out, staging, 1024)
        assert st == 0
        st, c_recv = pool.imp(staging, T)
        assert st == 0 and sh.vm.imp(sh.vm.materialize(c_root, 0, T)) == c_recv
        st, kids = pool.fork(c_recv, agents)
        assert st == 0 and sh.vm.fork(c_recv, agents) == kids
        assert pool.append_host(kids, [n_new] * agents, h_conts, d_conts) == 0
        for k, c in zip(kids, conts):
            sh.vm.append(k, c.tokens)
        st, merged = pool.compose(kids[:2], 0)
        assert st == 0 and sh.vm.compose(kids[:2]) == merged
        if rnd == 0:
            everything = [c_root, c_recv] + kids + [merged]
            assert pool.evict(everything)[0] == 0
            sh.vm.evict(everything)
    torch.cuda.synchronize()
    assert torch.equal(h_out, h_root)
    sh.check_buffer(seed, Paired(h_out.to(dev), root.tokens))
    sh.check_all_live(seed)
    check_conservation(gpu.snapshot(), g.n_blocks, g.block_size)
    assert pool.sync_status() == 0 and pool.stats()["cow_count"] == 2 * agents


def test_suffix_transfer_batches_value_model_all_layers():
    """Batched partial transfers at the 8B shape on the full pool: the 512-token continuations of 16 agents packed by
    one aaf_kv_materialize_batch call and registered by one aaf_kv_import_batch call; every buffer and every live
    context compared in all layers with the value model."""
    import torch

    from tests.value_check import Paired

    g, seed, _ = configs.config2(True)
    if not _fits(g, 12):
        pytest.skip("not enough free device memory for the 64 GiB pool")
    T, agents, n_new = 8187, 16, 512
    gpu = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), init_fill=False)
    sh = ShadowBackend(gpu)
    st, root = sh.imp(sh.payload(seed, 1, T), T)
    st, kids = sh.fork(root, agents)
    assert sh.append(kids, [n_new] * agents, [sh.payload(seed, 2 + i, n_new) for i in range(agents)])[0] == 0
    bufs = [torch.empty(n_new * g.bpt, dtype=torch.uint8, device=gpu.o.device) for _ in range(agents)]
    assert gpu.o.materialize_batch(kids, [T] * agents, [T + n_new] * agents, bufs) == 0
    seqs = [sh.vm.materialize(k, T, T + n_new) for k in kids]
    for b, seq in zip(bufs, seqs):
        sh.check_buffer(seed, Paired(b, seq))
    st, new = gpu.o.import_batch(bufs, [n_new] * agents)
    assert st == 0
    assert [sh.vm.imp(seq) for seq in seqs] == new
    sh.check_all_live(seed)
    check_conservation(gpu.snapshot(), g.n_blocks, g.block_size)
    assert gpu.o.sync_status() == 0 and len(sh.vm.ctx) == 1 + 2 * agents


def test_config4_llama70b_value_model_all_layers():
    g, seed, ops = configs.config4(True)
    if not _fits(g, 40):
        pytest.skip("not enough free device memory for the 40 GiB pool plus 10 GiB buffers")
    sh, n_bufs = value_model_run(g, seed, ops)
    assert n_bufs == 10 and len(sh.vm.ctx) == 10
    assert sh.planes_checked == 160 * (n_bufs + 10)


def test_cow_stress_value_model_all_layers():
    g = Geometry(32, 8, 128, 16, 2, 4096, 1100, 1024)
    ops = configs.cow_stress_ops(context_tokens=8187, n_children=64)  # 64 children: every one compared in full
    sh, _ = value_model_run(g, configs.SEED_BASE + 6, ops, max_batch=1024)
    assert len(sh.vm.ctx) == 65 and sh.gpu.o.stats()["cow_count"] == 64


def test_value_check_detects_one_wrong_byte():
    """The all-layer comparison is not vacuous: one flipped byte in the last layer of a buffer fails it."""
    g = Geometry(4, 8, 128, 16, 2, 64, 4, 32)
    seed = 5
    gpu = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), init_fill=False)
    sh = ShadowBackend(gpu)
    st, c = sh.imp(sh.payload(seed, 1, 100), 100)
    st, buf = sh.materialize(c, 3, 97)
    sh.check_buffer(seed, buf)
    buf.dev[buf.dev.numel() - 7] ^= 1
    with pytest.raises(AssertionError, match="layer 3 kv 1"):
        sh.check_buffer(seed, buf)
