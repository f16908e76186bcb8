"""Parity of the CUDA library against the CPU oracle, element by element, through the C ABI.

Bit-exact bar: every materialised byte, every pool byte of the compared layers (stale slots
included), all block tables, token counts, reference counts and the free list in ring order.
"""
from __future__ import annotations

import numpy as np
import pytest

from tests.helpers import GpuBackend, OracleBackend, check_conservation
from workloads import configs
from workloads.configs import Geometry
from workloads.replay import replay

pytestmark = pytest.mark.gpu

VEC, BULK, WARP = 1, 2, 3


def same_catalog_export(gpu, cpu):
    """columnar catalog export: every column identical to the oracle's"""
    got = {k: v.cpu().numpy() for k, v in gpu.o.export_catalog().items()}
    want = cpu.o.export_catalog()
    assert got.keys() == want.keys()
    for k in want:
        assert got[k].dtype == want[k].dtype and np.array_equal(got[k], want[k]), k


def lockstep(g, seed, ops, layers=None, engine=0, max_batch=0, order=None, init_fill=True):
    """Replays ops on the GPU library and on the oracle side by side and compares after every op."""
    layers = list(range(g.n_layers)) if layers is None else list(layers)
    order = configs.free_order(seed, g.n_blocks) if order is None else order
    gpu = GpuBackend(g, seed, free_order=order, engine=engine, max_batch=max_batch, init_fill=init_fill)
    cpu = OracleBackend(g, seed, layers=layers, free_order=order, init_fill=init_fill)
    for (i, op, st_g, res_g, _), (_, _, st_c, res_c, _) in zip(replay(ops, gpu, seed), replay(ops, cpu, seed)):
        assert st_g == st_c, (i, op, st_g, st_c)
        assert gpu.snapshot() == cpu.snapshot(), (i, op)
        assert gpu.o.catalog() == cpu.o.catalog(), (i, op)
        if op["op"] == "materialize" and st_c == 0:
            n = op["t1"] - op["t0"]
            assert np.array_equal(gpu.buf_layers(res_g, n, layers).reshape(-1), res_c), (i, op)
    assert np.array_equal(gpu.pool_layers(layers), cpu.o.pool_view()), "pool image differs"
    same_catalog_export(gpu, cpu)
    assert gpu.o.sync_status() == 0
    gs, cs = gpu.o.stats(), cpu.o.stats()
    for k in ("free_blocks", "live_blocks", "peak_live_blocks", "live_ctx", "cow_count"):
        assert gs[k] == cs[k], (k, gs[k], cs[k])
    assert gs["payload_bytes"] == cs["rows_copied"] * g.row * g.n_layers // len(layers)
    return gpu, cpu


@pytest.mark.parametrize("engine", [VEC, BULK, WARP])
@pytest.mark.parametrize("unaligned", [False, True])
def test_config1_tiny_pool(engine, unaligned):
    g, seed, ops = configs.config1(unaligned)
    gpu, cpu = lockstep(g, seed, ops, engine=engine)
    assert gpu.o.stats()["cow_count"] == (4 if unaligned else 0)
    assert sorted(gpu.o.free_list().tolist()) == list(range(g.n_blocks))


# odd geometry: row = 3*40*2 = 240 bytes (not a power of two), run = 1680 bytes, several chunks per
# launch and a ragged tail everywhere
ODD = Geometry(3, 3, 40, 7, 2, 48, 10, 24)


def random_walk(g: Geometry, seed: int, n_ops: int, engine: int):
    """Random operators chosen against the oracle's current state, applied to both sides and compared
    after every operator.  Lengths and counts are drawn so that out-of-blocks, out-of-handles and
    too-long failures occur naturally; a few operators are made invalid on purpose (dead handle,
    duplicate context, empty range).  Failures must be identical and change nothing."""
    rng = np.random.default_rng(seed)
    order = configs.free_order(seed, g.n_blocks)
    gpu = GpuBackend(g, seed, free_order=order, engine=engine)
    cpu = OracleBackend(g, seed, free_order=order)
    layers = list(range(g.n_layers))
    stream = 1
    outcomes = []
    for i in range(n_ops):
        live = cpu.o.live_ctxs()
        kind = str(rng.choice(["import", "fork", "append", "compose", "evict", "materialize", "roundtrip", "budget",
                               "compose_batch", "transfer_batch"],
                              p=[0.15, 0.11, 0.22, 0.11, 0.10, 0.11, 0.05, 0.04, 0.06, 0.05]))
        if not live:
            kind = "import"
        pick = lambda: int(rng.choice(live)) if rng.random() > 0.04 else int(rng.integers(0, g.max_ctx))
        both = (gpu, cpu)
        if kind == "import":
            n = int(rng.integers(1, 6 * g.block_size))
            res = [be.imp(be.payload(seed, stream, n), n) for be in both]
            stream += 1
        elif kind == "fork":
            c, k = pick(), int(rng.integers(0, 4))
            res = [be.fork(c, k) for be in both]
        elif kind == "append":
            m = int(rng.integers(1, 4))
            who = [pick() for _ in range(m)]  # duplicates possible -> INVALID_ARG
            nn = [int(rng.integers(1, 3 * g.block_size)) for _ in who]
            res = [be.append(who, nn, [be.payload(seed, stream + j, n) for j, n in enumerate(nn)]) for be in both]
            stream += m
        elif kind == "compose":
            segs = [pick() for _ in range(int(rng.integers(1, 4)))]
            fl = int(rng.integers(0, 2))
            res = [be.compose(segs, fl) for be in both]
        elif kind in ("compose_batch", "transfer_batch"):
            # Batched calls equal the oracle's loop of single calls when the loop succeeds throughout; when any
            # call of the loop fails, the batch must fail as a whole and change nothing (the loop is tried on a copy).
            import torch

            before = cpu.snapshot()
            trial = cpu.o.clone()
            if kind == "compose_batch":
                batch = [[pick() for _ in range(int(rng.integers(1, 4)))] for _ in range(int(rng.integers(1, 4)))]
                fl = int(rng.integers(0, 2))
                # (a result of the same batch cannot be a segment: every segment must be live before the call)
                loop_ok = all(c in live for segs in batch for c in segs) and \
                    all(trial.compose(segs, fl)[0] == 0 for segs in batch)
                st_g, r_g = gpu.o.compose_batch(batch, fl)
                r_c = [cpu.compose(segs, fl)[1] for segs in batch] if loop_ok else None
            else:
                ranges = []
                for _ in range(int(rng.integers(1, 4))):
                    c = pick()
                    T = cpu.o.ctx_len(c) or 4
                    a = int(rng.integers(0, T))
                    ranges.append((c, a, int(rng.integers(a, T + 1))))  # a == b -> INVALID_ARG
                outs = [torch.empty(max(b - a, 1) * g.bpt, dtype=torch.uint8, device=gpu.o.device)
                        for _, a, b in ranges]
                bufs_c = [trial.materialize(c, a, b) for c, a, b in ranges]
                loop_ok = all(st == 0 for st, _ in bufs_c) and \
                    all(trial.imp(buf, b - a)[0] == 0 for (st, buf), (_, a, b) in zip(bufs_c, ranges))
                st_g = gpu.o.materialize_batch([c for c, _, _ in ranges], [a for _, a, _ in ranges],
                                               [b for _, _, b in ranges], outs)
                r_g = None
                if all(st == 0 for st, _ in bufs_c):  # the gathers alone are valid: compare them, then register
                    assert st_g == 0, (i, kind, st_g)
                    for (c, a, b), o_dev in zip(ranges, outs):
                        assert np.array_equal(o_dev.cpu().numpy()[: (b - a) * g.bpt], cpu.materialize(c, a, b)[1])
                    st_g, r_g = gpu.o.import_batch(outs, [b - a for _, a, b in ranges])
                    r_c = [cpu.imp(buf, b - a)[1] for (_, buf), (_, a, b) in zip(bufs_c, ranges)] if loop_ok else None
                else:
                    assert st_g < 0, (i, kind)
                    r_c = None
            if loop_ok:
                res = [(st_g, r_g), (0, r_c)]
            else:
                assert st_g < 0 and gpu.snapshot() == before, (i, kind, st_g)
                res = [(st_g, None), (st_g, None)]
        elif kind == "evict":
            who = [pick() for _ in range(int(rng.integers(1, 3)))]
            res = [be.evict(who) for be in both]
        elif kind == "budget":  # scored eviction down to a random fraction of the current use
            w = [float(x) for x in rng.choice([0.0, 0.5, 1.0, 2.25], size=3)]
            budget = int(rng.integers(0, g.n_blocks))
            res = [be.o.evict_to_budget(w[0], w[1], w[2], budget) for be in both]
        else:
            c = pick()
            T = cpu.o.ctx_len(c) or 4
            a = int(rng.integers(0, T))
            b = int(rng.integers(a, T + 1)) if kind == "materialize" else T  # a == b -> INVALID_ARG
            a = a if kind == "materialize" else 0
            res = [be.materialize(c, a, b) for be in both]
            if res[1][0] == 0:
                assert np.array_equal(gpu.buf_layers(res[0][1], b - a, layers).reshape(-1), res[1][1]), (i, kind)
                if kind == "roundtrip":
                    res = [gpu.imp(res[0][1], b - a), cpu.imp(res[1][1], b - a)]
        (st_g, r_g), (st_c, r_c) = res
        assert st_g == st_c, (i, kind, st_g, st_c)
        if kind != "materialize":
            assert r_g == r_c or kind == "roundtrip" and st_c == 0 and r_g == r_c, (i, kind, r_g, r_c)
        snap = cpu.snapshot()
        assert gpu.snapshot() == snap, (i, kind)
        assert gpu.o.catalog() == cpu.o.catalog(), (i, kind)
        check_conservation(snap, g.n_blocks, g.block_size)
        if i % 8 == 7:
            assert np.array_equal(gpu.pool_layers(layers), cpu.o.pool_view()), (i, kind)
            same_catalog_export(gpu, cpu)
        outcomes.append((kind, st_c))
    assert np.array_equal(gpu.pool_layers(layers), cpu.o.pool_view())
    assert gpu.o.sync_status() == 0
    return outcomes


@pytest.mark.parametrize("engine", [VEC, BULK, WARP])
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_operator_sequences_on_odd_geometry(engine, seed):
    outcomes = random_walk(ODD, 7000 + seed, 200, engine)
    ok = {k for k, st in outcomes if st == 0}
    assert ok >= {"import", "fork", "append", "compose", "evict", "materialize"}
    failed = {st for _, st in outcomes if st < 0}
    assert -3 in failed, "the walk should run out of blocks at least once"


# 8B-shaped rows (2 KiB rows, 32 KiB runs) on a pool small enough for the oracle to hold all layers
MID = Geometry(4, 8, 128, 16, 2, 1024, 24, 256)


@pytest.mark.parametrize("engine", [VEC, BULK, WARP])
@pytest.mark.parametrize("unaligned", [False, True])
def test_fanout_with_8b_rows(engine, unaligned):
    T = 1019 if unaligned else 1024
    ops = configs.fanout_ops(T, 6, 100, compose_pair=True, evict_all=True, roundtrip=True)
    lockstep(MID, 4242, ops, engine=engine)


def test_batched_append_equals_single_appends():
    T = 1019
    a = configs.fanout_ops(T, 6, 37, compose_pair=False, evict_all=False, roundtrip=False, batched_append=True)
    b = configs.fanout_ops(T, 6, 37, compose_pair=False, evict_all=False, roundtrip=False, batched_append=False)
    ga, _ = lockstep(MID, 99, a)
    gb, _ = lockstep(MID, 99, b)
    assert ga.snapshot() == gb.snapshot()
    layers = list(range(MID.n_layers))
    assert np.array_equal(ga.pool_layers(layers), gb.pool_layers(layers))


@pytest.mark.parametrize("copy_all", [False, True])
def test_compose_tree_small(copy_all):
    g = Geometry(2, 8, 128, 16, 2, 2048, 40, 512)
    g2, seed, ops, lens = configs.config3(g, copy_all=copy_all, lo=100, hi=400)
    lockstep(g, seed, ops)


def test_cow_stress_many_children():
    g = Geometry(2, 8, 128, 16, 2, 1024, 300, 64)
    ops = configs.cow_stress_ops(context_tokens=507, n_children=256)
    gpu, cpu = lockstep(g, 5150, ops, max_batch=256)
    assert gpu.o.stats()["cow_count"] == 256  # every child copies: the parent keeps the old tail


@pytest.mark.parametrize("weights", [(0.0, 0.0, 1.0), (0.0, 1.0, 0.0), (1.0, 0.0, 0.0), (1.5, 0.25, 0.1), (10.0, 0.01, 3.3)])
@pytest.mark.parametrize("budget", [0, 6, 11, 400])
def test_scored_eviction_to_budget(weights, budget):
    """Alg. KV-Evict with the victims chosen on the device: same victims in the same order, same
    tables / reference counts / free list as the oracle's loop."""
    g = Geometry(2, 2, 64, 4, 2, 64, 12, 32)
    order = configs.free_order(31, g.n_blocks)
    gpu = GpuBackend(g, 31, free_order=order)
    cpu = OracleBackend(g, 31, free_order=order)
    for be in (gpu, cpu):
        pay = lambda s, n: be.payload(31, s, n)
        a = be.imp(pay(1, 10), 10)[1]
        b = be.imp(pay(2, 23), 23)[1]
        kids = be.fork(a, 3)[1]
        assert be.append([kids[0]], [5], [pay(3, 5)])[0] == 0
        be.materialize(b, 0, 23)
        be.materialize(b, 3, 9)
        z = be.compose([kids[1], b], 0)[1]
        assert be.append([kids[2]], [9], [pay(4, 9)])[0] == 0
        be.materialize(kids[0], 0, 15)
        be.compose([b, b], 0)
    assert gpu.o.catalog() == cpu.o.catalog()
    rg = gpu.o.evict_to_budget(*weights, budget)
    rc = cpu.o.evict_to_budget(*weights, budget)
    assert rg == rc and rc[0] == 0
    assert gpu.snapshot() == cpu.snapshot() and gpu.o.catalog() == cpu.o.catalog()
    check_conservation(cpu.snapshot(), g.n_blocks, g.block_size)
    assert gpu.o.stats()["live_blocks"] <= max(budget, 0) or not gpu.o.live_ctxs()
    # the pool keeps working with exact free accounting afterwards
    for be in (gpu, cpu):
        assert be.imp(be.payload(31, 9, 30), 30)[0] == 0
    assert gpu.snapshot() == cpu.snapshot()
    assert gpu.o.evict_to_budget(float("nan"), 0.0, 1.0, 3)[0] == -1
    assert gpu.o.evict_to_budget(0.0, 0.0, 1.0, -2)[0] == -1
    assert gpu.o.sync_status() == 0


def test_catalog_export_wraps_as_arrow_without_conversion():
    import pyarrow as pa

    g = Geometry(2, 2, 64, 4, 2, 64, 12, 32)
    gpu = GpuBackend(g, 77)
    cpu = OracleBackend(g, 77)
    same_catalog_export(gpu, cpu)  # empty pool: no state rows, offsets = [0]
    for be in (gpu, cpu):
        a = be.imp(be.payload(77, 1, 10), 10)[1]
        kids = be.fork(a, 3)[1]
        be.append(kids[:2], [5, 1], [be.payload(77, 2, 5), be.payload(77, 3, 1)])
        be.compose([kids[0], kids[2]], 0)
        be.evict([kids[1]])
    same_catalog_export(gpu, cpu)
    cols = {k: v.cpu().numpy() for k, v in gpu.o.export_catalog().items()}
    lst = pa.ListArray.from_arrays(pa.array(cols["block_offsets"], type=pa.int32()),
                                   pa.array(cols["block_id"], type=pa.int32()))
    lst.validate(full=True)
    assert lst.to_pylist() == [gpu.o.table(int(c)).tolist() for c in cols["state_id"]]
    tbl = pa.table({"state_id": cols["state_id"], "n_tokens": cols["n_tokens"], "reuse": cols["reuse"],
                    "last_access": cols["last_access"], "blocks": lst})
    assert tbl.num_rows == len(gpu.o.live_ctxs())


# degenerate and extreme geometries: one-token blocks, 16-byte rows, odd block sizes, a single handle,
# runs larger than every engine's chunk
EDGE_GEOMETRIES = [
    Geometry(1, 1, 8, 1, 2, 40, 6, 24),        # block = 1 token, row = 16 B, run = 16 B
    Geometry(2, 1, 8, 3, 2, 50, 5, 20),        # row 16 B, block of 3 tokens
    Geometry(1, 8, 128, 64, 2, 24, 4, 8),      # run = 128 KiB (> bulk chunk, several chunks per piece)
    Geometry(5, 2, 24, 5, 4, 64, 7, 16),       # 4-byte elements, row 192 B, run 960 B
    Geometry(1, 1, 8, 4, 2, 12, 1, 12),        # a single context handle
]


@pytest.mark.parametrize("engine", [0, VEC, BULK, WARP])
@pytest.mark.parametrize("gi", range(len(EDGE_GEOMETRIES)))
def test_random_walks_on_edge_geometries(engine, gi):
    g = EDGE_GEOMETRIES[gi]
    outcomes = random_walk(g, 8100 + gi, 120, engine)
    assert sum(st == 0 for _, st in outcomes) >= 25


def test_capacity_limits_are_exact():
    """Longest table, largest batch, last free block, last free handle: accepted at the limit, refused one past it."""
    g = Geometry(1, 1, 8, 2, 2, 64, 6, 10)
    gpu = GpuBackend(g, 3, max_batch=4)
    cpu = OracleBackend(g, 3)
    for be in (gpu, cpu):
        pay = lambda s, n: be.payload(3, s, n)
        assert be.imp(pay(1, 20), 20) == (0, 0)                                   # exactly max_blocks_per_ctx blocks
        assert be.imp(pay(2, 21), 21)[0] == -5                                    # one token too long
        assert be.append([0], [1], [pay(3, 1)])[0] == -5
        assert be.fork(0, 4) == (0, [1, 2, 3, 4])                                 # k = max_batch
        assert be.compose([1, 2], 0)[0] == -5                                     # 40 tokens > 10 blocks
        assert be.evict([1, 2, 3, 4])[0] == 0                                     # n = max_batch
        assert be.imp(pay(4, 19), 19) == (0, 1)                                   # 10 more blocks
        assert be.fork(1, 4) == (0, [2, 3, 4, 5])                                 # uses the last free handle
        assert be.imp(pay(5, 1), 1)[0] == -4                                      # no handle left
        assert be.evict([5])[0] == 0
        assert be.append([1, 2, 3, 4], [1, 1, 1, 1], [pay(6 + i, 1) for i in range(4)])[0] == 0  # 3 COW + in place
    assert gpu.o.fork(0, 5)[0] == binding_too_many()
    assert gpu.snapshot() == cpu.snapshot()
    assert np.array_equal(gpu.pool_layers([0]), cpu.o.pool_view())
    assert gpu.o.stats()["cow_count"] == cpu.o.stats()["cow_count"] == 3


def binding_too_many():
    from paper_2607_10987_b200 import binding

    return binding.AAF_ERR_TOO_MANY


# ------------------------------------------------------------------------------------------------------------
# The hand-derived worked examples, replayed on the library and compared with the written-out values directly
# (no oracle in between): block tables, reference counts, block contents and the order of the free list.


def _golden(name):
    import os

    out = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", name)):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=", 1)
            out[k.strip()] = v.strip()
    return out


def _named_pool(g, gold, names):
    """library pool with the golden ring, zeroed image, and an encoder of named tokens into device payloads"""
    import torch

    from tests.helpers import encode_tokens

    ring = [int(x) for x in gold["ring"].split()]
    be = GpuBackend(g, 1, free_order=ring, init_fill="zero")
    enc = lambda toks: torch.from_numpy(encode_tokens([names[t] for t in toks], g.n_layers, g.row).copy()).to(be.o.device)
    return be, enc


def _block_holds(be, g, b, toks, names):
    from tests.helpers import token_row

    img = be.pool_layers(range(g.n_layers))
    for s, tok in enumerate(toks):
        for l in range(g.n_layers):
            for kv in range(2):
                want = bytes(g.row) if tok == "." else token_row(names[tok], l, kv, g.row)
                assert bytes(img[l, b, kv, s]) == want, (b, s, tok)


@pytest.mark.parametrize("engine", [VEC, BULK, WARP])
def test_worked_example_w1_against_the_hand_derived_values(engine):
    gold = _golden("worked_example_w1.txt")
    ints = lambda k: [int(x) for x in gold[k].split()]
    g = Geometry(2, 1, 8, int(gold["BS"]), 2, int(gold["NB"]), 4, 8)  # 16-byte rows
    names = {f"p{i}": i for i in range(6)}
    names.update({f"x{i}": 100 + i for i in range(3)})
    be, enc = _named_pool(g, gold, names)
    be.o.set_copy_engine(engine)
    assert be.imp(enc([f"p{i}" for i in range(6)]), 6) == (0, 0)
    assert be.o.table(0).tolist() == ints("P.table")
    assert be.fork(0, 2) == (0, [1, 2])
    assert be.append([1], [3], [enc(["x0", "x1", "x2"])])[0] == 0
    assert be.o.table(1).tolist() == ints("c1.table")
    assert be.compose([1, 2], 0) == (0, 3)
    assert be.o.table(3).tolist() == ints("Z.table")
    for key in ("block4", "block0", "block5", "block2"):
        _block_holds(be, g, int(key[5:]), gold[key].split(), names)
    assert be.evict([0, 2])[0] == 0
    assert be.o.refcounts().tolist() == ints("refcount")
    assert be.o.free_list().tolist() == ints("free_list")
    assert be.o.sync_status() == 0


def test_worked_example_w1_copy_all_against_the_hand_derived_values():
    gold = _golden("worked_example_w1.txt")
    g = Geometry(2, 1, 8, int(gold["BS"]), 2, int(gold["NB"]), 4, 8)
    names = {f"p{i}": i for i in range(6)}
    names.update({f"x{i}": 100 + i for i in range(3)})
    be, enc = _named_pool(g, gold, names)
    assert be.imp(enc([f"p{i}" for i in range(6)]), 6) == (0, 0)
    assert be.fork(0, 2) == (0, [1, 2])
    assert be.append([1], [3], [enc(["x0", "x1", "x2"])])[0] == 0
    assert be.compose([1, 2], configs.COMPOSE_COPY_ALL) == (0, 3)
    assert be.o.table(3).tolist() == [int(x) for x in gold["Zc.table"].split()]
    for key in ("Zc.block5", "Zc.block2", "Zc.block7", "Zc.block6"):
        _block_holds(be, g, int(key[8:]), gold[key].split(), names)
    assert be.o.free_list().tolist() == [] and be.o.sync_status() == 0


def test_worked_example_w2_free_order_against_the_hand_derived_values():
    gold = _golden("worked_example_w2.txt")
    ints = lambda k: [int(x) for x in gold[k].split()]
    g = Geometry(2, 1, 8, int(gold["BS"]), 2, int(gold["NB"]), 6, 8)
    names = {f"a{i}": i for i in range(8)}
    names.update({f"c{i}": 50 + i for i in range(5)})
    names["y0"] = 90

    def state():
        be, enc = _named_pool(g, gold, names)
        assert be.imp(enc([f"a{i}" for i in range(8)]), 8) == (0, 0)
        assert be.compose([0, 0], 0) == (0, 1)
        assert be.o.table(1).tolist() == ints("B.table")
        assert be.imp(enc([f"c{i}" for i in range(5)]), 5) == (0, 2)
        assert be.fork(2, 1) == (0, [3])
        assert be.append([3], [1], [enc(["y0"])])[0] == 0
        assert be.o.table(3).tolist() == ints("D.table")
        _block_holds(be, g, 3, gold["block3"].split(), names)
        assert be.o.refcounts().tolist() == ints("refcount.before_evict")
        return be

    be = state()
    assert be.evict([1, 3, 0])[0] == 0  # B, D, A
    assert be.o.refcounts().tolist() == ints("refcount.after_evict")
    assert be.o.free_list().tolist() == ints("free_list.after_evict")
    assert be.o.live_ctxs() == ints("live.after_evict") and be.o.sync_status() == 0
    # the scored eviction loop on the same state
    be = state()
    assert be.materialize(0, 0, 8)[0] == 0
    st, victims = be.o.evict_to_budget(0.0, 0.0, 1.0, 3)
    assert st == 0 and victims == ints("budget.victims")
    assert be.o.refcounts().tolist() == ints("budget.refcount")
    assert be.o.free_list().tolist() == ints("budget.free_list")
    assert be.o.live_ctxs() == [0] and be.o.sync_status() == 0


def test_small_batch_with_many_entries_takes_the_grid_evict_path():
    """Two contexts (a small batch, which would travel as kernel parameters) with 70 000 table entries between
    them (beyond what one CTA compacts): the argument records must go through memory and the grid-wide
    count / scan / scatter must free the same blocks in the same order as the oracle."""
    g = Geometry(1, 1, 8, 1, 2, 70000, 8, 80000)  # one token per block, 16-byte rows
    ops = [
        {"op": "import", "out": "a", "n": 35000, "stream": 1},
        {"op": "fork", "ctx": "a", "k": 1, "out": ["b"]},
        {"op": "import", "out": "c", "n": 30000, "stream": 2},
        {"op": "evict", "ctxs": ["c", "a"]},   # frees c's 30 000 blocks; a's stay referenced by b
        {"op": "compose", "segs": ["b", "b"], "flags": 0, "out": "bb"},
        {"op": "evict", "ctxs": ["bb", "b"]},  # 105 000 entries on 35 000 blocks, each named three times
    ]
    gpu, cpu = lockstep(g, 77, ops)
    assert sorted(gpu.o.free_list().tolist()) == list(range(g.n_blocks))


# ------------------------------------------------------------------------------------------------------------
# aaf_kv_compose_batch: several merges in one planner launch and one copy launch == the loop of single merges


def _merge_pool(seed, lens, g=None):
    g = g or Geometry(3, 4, 64, 16, 2, 512, 40, 96)  # 512-byte rows, 8 KiB runs
    order = configs.free_order(seed, g.n_blocks)
    gpu = GpuBackend(g, seed, free_order=order)
    cpu = OracleBackend(g, seed, free_order=order)
    for i, n in enumerate(lens):
        for be in (gpu, cpu):
            assert be.imp(be.payload(seed, 1 + i, n), n) == (0, i)
    return g, gpu, cpu


@pytest.mark.parametrize("flags", [0, configs.COMPOSE_COPY_ALL])
def test_compose_batch_equals_the_loop_of_single_merges(flags):
    lens = [37, 64, 16, 5, 100, 48, 33, 1, 80, 250]
    g, gpu, cpu = _merge_pool(31, lens)
    # a source used by several merges, an aligned first segment, a merge of one (== fork), a long merge, repeats
    batch = [[0, 1], [1, 2, 3], [4], [2, 2, 5, 0], [9, 8, 7, 6, 5, 4, 3], [1, 0]]
    st, outs = gpu.o.compose_batch(batch, flags)
    assert st == 0
    want = []
    for segs in batch:
        st_c, c = cpu.compose(segs, flags)
        assert st_c == 0
        want.append(c)
    assert outs == want
    assert gpu.snapshot() == cpu.snapshot()
    assert gpu.o.catalog() == cpu.o.catalog()
    same_catalog_export(gpu, cpu)
    assert np.array_equal(gpu.pool_layers(range(g.n_layers)), cpu.o.pool_view())
    for c in outs:
        n = cpu.o.ctx_len(c)
        assert np.array_equal(gpu.buf_layers(gpu.materialize(c, 0, n)[1], n, range(g.n_layers)).reshape(-1),
                              cpu.materialize(c, 0, n)[1])
    gs, cs = gpu.o.stats(), cpu.o.stats()
    assert gs["copy_launches"]["compose"] == 1 and gs["payload_bytes"] == cs["rows_copied"] * g.row
    # results of a batch are ordinary contexts: merge them again, as one more batch, then evict everything
    st, outs2 = gpu.o.compose_batch([outs[:3], outs[3:]], flags)
    assert st == 0
    assert [cpu.compose(outs[:3], flags)[1], cpu.compose(outs[3:], flags)[1]] == outs2
    everything = cpu.o.live_ctxs()
    assert gpu.evict(everything)[0] == 0 and cpu.evict(everything)[0] == 0
    assert gpu.snapshot() == cpu.snapshot() and gpu.o.sync_status() == 0
    assert sorted(gpu.o.free_list().tolist()) == list(range(g.n_blocks))


def test_compose_batch_is_all_or_nothing():
    from paper_2607_10987_b200 import binding

    lens = [700, 700, 90, 21]
    g, gpu, cpu = _merge_pool(32, lens, Geometry(2, 4, 64, 16, 2, 160, 6, 90))  # 90-block tables, 160 blocks, 6 handles
    before = gpu.snapshot()
    assert before == cpu.snapshot()
    # second merge too long (1400 tokens = 88 blocks fits, 1490 = 94 does not); first merge alone would succeed
    assert gpu.o.compose_batch([[2, 3], [0, 1, 2]], 0)[0] == binding.AAF_ERR_TOO_LONG
    # not enough blocks for both copies: 96 blocks are live, 64 free; each copy-all merge of [0, 3] needs 46
    assert gpu.o.compose_batch([[0, 3], [0, 3]], configs.COMPOSE_COPY_ALL)[0] == binding.AAF_ERR_OOM_BLOCKS
    # three results but only two free handles
    assert gpu.o.compose_batch([[2], [3], [2, 3]], 0)[0] == binding.AAF_ERR_OOM_CTX
    assert gpu.o.compose_batch([[2, 3], [5]], 0)[0] == binding.AAF_ERR_BAD_CTX
    assert gpu.o.compose_batch([[2, 3], []], 0)[0] == binding.AAF_ERR_INVALID_ARG
    assert gpu.snapshot() == before and gpu.o.catalog() == cpu.o.catalog()
    # and one of them alone goes through, identically on both sides
    assert gpu.o.compose_batch([[0, 3]], configs.COMPOSE_COPY_ALL) == (0, [4])
    assert cpu.compose([0, 3], configs.COMPOSE_COPY_ALL) == (0, 4)
    assert gpu.snapshot() == cpu.snapshot() and gpu.o.sync_status() == 0


def test_batches_at_the_batch_limit_go_through_the_argument_ring():
    """1000 segments in one merge, 1000 merges in one batch, 1000 transfers in one batch: the records travel
    through the pinned argument ring (not as kernel parameters) and must fit it."""
    g = Geometry(2, 1, 8, 16, 2, 4096, 1030, 800)  # 16-byte rows
    seed = 41
    order = configs.free_order(seed, g.n_blocks)
    gpu = GpuBackend(g, seed, free_order=order)
    cpu = OracleBackend(g, seed, free_order=order)
    for be in (gpu, cpu):
        assert be.imp(be.payload(seed, 1, 3), 3) == (0, 0)
        assert be.imp(be.payload(seed, 2, 21), 21) == (0, 1)
    # one merge of 1000 segments
    segs = [0, 1] * 500
    assert gpu.compose(segs, 0) == cpu.compose(segs, 0) == (0, 2)
    assert gpu.snapshot() == cpu.snapshot()
    # 1000 merges of one or two segments in one batch, 1024 segments in all (results 3 .. 1002)
    batch = [[1, 0] if i < 24 else [i % 3] for i in range(1000)]
    st, outs = gpu.o.compose_batch(batch, 0)
    assert st == 0 and outs == list(range(3, 1003))
    for b in batch:
        assert cpu.compose(b, 0)[0] == 0
    assert gpu.snapshot() == cpu.snapshot() and gpu.o.catalog() == cpu.o.catalog()
    # 1000 gathers in one batch, compared with the oracle's loop
    import torch

    ctxs = [3 + i for i in range(1000)]
    lens = [min(cpu.o.ctx_len(c), 20) for c in ctxs]  # the first 20 tokens of each: at most two blocks per entry
    outs_dev = [torch.empty(n * g.bpt, dtype=torch.uint8, device=gpu.o.device) for n in lens]
    assert gpu.o.materialize_batch(ctxs, [0] * 1000, lens, outs_dev) == 0
    for c, n, d in zip(ctxs, lens, outs_dev):
        st, want = cpu.materialize(c, 0, n)
        assert st == 0 and np.array_equal(d.cpu().numpy(), want), c
    assert gpu.o.catalog() == cpu.o.catalog()
    assert np.array_equal(gpu.pool_layers(range(g.n_layers)), cpu.o.pool_view())
    assert gpu.o.sync_status() == 0


def test_materialize_and_import_batches_equal_the_loops():
    """aaf_kv_materialize_batch / aaf_kv_import_batch against the oracle's loops of single calls: ragged ranges,
    a context gathered twice, block tables and handles of the imported batch, catalog stamps, one copy launch each."""
    import torch

    from paper_2607_10987_b200 import binding

    lens = [37, 64, 16, 5, 100, 48, 33, 1, 80, 250]
    g, gpu, cpu = _merge_pool(33, lens)
    dev = gpu.o.device
    ranges = [(0, 0, 37), (1, 16, 64), (4, 3, 99), (9, 17, 250), (4, 0, 100), (7, 0, 1), (3, 2, 5), (8, 79, 80),
              (2, 0, 16), (5, 15, 17)]
    outs = [torch.full(((b - a) * g.bpt,), 0xEE, dtype=torch.uint8, device=dev) for _, a, b in ranges]
    l0 = gpu.o.stats()["copy_launches"]["materialize"]
    assert gpu.o.materialize_batch([c for c, _, _ in ranges], [a for _, a, _ in ranges], [b for _, _, b in ranges],
                                   outs) == 0
    assert gpu.o.stats()["copy_launches"]["materialize"] == l0 + 1
    want = []
    for (c, a, b), d in zip(ranges, outs):
        st, w = cpu.materialize(c, a, b)
        assert st == 0 and np.array_equal(d.cpu().numpy(), w), (c, a, b)
        want.append(w)
    assert gpu.o.catalog() == cpu.o.catalog()
    # register all ten buffers as new contexts in one call
    st, new = gpu.o.import_batch(outs, [b - a for _, a, b in ranges])
    assert st == 0 and gpu.o.stats()["copy_launches"]["import"] == len(lens) + 1
    for w, (c, a, b), h in zip(want, ranges, new):
        assert cpu.imp(w, b - a) == (0, h)
    assert gpu.snapshot() == cpu.snapshot() and gpu.o.catalog() == cpu.o.catalog()
    same_catalog_export(gpu, cpu)
    assert np.array_equal(gpu.pool_layers(range(g.n_layers)), cpu.o.pool_view())
    # all-or-nothing
    before = gpu.snapshot()
    small = torch.empty(16, dtype=torch.uint8, device=dev)
    assert gpu.o.materialize_batch([0, 1], [0, 0], [37, 64], [outs[0], small]) == binding.AAF_ERR_DST_TOO_SMALL
    assert gpu.o.materialize_batch([0, 39], [0, 0], [37, 1], [outs[0], outs[5]]) == binding.AAF_ERR_BAD_CTX
    assert gpu.o.materialize_batch([0, 1], [0, 0], [37, 65], [outs[0], outs[1]]) == binding.AAF_ERR_INVALID_ARG
    big = [gpu.payload(33, 50, 1500)] * 5
    assert gpu.o.stats()["free_blocks"] < 5 * 94
    assert gpu.o.import_batch(big, [1500] * 5)[0] == binding.AAF_ERR_OOM_BLOCKS  # 5 x 94 blocks, fewer are free
    assert gpu.o.import_batch([big[0]], [1600])[0] == binding.AAF_ERR_TOO_LONG     # 100 blocks > 96
    assert gpu.o.import_batch([outs[0]] * 25, [37] * 25)[0] == binding.AAF_ERR_OOM_CTX  # 40 handles, 20 live
    assert gpu.snapshot() == before and gpu.o.catalog() == cpu.o.catalog() and gpu.o.sync_status() == 0
