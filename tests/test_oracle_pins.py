"""Pins of the CPU oracle: what the paper and the mathematics fix about the operators,
checked without reference to the CUDA path (runs on a CPU-only box)."""
from __future__ import annotations

import os

import numpy as np
import pytest

from oracle import paged
from oracle.value_model import ValueModel
from tests.helpers import (check_against_value_model, check_conservation, encode_tokens, snapshot, token_row)

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_kv(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=", 1)
                out[k.strip()] = v.strip()
    return out


def small_pool(NB=16, BS=4, L=2, H=1, D=4, E=2, max_ctx=8, max_blk=16, order=None):
    return paged.PagedOracle(L, H, D, BS, E, NB, max_ctx, max_blk, order)


def rand_buf(rng, o, n):
    return rng.integers(0, 256, size=n * o.bpt, dtype=np.uint8)


# ---------------------------------------------------------------- closed forms the paper prints


def test_bytes_per_token_matches_printed_transfer_time():
    g = _read_kv(os.path.join(GOLD, "transfer_time_max_context.txt"))
    o = paged.PagedOracle(int(g["n_layers"]), int(g["n_kv_heads"]), int(g["head_dim"]), 16, int(g["elt_bytes"]),
                          4, 2, 4)
    assert o.bpt == 131072
    # the oracle's own buffer size for one token is what materialize demands
    st, c = o.imp(np.zeros(o.bpt, np.uint8), 1)
    assert st == 0
    assert o.materialize(c, 0, 1, dst_bytes=o.bpt - 1)[0] == paged.DST_TOO_SMALL
    assert o.materialize(c, 0, 1, dst_bytes=o.bpt)[0] == 0
    t = (int(g["context_tokens"]) * o.bpt / float(g["bandwidth_bytes_per_sec"]) + float(g["network_latency_sec"])
         + float(g["resume_overhead_sec"]))
    assert round(t, int(g["printed_digits"])) == float(g["printed_ttft_sec"])


# ---------------------------------------------------------------- worked example (conventions)


def test_worked_example_w1():
    g = _read_kv(os.path.join(GOLD, "worked_example_w1.txt"))
    NB, BS = int(g["NB"]), int(g["BS"])
    ring = [int(x) for x in g["ring"].split()]
    L, row = 2, 8
    o = paged.PagedOracle(L, 1, 4, BS, 2, NB, 4, 8, ring)
    names = {f"p{i}": i for i in range(6)}
    names.update({f"x{i}": 100 + i for i in range(3)})
    enc = lambda toks: encode_tokens([names[t] for t in toks], L, row)

    st, P = o.imp(enc([f"p{i}" for i in range(6)]), 6)
    assert (st, P) == (0, 0)
    assert o.table(P).tolist() == [int(x) for x in g["P.table"].split()]
    st, (c1, c2) = o.fork(P, 2)
    assert (c1, c2) == (1, 2)
    assert o.refcounts()[1] == 3 and o.refcounts()[3] == 3
    st, _ = o.append([c1], [3], [enc(["x0", "x1", "x2"])])
    assert st == 0
    assert o.table(c1).tolist() == [int(x) for x in g["c1.table"].split()]
    assert np.array_equal(o.materialize(P, 0, 6)[1], enc([f"p{i}" for i in range(6)]))
    # the merge policy that forbids aliasing, on a copy of the state: fresh blocks in increasing table position
    oc = o.clone()
    st, Zc = oc.compose([c1, c2], paged.COMPOSE_COPY_ALL)
    assert (st, Zc) == (0, 3)
    assert oc.table(Zc).tolist() == [int(x) for x in g["Zc.table"].split()]
    pvc = oc.pool_view()
    for key in ("Zc.block5", "Zc.block2", "Zc.block7", "Zc.block6"):
        b = int(key[8:])
        for s, tok in enumerate(g[key].split()):
            for l in range(L):
                for kv in range(2):
                    want = bytes(row) if tok == "." else token_row(names[tok], l, kv, row)
                    assert bytes(pvc[l, b, kv, s]) == want, (key, s)
    assert oc.stats()["rows_copied"] == int(g["Zc.rows_copied"])
    assert oc.refcounts().tolist() == [1, 2, 1, 3, 1, 1, 1, 1] and oc.free_list().tolist() == []
    st, Z = o.compose([c1, c2])
    assert (st, Z) == (0, 3)
    assert o.table(Z).tolist() == [int(x) for x in g["Z.table"].split()]
    assert o.ctx_len(Z) == 15
    pv = o.pool_view()
    for key in ("block4", "block0", "block5", "block2"):
        b = int(key[5:])
        for s, tok in enumerate(g[key].split()):
            for l in range(L):
                for kv in range(2):
                    got = bytes(pv[l, b, kv, s])
                    if tok == ".":
                        assert got == bytes(row), "a never-written slot must keep its initial bytes"
                    else:
                        assert got == token_row(names[tok], l, kv, row)
    assert o.stats()["rows_copied"] == int(g["rows_copied"])
    st, _ = o.evict([P, c2])
    assert st == 0
    assert o.refcounts().tolist() == [int(x) for x in g["refcount"].split()]
    assert o.free_list().tolist() == [int(x) for x in g["free_list"].split()]
    check_conservation(snapshot(o), NB, BS)


def _w2_state():
    """Steps 1-5 of the second worked example; returns (oracle, golden values, handles)."""
    g = _read_kv(os.path.join(GOLD, "worked_example_w2.txt"))
    NB, BS = int(g["NB"]), int(g["BS"])
    L, row = 2, 8
    o = paged.PagedOracle(L, 1, 4, BS, 2, NB, 6, 8, [int(x) for x in g["ring"].split()])
    names = {f"a{i}": i for i in range(8)}
    names.update({f"c{i}": 50 + i for i in range(5)})
    names["y0"] = 90
    enc = lambda toks: encode_tokens([names[t] for t in toks], L, row)
    ints = lambda key: [int(x) for x in g[key].split()]

    st, A = o.imp(enc([f"a{i}" for i in range(8)]), 8)
    assert (st, A) == (0, 0) and o.table(A).tolist() == ints("A.table")
    st, B = o.compose([A, A])
    assert (st, B) == (0, 1) and o.table(B).tolist() == ints("B.table")
    assert o.refcounts().tolist() == ints("refcount.after_compose")
    st, Cc = o.imp(enc([f"c{i}" for i in range(5)]), 5)
    assert (st, Cc) == (0, 2) and o.table(Cc).tolist() == ints("C.table")
    st, (D,) = o.fork(Cc, 1)
    assert (st, D) == (0, 3)
    assert o.append([D], [1], [enc(["y0"])])[0] == 0
    assert o.table(D).tolist() == ints("D.table")
    pv = o.pool_view()
    for s, tok in enumerate(g["block3"].split()):
        for l in range(L):
            for kv in range(2):
                want = bytes(row) if tok == "." else token_row(names[tok], l, kv, row)
                assert bytes(pv[l, 3, kv, s]) == want
    assert o.refcounts().tolist() == ints("refcount.before_evict")
    assert o.stats()["rows_copied"] == int(g["rows_copied.before_evict"])
    return o, g, (A, B, Cc, D)


def test_worked_example_w2_order_of_blocks_freed_by_one_evict():
    """Pins the push order of a batched evict: flattened (context, table position) order, a block
    pushed at its last occurrence -- with a block named twice by one victim and once more by another."""
    o, g, (A, B, Cc, D) = _w2_state()
    ints = lambda key: [int(x) for x in g[key].split()]
    assert o.evict([B, D, A])[0] == 0
    assert o.refcounts().tolist() == ints("refcount.after_evict")
    assert o.free_list().tolist() == ints("free_list.after_evict")
    assert o.live_ctxs() == ints("live.after_evict")
    check_conservation(snapshot(o), o.NB, o.BS)


def test_worked_example_w2_order_of_blocks_freed_by_scored_eviction():
    """The same pin for the scored eviction loop: victims oldest first, each victim's blocks released
    front to back, shared blocks survive until their last holder goes."""
    o, g, (A, B, Cc, D) = _w2_state()
    ints = lambda key: [int(x) for x in g[key].split()]
    assert o.materialize(A, 0, 8)[0] == 0
    st, victims = o.evict_to_budget(0.0, 0.0, 1.0, 3)
    assert st == 0 and victims == ints("budget.victims")
    assert o.refcounts().tolist() == ints("budget.refcount")
    assert o.free_list().tolist() == ints("budget.free_list")
    assert o.live_ctxs() == [A]
    check_conservation(snapshot(o), o.NB, o.BS)


# ---------------------------------------------------------------- P1 / P2: transfer preserves content


@pytest.mark.parametrize("n", [1, 3, 4, 5, 16, 17, 31, 33])
def test_materialize_of_import_is_identity(n):
    rng = np.random.default_rng(n)
    o = small_pool(order=rng.permutation(16))
    buf = rand_buf(rng, o, n)
    st, c = o.imp(buf, n)
    assert st == 0
    st, out = o.materialize(c, 0, n)
    assert st == 0 and np.array_equal(out, buf)
    # import(materialize(c)) is the same logical context
    st, c2 = o.imp(out, n)
    if st == 0:
        assert np.array_equal(o.materialize(c2, 0, n)[1], buf)
        assert set(o.table(c)).isdisjoint(set(o.table(c2)))


def test_materialize_equals_numpy_fancy_index():
    rng = np.random.default_rng(7)
    o = small_pool(NB=32, BS=4, L=3, H=2, D=4, max_blk=32, order=rng.permutation(32))
    n = 45
    st, c = o.imp(rand_buf(rng, o, n), n)
    assert st == 0
    table = o.table(c)
    pv = o.pool_view()  # [L, NB, 2, BS, row]
    # library routine: gather blocks, put K/V in front of the block axis, flatten tokens
    gathered = pv[:, table]  # [L, nblk, 2, BS, row]
    tokens = np.transpose(gathered, (0, 2, 1, 3, 4)).reshape(o.L, 2, len(table) * o.BS, o.row)
    for t0, t1 in [(0, n), (0, 1), (5, 22), (4, 8), (44, 45), (13, 45)]:
        st, out = o.materialize(c, t0, t1)
        assert st == 0
        assert np.array_equal(out.reshape(o.L, 2, t1 - t0, o.row), tokens[:, :, t0:t1])


# ---------------------------------------------------------------- P3: fork


@pytest.mark.parametrize("n,k", [(6, 1), (8, 3), (13, 5)])
def test_fork_aliases_blocks_and_copies_nothing(n, k):
    rng = np.random.default_rng(n * 10 + k)
    o = small_pool(order=rng.permutation(16))
    st, p = o.imp(rand_buf(rng, o, n), n)
    before = snapshot(o)
    image = o.pool_view().copy()
    st, kids = o.fork(p, k)
    assert st == 0 and len(kids) == k
    after = snapshot(o)
    assert np.array_equal(o.pool_view(), image), "fork must not touch pool bytes"
    assert after["free_list"] == before["free_list"], "fork must not allocate"
    for c in kids:
        assert after["tables"][c] == before["tables"][p] and after["lens"][c] == n
    for b in range(o.NB):
        mult = before["tables"][p].count(b)
        assert after["refcounts"][b] == before["refcounts"][b] + k * mult
    check_conservation(after, o.NB, o.BS)


# ---------------------------------------------------------------- P4 / P7: append and copy-on-write


@pytest.mark.parametrize("T,n_new", [(6, 3), (8, 3), (5, 1), (7, 9), (4, 4), (3, 1)])
def test_append_never_mutates_the_parent(T, n_new):
    rng = np.random.default_rng(T * 31 + n_new)
    o = small_pool(order=rng.permutation(16))
    base = rand_buf(rng, o, T)
    st, p = o.imp(base, T)
    st, (a, b) = o.fork(p, 2)
    free0 = len(o.free_list())
    x = rand_buf(rng, o, n_new)
    st, _ = o.append([a], [n_new], [x])
    assert st == 0
    cow = 1 if T % o.BS else 0
    used = free0 - len(o.free_list())
    assert used == cow + (-(-(T + n_new) // o.BS)) - (-(-T // o.BS))
    assert o.stats()["cow_count"] == cow
    assert np.array_equal(o.materialize(p, 0, T)[1], base)
    assert np.array_equal(o.materialize(b, 0, T)[1], base)
    got = o.materialize(a, 0, T + n_new)[1].reshape(o.L, 2, T + n_new, o.row)
    assert np.array_equal(got[:, :, :T], base.reshape(o.L, 2, T, o.row))
    assert np.array_equal(got[:, :, T:], x.reshape(o.L, 2, n_new, o.row))
    # the full shared blocks stay aliased
    full = T // o.BS
    assert o.table(a)[:full].tolist() == o.table(p)[:full].tolist()
    check_conservation(snapshot(o), o.NB, o.BS)


def test_unshared_tail_is_written_in_place():
    rng = np.random.default_rng(3)
    o = small_pool()
    st, c = o.imp(rand_buf(rng, o, 6), 6)
    t0 = o.table(c).tolist()
    st, _ = o.append([c], [1], [rand_buf(rng, o, 1)])
    assert o.table(c).tolist() == t0 and o.stats()["cow_count"] == 0


def test_live_blocks_grow_with_continuation_not_with_context():
    # fork k + aligned append n: live = nblk(T) + k * nblk(n), not k * nblk(T + n)
    rng = np.random.default_rng(11)
    T, k, n = 32, 5, 8
    o = small_pool(NB=64, max_blk=32, max_ctx=8)
    st, p = o.imp(rand_buf(rng, o, T), T)
    st, kids = o.fork(p, k)
    st, _ = o.append(kids, [n] * k, [rand_buf(rng, o, n) for _ in kids])
    assert st == 0
    assert o.stats()["live_blocks"] == T // 4 + k * (n // 4)
    assert o.stats()["live_blocks"] < k * ((T + n) // 4)


def test_batched_append_equals_loop_of_single_appends():
    rng = np.random.default_rng(5)
    for T in (6, 8, 11):
        a = small_pool(NB=32, order=np.random.default_rng(1).permutation(32))
        b = small_pool(NB=32, order=np.random.default_rng(1).permutation(32))
        base = rand_buf(rng, a, T)
        xs = [rand_buf(rng, a, n) for n in (1, 5, 2, 7)]
        for o in (a, b):
            st, p = o.imp(base, T)
            st, kids = o.fork(p, 3)
        st, _ = a.append([p] + kids, [1, 5, 2, 7], xs)  # parent first: it must COW too (refcount 4)
        assert st == 0
        for c, n, x in zip([p] + kids, [1, 5, 2, 7], xs):
            assert b.append([c], [n], [x])[0] == 0
        assert snapshot(a) == snapshot(b)
        assert np.array_equal(a.pool_view(), b.pool_view())
        # the last sharer of the old tail finds refcount 1 and writes in place
        assert a.stats()["cow_count"] == (3 if T % 4 else 0)


# ---------------------------------------------------------------- P5: compose


def _ctx_bytes(o, c):
    n = o.ctx_len(c)
    return o.materialize(c, 0, n)[1].reshape(o.L, 2, n, o.row)


@pytest.mark.parametrize("lens", [(8, 8), (8, 5), (5, 8), (6, 7), (3, 1), (1, 1), (9, 4, 6), (4, 3, 8, 2)])
@pytest.mark.parametrize("flags", [0, paged.COMPOSE_COPY_ALL])
def test_compose_is_concatenation(lens, flags):
    rng = np.random.default_rng(sum(lens) + flags)
    o = small_pool(NB=32, max_blk=16, order=rng.permutation(32))
    cs = [o.imp(rand_buf(rng, o, n), n)[1] for n in lens]
    before = {c: _ctx_bytes(o, c).copy() for c in cs}
    tabs = {c: o.table(c).tolist() for c in cs}
    st, z = o.compose(cs, flags)
    assert st == 0
    assert np.array_equal(_ctx_bytes(o, z), np.concatenate([before[c] for c in cs], axis=2))
    for c in cs:  # sources stay live and unchanged
        assert np.array_equal(_ctx_bytes(o, c), before[c]) and o.table(c).tolist() == tabs[c]
    check_conservation(snapshot(o), o.NB, o.BS)
    if flags:
        assert set(o.table(z)).isdisjoint(set().union(*tabs.values()))
    elif all(n % o.BS == 0 for n in lens):
        assert o.table(z).tolist() == sum((tabs[c] for c in cs), [])  # table-only compose


def test_compose_of_one_is_fork_of_one():
    rng = np.random.default_rng(2)
    a, b = small_pool(), small_pool()
    buf = rand_buf(rng, a, 7)
    ca, cb = a.imp(buf, 7)[1], b.imp(buf, 7)[1]
    assert a.compose([ca])[0] == 0 and b.fork(cb, 1)[0] == 0
    assert snapshot(a) == snapshot(b)
    assert np.array_equal(a.pool_view(), b.pool_view())


def test_compose_is_associative_in_content_and_allows_repeats():
    rng = np.random.default_rng(9)
    o = small_pool(NB=64, max_blk=32, max_ctx=12)
    a, b, c = (o.imp(rand_buf(rng, o, n), n)[1] for n in (5, 9, 6))
    ab = o.compose([a, b])[1]
    ab_c = o.compose([ab, c])[1]
    abc = o.compose([a, b, c])[1]
    bc = o.compose([b, c])[1]
    a_bc = o.compose([a, bc])[1]
    assert np.array_equal(_ctx_bytes(o, ab_c), _ctx_bytes(o, abc))
    assert np.array_equal(_ctx_bytes(o, a_bc), _ctx_bytes(o, abc))
    aa = o.compose([a, a])[1]
    assert np.array_equal(_ctx_bytes(o, aa), np.concatenate([_ctx_bytes(o, a)] * 2, axis=2))
    check_conservation(snapshot(o), o.NB, o.BS)


# ---------------------------------------------------------------- P6: eviction


def test_evict_frees_exactly_the_unreferenced_blocks():
    rng = np.random.default_rng(4)
    o = small_pool(NB=32, order=rng.permutation(32))
    p = o.imp(rand_buf(rng, o, 10), 10)[1]
    kids = o.fork(p, 3)[1]
    o.append(kids[:2], [3, 6], [rand_buf(rng, o, 3), rand_buf(rng, o, 6)])
    z = o.compose([kids[0], kids[2]])[1]
    snap = snapshot(o)
    victims = [p, kids[0]]
    mult = {}
    for c in victims:
        for b in snap["tables"][c]:
            mult[b] = mult.get(b, 0) + 1
    expect_freed = {b for b, m in mult.items() if snap["refcounts"][b] == m}
    st, _ = o.evict(victims)
    assert st == 0
    after = snapshot(o)
    assert set(after["free_list"]) - set(snap["free_list"]) == expect_freed
    assert after["free_list"][: len(snap["free_list"])] == snap["free_list"]  # FIFO: old entries stay in front
    check_conservation(after, o.NB, o.BS)
    o.evict([kids[1], kids[2], z])
    assert sorted(o.free_list().tolist()) == list(range(o.NB))
    assert o.refcounts().sum() == 0 and o.live_ctxs() == []


# ---------------------------------------------------------------- P11: no stray writes


def test_bytes_outside_stored_tokens_are_never_written():
    rng = np.random.default_rng(8)
    o = small_pool(NB=32, order=rng.permutation(32))
    pv = o.pool_view()
    pv[:] = rng.integers(0, 256, size=pv.shape, dtype=np.uint8)
    image0 = pv.copy()
    written = np.zeros((o.NB, o.BS), dtype=bool)  # (block, slot) pairs some operator stored a token in

    def mark_new_tokens(c, first, count):
        t = o.table(c)
        for pos in range(first, first + count):
            written[t[pos // o.BS], pos % o.BS] = True

    p = o.imp(rand_buf(rng, o, 10), 10)[1]
    mark_new_tokens(p, 0, 10)
    kids = o.fork(p, 2)[1]
    o.append([kids[0]], [3], [rand_buf(rng, o, 3)])
    mark_new_tokens(kids[0], 8, 5)  # COW block holds positions 8..9 plus the 3 new tokens
    z = o.compose([kids[0], kids[1]])[1]
    tz, t0 = o.table(z), o.table(kids[0])
    first_fresh = next(i for i in range(len(tz)) if i >= len(t0) or tz[i] != t0[i])
    mark_new_tokens(z, first_fresh * o.BS, o.ctx_len(z) - first_fresh * o.BS)
    o.evict([p, kids[0], kids[1], z])
    now = np.transpose(o.pool_view(), (1, 3, 0, 2, 4))  # [NB, BS, L, 2, row]
    was = np.transpose(image0, (1, 3, 0, 2, 4))
    assert written.sum() < written.size
    assert np.array_equal(now[~written], was[~written])
    assert not np.array_equal(now[written], was[written])


# ---------------------------------------------------------------- failures change nothing


def test_failing_operators_change_no_state():
    rng = np.random.default_rng(6)
    o = small_pool(NB=6, BS=4, max_ctx=3, max_blk=4)
    a = o.imp(rand_buf(rng, o, 9), 9)[1]  # 3 blocks
    b = o.fork(a, 1)[1][0]
    image, snap = o.pool_view().copy(), snapshot(o)

    def unchanged():
        return snapshot(o) == snap and np.array_equal(o.pool_view(), image)

    assert o.imp(rand_buf(rng, o, 13), 13)[0] == paged.OOM_BLOCKS and unchanged()  # 4 blocks > 3 free
    assert o.imp(rand_buf(rng, o, 17), 17)[0] == paged.TOO_LONG and unchanged()
    assert o.append([a], [8], [rand_buf(rng, o, 8)])[0] == paged.TOO_LONG and unchanged()
    assert o.append([a, a], [1, 1], [rand_buf(rng, o, 1)] * 2)[0] == paged.INVALID_ARG and unchanged()
    assert o.append([2], [1], [rand_buf(rng, o, 1)])[0] == paged.BAD_CTX and unchanged()
    assert o.fork(a, 2)[0] == paged.OOM_CTX and unchanged()
    assert o.fork(a, 0)[0] == paged.INVALID_ARG and unchanged()
    assert o.materialize(a, 3, 3)[0] == paged.INVALID_ARG
    assert o.materialize(a, 0, 10)[0] == paged.INVALID_ARG
    assert o.materialize(2, 0, 1)[0] == paged.BAD_CTX
    assert o.evict([a, a])[0] == paged.INVALID_ARG and unchanged()
    assert o.evict([a, 2])[0] == paged.BAD_CTX and unchanged()
    assert o.compose([a, b])[0] == paged.TOO_LONG and unchanged()
    # batch append is all-or-nothing: with 2 free blocks, a (COW 1 + 1 new) fits alone, a then b (in place, 1 new) does not
    c = o.imp(rand_buf(rng, o, 2), 2)[1]
    image, snap = o.pool_view().copy(), snapshot(o)
    assert len(o.free_list()) == 2
    assert o.append([a, b], [4, 7], [rand_buf(rng, o, 4), rand_buf(rng, o, 7)])[0] == paged.OOM_BLOCKS and unchanged()
    assert o.compose([a])[0] == paged.OOM_CTX and unchanged()
    assert o.append([a], [4], [rand_buf(rng, o, 4)])[0] == 0 and not unchanged()


# ---------------------------------------------------------------- P9: exhaustive search on tiny pools


L_BF, ROW_BF, BS_BF = 1, 16, 2


def _menu(o, vm):
    live = sorted(vm.ctx.keys())
    ops = [("import", n) for n in (1, 2, 3, 4)]
    for c in live:
        ops += [("fork", c, k) for k in (1, 2)]
        ops += [("append", c, n) for n in (1, 2, 3)]
        ops += [("evict", c)]
    ops += [("compose", a, b) for a in live for b in live]
    return ops


def _apply(o, vm, op, next_tok):
    """apply op to both models; returns (status, next_tok). The paged oracle decides success."""
    free0 = len(o.free_list())
    snap0 = snapshot(o)
    kind = op[0]
    if kind == "import":
        toks = list(range(next_tok, next_tok + op[1]))
        st, c = o.imp(encode_tokens(toks, L_BF, ROW_BF), op[1])
        need = -(-op[1] // BS_BF)
        if st == 0:
            assert vm.imp(toks) == c
            next_tok += op[1]
    elif kind == "fork":
        st, kids = o.fork(op[1], op[2])
        need = 0
        if st == 0:
            assert vm.fork(op[1], op[2]) == kids
    elif kind == "append":
        c, n = op[1], op[2]
        T = len(vm.ctx[c])
        toks = list(range(next_tok, next_tok + n))
        cow = 1 if (T % BS_BF and snap0["refcounts"][snap0["tables"][c][-1]] > 1) else 0
        need = cow + (-(-(T + n) // BS_BF)) - (-(-T // BS_BF))
        st, _ = o.append([c], [n], [encode_tokens(toks, L_BF, ROW_BF)])
        if st == 0:
            vm.append(c, toks)
            next_tok += n
    elif kind == "compose":
        st, z = o.compose([op[1], op[2]])
        need = None
        if st == 0:
            assert vm.compose([op[1], op[2]]) == z
    elif kind == "evict":
        st, _ = o.evict([op[1]])
        need = None
        if st == 0:
            vm.evict([op[1]])
    if st == 0:
        if need is not None:
            assert free0 - len(o.free_list()) == need
    else:
        assert snapshot(o) == snap0, "a failing operator changed state"
        if st == paged.OOM_BLOCKS and need is not None:
            assert free0 < need
        if st == paged.OOM_CTX:
            assert len(vm.ctx) + (op[2] if kind == "fork" else 1) > vm.max_ctx
    return st, next_tok


def _dfs(o, vm, next_tok, depth, counter):
    if depth == 0:
        return
    for op in _menu(o, vm):
        o2, vm2 = o.clone(), vm.clone()
        st, nt = _apply(o2, vm2, op, next_tok)
        counter[0] += 1
        if st == 0:
            check_conservation(snapshot(o2), o2.NB, BS_BF)
            check_against_value_model(o2, vm2, L_BF, ROW_BF)
            _dfs(o2, vm2, nt, depth - 1, counter)
        o2.close()


@pytest.mark.parametrize("NB,depth", [(3, 5), (4, 5), (5, 4), (6, 4)])
def test_exhaustive_operator_sequences_match_value_model(NB, depth):
    order = np.random.default_rng(NB).permutation(NB)
    o = paged.PagedOracle(L_BF, 1, 8, BS_BF, 2, NB, 3, 4, order)
    vm = ValueModel(3)
    counter = [0]
    _dfs(o, vm, 0, depth, counter)
    assert counter[0] > 1000


@pytest.mark.parametrize("seed", range(12))
def test_random_walks_match_value_model(seed):
    rng = np.random.default_rng(1000 + seed)
    NB = int(rng.integers(3, 12))
    o = paged.PagedOracle(L_BF, 1, 8, BS_BF, 2, NB, 4, 6, rng.permutation(NB))
    vm = ValueModel(4)
    nt = 0
    ok = 0
    for _ in range(200):
        menu = _menu(o, vm)
        op = menu[int(rng.integers(len(menu)))]
        st, nt = _apply(o, vm, op, nt)
        ok += st == 0
        check_conservation(snapshot(o), NB, BS_BF)
        check_against_value_model(o, vm, L_BF, ROW_BF)
    assert ok > 15


# ---------------------------------------------------------------- Alg. KV-Evict: score and budget loop


def _busy_pool(seed=21):
    """A pool with shared, forked, appended, composed contexts and a spread of reuse / age / size."""
    rng = np.random.default_rng(seed)
    o = small_pool(NB=64, BS=4, max_ctx=12, max_blk=32, order=rng.permutation(64))
    a = o.imp(rand_buf(rng, o, 10), 10)[1]
    b = o.imp(rand_buf(rng, o, 23), 23)[1]
    kids = o.fork(a, 3)[1]
    o.append([kids[0]], [5], [rand_buf(rng, o, 5)])
    o.materialize(b, 0, 23)
    o.materialize(b, 3, 9)
    z = o.compose([kids[1], b])[1]
    o.append([kids[2]], [9], [rand_buf(rng, o, 9)])
    o.materialize(kids[0], 0, 15)
    return o, rng


def test_catalog_counts_reads_and_stamps_the_clock():
    o, _ = _busy_pool()
    cat = o.catalog()
    # operators so far: import a(1) import b(2) fork(3) append(4) materialize b(5,6) compose(7) append(8) materialize(9)
    assert cat["clock"] == 9
    # handles: a=0 b=1 kids=2,3,4 z=5
    assert cat["reuse"][:6] == [1, 3, 1, 1, 0, 0]          # a: fork; b: 2 materialize + compose; k0: materialize; k1: compose
    assert cat["last_access"][:6] == [3, 7, 9, 7, 8, 7]
    assert cat["reuse"][6] == -1 and cat["last_access"][6] == -1


def _evict_in_order_until(o, order, budget):
    victims = []
    for c in order:
        if o.stats()["live_blocks"] <= budget:
            break
        assert o.evict([c])[0] == 0
        victims.append(c)
    return victims


@pytest.mark.parametrize("budget", [0, 5, 9, 14, 1000])
def test_age_only_score_is_lru(budget):
    o, _ = _busy_pool()
    ref = o.clone()
    cat = o.catalog()
    live = o.live_ctxs()
    lru_order = sorted(live, key=lambda c: (cat["last_access"][c], c))  # oldest first: largest age, lowest score
    st, victims = o.evict_to_budget(0.0, 0.0, 1.0, budget)
    assert st == 0
    assert victims == _evict_in_order_until(ref, lru_order, budget)
    a, b = snapshot(o), snapshot(ref)
    assert a == b and np.array_equal(o.pool_view(), ref.pool_view())
    check_conservation(a, o.NB, o.BS)
    if budget == 1000:
        assert victims == []
    if budget == 0:
        assert sorted(victims) == sorted(live) and sorted(o.free_list().tolist()) == list(range(o.NB))


def test_size_only_and_reuse_only_scores():
    o, _ = _busy_pool()
    ref = o.clone()
    live = o.live_ctxs()
    by_size = sorted(live, key=lambda c: (-(-(-o.ctx_len(c) // o.BS)), c))  # most blocks first
    st, victims = o.evict_to_budget(0.0, 1.0, 0.0, 6)
    assert victims == _evict_in_order_until(ref, by_size, 6) and snapshot(o) == snapshot(ref)
    o, _ = _busy_pool()
    ref = o.clone()
    cat = o.catalog()
    by_reuse = sorted(o.live_ctxs(), key=lambda c: (cat["reuse"][c], c))  # least reused first
    st, victims = o.evict_to_budget(1.0, 0.0, 0.0, 6)
    assert victims == _evict_in_order_until(ref, by_reuse, 6) and snapshot(o) == snapshot(ref)


@pytest.mark.parametrize("weights", [(1.5, 0.25, 0.1), (0.3, 2.0, 0.7), (10.0, 0.01, 3.3)])
def test_mixed_score_orders_victims_by_the_formula(weights):
    al, be, ga = weights
    o, _ = _busy_pool()
    ref = o.clone()
    cat = o.catalog()
    clock = cat["clock"] + 1  # the eviction call itself advances the clock before ages are taken
    score = {c: (al * cat["reuse"][c] - be * (-(-o.ctx_len(c) // o.BS))) - ga * (clock - cat["last_access"][c])
             for c in o.live_ctxs()}
    order = sorted(score, key=lambda c: (score[c], c))
    st, victims = o.evict_to_budget(al, be, ga, 7)
    assert st == 0 and victims == _evict_in_order_until(ref, order, 7)
    assert snapshot(o) == snapshot(ref)


def test_shared_prefix_survives_scored_eviction():
    rng = np.random.default_rng(5)
    o = small_pool(NB=32, BS=4, max_ctx=8, max_blk=16)
    p = o.imp(rand_buf(rng, o, 16), 16)[1]            # 4 blocks
    kids = o.fork(p, 3)[1]
    o.append(kids, [4, 4, 4], [rand_buf(rng, o, 4) for _ in kids])  # one private block each -> 7 live
    o.materialize(p, 0, 16)                           # the parent is the most recently used
    st, victims = o.evict_to_budget(0.0, 0.0, 1.0, 5)
    # evicting a child frees only its private block: two children go, the prefix stays with p and the third
    assert victims == kids[:2]
    assert o.stats()["live_blocks"] == 5
    assert np.array_equal(o.table(p), o.table(kids[2])[:4])
    assert o.evict_to_budget(0.0, 0.0, 1.0, -1)[0] == paged.INVALID_ARG


# ---------------------------------------------------------------- columnar catalog export


def test_catalog_export_is_an_arrow_list_of_block_rows():
    import pyarrow as pa

    o, _ = _busy_pool()
    cols = o.export_catalog()
    live = o.live_ctxs()
    cat = o.catalog()
    assert cols["state_id"].tolist() == live
    assert cols["n_tokens"].tolist() == [o.ctx_len(c) for c in live]
    assert cols["reuse"].tolist() == [cat["reuse"][c] for c in live]
    assert cols["last_access"].tolist() == [cat["last_access"][c] for c in live]
    tables = [o.table(c) for c in live]
    # offsets = running sum of the table lengths; block ids = the tables laid end to end (library routines)
    assert cols["block_offsets"].tolist() == [0] + np.cumsum([len(t) for t in tables]).tolist()
    assert np.array_equal(cols["block_id"], np.concatenate(tables))
    # the offsets and values buffers are a valid Arrow ListArray without any copy or conversion
    lst = pa.ListArray.from_arrays(pa.array(cols["block_offsets"], type=pa.int32()),
                                   pa.array(cols["block_id"], type=pa.int32()))
    lst.validate(full=True)
    assert lst.to_pylist() == [t.tolist() for t in tables]
    # position ranges tile [0, n_tokens) of each state in steps of the block size
    for i, c in enumerate(live):
        a, b = cols["block_offsets"][i], cols["block_offsets"][i + 1]
        begins, ends = cols["pos_begin"][a:b], cols["pos_end"][a:b]
        assert begins[0] == 0 and ends[-1] == o.ctx_len(c)
        assert np.array_equal(begins[1:], ends[:-1]) and np.all(ends - begins <= o.BS) and np.all(ends > begins)
        assert np.all((ends - begins)[:-1] == o.BS)
    assert np.array_equal(cols["refcount"], o.refcounts()[cols["block_id"]])
    # the address column locates the block's rows: layer 0, K, slot 0 of block b
    pv = o.pool_view()
    flat = pv.reshape(-1)
    for r in (0, len(cols["block_id"]) // 2, len(cols["block_id"]) - 1):
        b = int(cols["block_id"][r])
        addr = int(cols["address"][r])
        assert np.array_equal(flat[addr:addr + o.row], pv[0, b, 0, 0])


def test_catalog_export_of_an_empty_pool():
    o = small_pool()
    cols = o.export_catalog()
    assert cols["state_id"].size == 0 and cols["block_offsets"].tolist() == [0] and cols["block_id"].size == 0


def test_catalog_lineage_columns():
    """Lineage (how a state was produced, from which state): hand-derived for the sequence of _busy_pool:
    import a (clock 1), import b (2), fork a -> 2,3,4 (3), ..., compose [kid1, b] -> 5 (7)."""
    o, rng = _busy_pool()
    cols = o.export_catalog()
    assert cols["origin"].tolist() == [1, 1, 2, 2, 2, 3]          # 1 registered buffer, 2 fork, 3 merge
    assert cols["parent"].tolist() == [-1, -1, 0, 0, 0, 3]        # fork parent / first merged segment
    assert cols["born"].tolist() == [1, 2, 3, 3, 3, 7]
    assert cols["parent_born"].tolist() == [-1, -1, 1, 1, 1, 3]
    # a handle is reused after eviction; (handle, born) still tells the two states apart
    o.evict([0])                                                  # clock 10
    c = o.imp(rand_buf(rng, o, 3), 3)[1]                          # clock 11, takes handle 0 again
    assert c == 0
    cols = o.export_catalog()
    assert cols["born"].tolist()[0] == 11 and cols["origin"].tolist()[0] == 1
    assert cols["parent"].tolist()[2:5] == [0, 0, 0] and cols["parent_born"].tolist()[2:5] == [1, 1, 1]
