"""Test-side adapters: the CPU oracle behind the replay-backend interface, state snapshots
and the convention-free checks (value-model equality, reference-count conservation)."""
from __future__ import annotations

import numpy as np

from oracle import paged
from oracle.value_model import ValueModel
from workloads import fill
from workloads.configs import Geometry


class OracleBackend:
    """The paged CPU oracle restricted to a subset of layers.

    Layers are independent on this path (same block ids in every layer), so running
    the oracle on layers ``layers`` of a geometry gives the exact metadata of the
    full geometry and the exact bytes of those layers, at a fraction of the memory.
    """

    def __init__(self, g: Geometry, seed: int, layers=None, free_order=None, init_fill=True):
        self.g = g
        self.seed_ = seed
        self.layers = list(range(g.n_layers)) if layers is None else list(layers)
        self.o = paged.PagedOracle(len(self.layers), g.n_kv_heads, g.head_dim, g.block_size, g.elt_bytes,
                                   g.n_blocks, g.max_ctx, g.max_blocks_per_ctx, free_order)
        if init_fill and init_fill != "zero":  # "zero": keep the all-zero image the oracle starts with
            pv = self.o.pool_view()
            per_layer = g.layer_stride // 2  # elements
            step = 1 << 24  # elements per chunk: keeps the generator's temporaries small
            for i, l in enumerate(self.layers):
                flat = pv[i].reshape(-1).view(np.uint16)
                for a in range(0, per_layer, step):
                    c = min(step, per_layer - a)
                    flat[a:a + c] = fill.fill_np(seed, 0, l * per_layer + a, c)

    def payload(self, seed, stream, n):
        g = self.g
        per_layer = 2 * n * g.row // 2  # elements of one layer of the [L,2,n,H,D] buffer
        parts = [fill.fill_np(seed, stream, l * per_layer, per_layer) for l in self.layers]
        return np.concatenate(parts).view(np.uint8)

    def window(self, op_index, n):
        """n-token payload read from a window of stream 1 (churn workload): the same elements the GPU
        backend's window holds, restricted to this oracle's layers."""
        from workloads.churn import MAX_SEG_TOKENS, WINDOW_SLACK

        g = self.g
        hd = g.row // 2
        if getattr(self, "_big", None) is None:
            total = g.n_layers * 2 * MAX_SEG_TOKENS * hd + WINDOW_SLACK
            self._big = np.empty(total, dtype=np.uint16)
            for a in range(0, total, 1 << 24):
                c = min(1 << 24, total - a)
                self._big[a:a + c] = fill.fill_np(self.seed_, 1, a, c)
        o = (op_index * 8) % WINDOW_SLACK
        per_layer = 2 * n * hd
        return np.concatenate([self._big[o + l * per_layer: o + (l + 1) * per_layer] for l in self.layers]).view(np.uint8)

    def imp(self, buf, n):
        return self.o.imp(buf, n)

    def materialize(self, c, t0, t1):
        return self.o.materialize(c, t0, t1)

    def fork(self, c, k):
        return self.o.fork(c, k)

    def append(self, ctxs, n_new, bufs):
        return self.o.append(ctxs, n_new, bufs)

    def compose(self, ctxs, flags):
        return self.o.compose(ctxs, flags)

    def evict(self, ctxs):
        return self.o.evict(ctxs)

    def snapshot(self):
        return snapshot(self.o)


def check_conservation(snap: dict, n_blocks: int, block_size: int):
    """Reference-count conservation, recounted from the tables alone:
    refcount[b] = number of table entries naming b; free ring = exactly the
    unreferenced blocks, each once; table lengths match the token counts."""
    counts = [0] * n_blocks
    for c, t in snap["tables"].items():
        assert len(t) == -(-snap["lens"][c] // block_size), (c, len(t), snap["lens"][c])
        for b in t:
            assert 0 <= b < n_blocks
            counts[b] += 1
    assert counts == snap["refcounts"]
    fl = snap["free_list"]
    assert len(set(fl)) == len(fl), "a block is on the free ring twice"
    assert set(fl) == {b for b in range(n_blocks) if counts[b] == 0}
    assert sum(snap["refcounts"]) == sum(len(t) for t in snap["tables"].values())


def token_row(tok: int, l: int, kv: int, row_bytes: int) -> bytes:
    """Distinct, recognisable bytes for token id `tok` (tests with named tokens)."""
    base = tok * 131 + l * 17 + kv * 7
    return bytes((base + 3 * i) % 251 for i in range(row_bytes))


def encode_tokens(tokens, n_layers: int, row_bytes: int) -> np.ndarray:
    from oracle.value_model import encode

    return encode(tokens, lambda t, l, kv: token_row(t, l, kv, row_bytes), n_layers, row_bytes).reshape(-1)


def check_against_value_model(o, vm: ValueModel, n_layers: int, row_bytes: int):
    """Every live context of the paged oracle materialises to the value model's sequence."""
    assert sorted(o.live_ctxs()) == sorted(vm.ctx.keys())
    for c, seq in vm.ctx.items():
        assert o.ctx_len(c) == len(seq)
        st, buf = o.materialize(c, 0, len(seq))
        assert st == 0
        assert np.array_equal(buf, encode_tokens(seq, n_layers, row_bytes)), f"ctx {c} differs from value model"


class ProvenanceBackend:
    """The value model behind the replay-backend interface: tokens are (stream, t, n)
    triples naming element t of an n-token payload stream, so expected bytes of any
    token can be regenerated from workloads.fill without holding data."""

    def __init__(self, g: Geometry):
        self.g = g
        self.vm = ValueModel(g.max_ctx)

    def payload(self, seed, stream, n):
        return [(stream, t, n) for t in range(n)]

    def imp(self, buf, n):
        assert len(buf) == n
        return 0, self.vm.imp(buf)

    def materialize(self, c, t0, t1):
        return 0, self.vm.materialize(c, t0, t1)

    def fork(self, c, k):
        return 0, self.vm.fork(c, k)

    def append(self, ctxs, n_new, bufs):
        for c, b in zip(ctxs, bufs):
            self.vm.append(c, b)
        return 0, None

    def compose(self, ctxs, flags):
        return 0, self.vm.compose(ctxs)

    def evict(self, ctxs):
        self.vm.evict(ctxs)
        return 0, None


def expected_bytes(seed: int, g: Geometry, tokens, layers=None) -> np.ndarray:
    """uint8 [len(layers), 2, len(tokens), row]: the transfer-buffer bytes of a sequence of
    provenance tokens (stream, t, n), regenerated from the fill function."""
    layers = list(range(g.n_layers)) if layers is None else list(layers)
    hd = g.n_kv_heads * g.head_dim
    assert g.elt_bytes == 2
    out = np.empty((len(layers), 2, len(tokens), hd), dtype=np.uint16)
    streams = np.array([t[0] for t in tokens], dtype=np.int64)
    tt = np.array([t[1] for t in tokens], dtype=np.int64)
    nn = np.array([t[2] for t in tokens], dtype=np.int64)
    lane = np.arange(hd, dtype=np.int64)
    for s in np.unique(streams):
        sel = np.nonzero(streams == s)[0]
        for i, l in enumerate(layers):
            for kv in range(2):
                idx = (((l * 2 + kv) * nn[sel] + tt[sel]) * hd)[:, None] + lane[None, :]
                out[i, kv, sel] = fill.fill_np_at(seed, int(s), idx)
    return out.view(np.uint8).reshape(len(layers), 2, len(tokens), g.row)


from tests.gpu_backend import GpuBackend, snapshot  # noqa: E402,F401  (re-exported for the tests)
