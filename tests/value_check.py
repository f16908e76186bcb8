"""Convention-free check of the CUDA library at full size: the value model beside the library.

The value model (oracle/value_model.py) knows nothing about blocks: a context is a sequence of tokens.
``ShadowBackend`` runs every operator on the CUDA library and, when it succeeds, on the value model,
with tokens named by their provenance ``(stream, t, n, base)``: token ``t`` of an ``n``-token payload
whose element ``(l, kv, t, lane)`` is element ``base + ((2 l + kv) n + t) hd + lane`` of fill stream
``stream``.  The bytes a materialisation must return are then regenerated ON THE DEVICE from the fill
function (workloads.fill) for EVERY layer, so that all of a transfer buffer is compared at HBM speed,
not a sample of its layers.  Nothing here depends on block ids, free-list order or handles beyond the
smallest-free-handle rule the value model shares.
"""
from __future__ import annotations

import numpy as np

from oracle.value_model import ValueModel
from workloads import fill


def token_tensor(seed, tokens, device):
    """(keys, t, n, base) int64 tensors of a provenance token list (stream, t, n, base)."""
    import torch

    tok = torch.from_numpy(np.asarray(tokens, dtype=np.int64).reshape(len(tokens), 4)).to(device)
    streams, inv = torch.unique(tok[:, 0], return_inverse=True)
    keys = torch.tensor([fill.key_s64(seed, int(s)) for s in streams.tolist()], dtype=torch.int64, device=device)[inv]
    return keys, tok[:, 1], tok[:, 2], tok[:, 3]


def expected_plane(tt, l, kv, hd, q):
    """int16 [n_tokens, hd]: plane (layer l, K/V kv) of the transfer buffer that encodes the token sequence."""
    import torch

    keys, t, nn, base = tt
    lane = torch.arange(hd, dtype=torch.int64, device=t.device)
    idx = (base + ((2 * l + kv) * nn + t) * hd)[:, None] + lane[None, :]
    return fill.fill_torch_at(keys[:, None], idx, q)


class Paired:
    """A transfer buffer on both sides: the device tensor and the token sequence it encodes."""

    def __init__(self, dev, tokens):
        self.dev, self.tokens = dev, tokens


class ShadowBackend:
    """Replay-backend interface over (GpuBackend, ValueModel)."""

    def __init__(self, gpu):
        self.gpu, self.g = gpu, gpu.g
        self.vm = ValueModel(gpu.g.max_ctx)
        self.q = fill.quantile_table_torch(gpu.o.device)
        self.planes_checked = 0

    # ---- payloads
    def payload(self, seed, stream, n):
        return Paired(self.gpu.payload(seed, stream, n), [(stream, t, n, 0) for t in range(n)])

    def window(self, op_index, n):
        from workloads.churn import WINDOW_SLACK

        base = (op_index * 8) % WINDOW_SLACK
        return Paired(self.gpu.window(op_index, n), [(1, t, n, base) for t in range(n)])

    # ---- operators: the library first; the value model follows only a success
    def imp(self, buf, n):
        st, c = self.gpu.imp(buf.dev, n)
        if st == 0:
            assert self.vm.imp(buf.tokens) == c, "handles differ from the smallest-free-handle rule"
        return st, c

    def materialize(self, c, t0, t1):
        st, out = self.gpu.materialize(c, t0, t1)
        return st, (Paired(out, self.vm.materialize(c, t0, t1)) if st == 0 else None)

    def fork(self, c, k):
        st, kids = self.gpu.fork(c, k)
        if st == 0:
            assert self.vm.fork(c, k) == kids
        return st, kids

    def append(self, ctxs, n_new, bufs):
        st, _ = self.gpu.append(ctxs, n_new, [b.dev for b in bufs])
        if st == 0:
            for c, b in zip(ctxs, bufs):
                self.vm.append(c, b.tokens)
        return st, None

    def compose(self, ctxs, flags):
        st, c = self.gpu.compose(ctxs, flags)
        if st == 0:
            assert self.vm.compose(ctxs) == c
        return st, c

    def evict(self, ctxs):
        st, _ = self.gpu.evict(ctxs)
        if st == 0:
            self.vm.evict(ctxs)
        return st, None

    # ---- checks
    def check_buffer(self, seed, buf: Paired):
        """Every (layer, K/V) plane of a materialised buffer equals the bytes its token sequence defines."""
        import torch

        g, dev = self.g, self.gpu.o.device
        n, hd = len(buf.tokens), g.row // 2
        assert g.elt_bytes == 2
        tt = token_tensor(seed, buf.tokens, dev)
        got = buf.dev[: n * g.bpt].view(torch.int16).view(g.n_layers, 2, n, hd)
        for l in range(g.n_layers):
            for kv in range(2):
                assert torch.equal(got[l, kv], expected_plane(tt, l, kv, hd, self.q)), \
                    f"layer {l} kv {kv} differs from the value model"
                self.planes_checked += 1

    def check_all_live(self, seed, scratch=None):
        """Value-model equality of every live context (all layers), and the same set of live handles."""
        import torch

        g = self.g
        assert sorted(self.gpu.o.live_ctxs()) == sorted(self.vm.ctx.keys())
        for c, seq in self.vm.ctx.items():
            assert self.gpu.o.ctx_len(c) == len(seq)
            out = scratch[: len(seq) * g.bpt] if scratch is not None else None
            st, dev_buf = self.gpu.o.materialize(c, 0, len(seq), out=out)
            assert st == 0
            self.check_buffer(seed, Paired(dev_buf, seq))
            del dev_buf
        torch.cuda.synchronize()
