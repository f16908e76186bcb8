"""The CUDA library behind the replay-backend interface of ``workloads.replay`` / ``workloads.churn``.

Harness code for the tests, the smoke check and the benchmark (not part of the product package): it owns a ``KVPool``, produces payloads on the device with
``workloads.fill`` and forwards every operator to the library.  Nothing is computed here.
"""
from __future__ import annotations

import numpy as np

from workloads import fill
from workloads.configs import Geometry


def snapshot(o) -> dict:
    """Everything observable about a pool except its bytes (works on the library's KVPool and on the oracle's
    PagedOracle: both expose the same introspection names)."""
    live = o.live_ctxs()
    return {
        "lens": {c: o.ctx_len(c) for c in live},
        "tables": {c: o.table(c).tolist() for c in live},
        "refcounts": o.refcounts().tolist(),
        "free_list": o.free_list().tolist(),
    }


class GpuBackend:
    """The CUDA library (through its Python binding) behind the replay-backend interface."""

    def __init__(self, g: Geometry, seed: int, free_order=None, engine: int = 0, init_fill=True, max_batch=0,
                 staging_tokens: int = 0):
        import torch

        from paper_2607_10987_b200.binding import KVPool

        self.g, self.torch, self.seed_ = g, torch, seed
        self._big = None
        self.o = KVPool(g.n_layers, g.n_kv_heads, g.head_dim, g.block_size, g.elt_bytes, g.n_blocks, g.max_ctx,
                        g.max_blocks_per_ctx, free_order=free_order, max_batch=max_batch)
        self.o.set_copy_engine(engine)
        if init_fill == "zero":  # all-zero pool image (matches a freshly created oracle pool)
            self.o.pool.zero_()
        elif init_fill:
            fill.fill_torch(seed, 0, 0, g.pool_bytes // 2, self.o.device, out=self.o.pool.view(torch.int16))
        self.staging = (torch.empty(staging_tokens * g.bpt, dtype=torch.uint8, device=self.o.device)
                        if staging_tokens else None)
        torch.cuda.synchronize()

    def window(self, op_index, n):
        """n-token payload read from a window of stream 1 (churn workload), 16-byte aligned."""
        from workloads.churn import MAX_SEG_TOKENS, WINDOW_SLACK

        g = self.g
        if self._big is None:
            total = g.n_layers * 2 * MAX_SEG_TOKENS * (g.row // 2) + WINDOW_SLACK
            self._big = fill.fill_torch(self.seed_, 1, 0, total, self.o.device)
        o = (op_index * 8) % WINDOW_SLACK
        return self._big[o:o + g.n_layers * 2 * n * (g.row // 2)].view(self.torch.uint8)

    def payload(self, seed, stream, n):
        g = self.g
        return fill.fill_torch(seed, stream, 0, g.n_layers * 2 * n * g.row // 2, self.o.device).view(self.torch.uint8)

    def imp(self, buf, n):
        return self.o.imp(buf, n)

    def materialize(self, c, t0, t1):
        if self.staging is not None and 0 <= t0 < t1 and (t1 - t0) * self.g.bpt <= self.staging.numel():
            return self.o.materialize(c, t0, t1, out=self.staging[: (t1 - t0) * self.g.bpt])
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

    def pool_layers(self, layers) -> np.ndarray:
        """uint8 [len(layers), NB, 2, BS, row] copy of the given layers of the device pool."""
        g = self.g
        v = self.o.pool[: g.pool_bytes].view(g.n_layers, g.n_blocks, 2, g.block_size, g.row)
        return v[list(layers)].cpu().numpy()

    def buf_layers(self, buf, n, layers) -> np.ndarray:
        """uint8 [len(layers), 2, n, row] copy of the given layers of a device transfer buffer."""
        g = self.g
        v = buf[: n * g.bpt].view(g.n_layers, 2, n, g.row)
        return v[list(layers)].cpu().numpy()
