"""Churn workload: a seeded stream of agent operations under memory pressure (harness code).

64 agent slots; 10,000 operations drawn with the mix 30 % append, 20 % fork, 20 % compose,
15 % transfer (materialize / import), 15 % evict; segment lengths lognormal with median 2048 tokens.
The pool is capped at 75 % of the demand (= peak live blocks of the same seed on a pool that never
runs out), and the caller's eviction policy is LRU: when an operator reports out-of-blocks the
driver evicts the least recently used agent that the operator does not use and retries.  That
policy is the caller's side of Alg. "KV-Evict" (score = -age); the library only releases blocks.

The driver knows nothing about blocks: it tracks handles, token counts and LRU stamps, calls the
backend's operators and reacts to their status codes.  Because out-of-blocks is exact and a
failing operator changes nothing, two correct backends see the same call sequence; the driver
records every call with its status so that two runs can be compared call by call.

Payloads: every import/append reads a window of one pre-generated stream (workloads.fill, stream
1), so that generating inputs costs nothing per operation.  ``backend.window(op_index, n_tokens)``
returns the n-token transfer buffer that starts at element ``(op_index * 8) % slack`` of it.

Details the workload description leaves open and this driver fixes:
  * lengths = round(lognormal(mu = ln median, sigma = 0.8)) clamped to [1, max_seg_tokens];
  * contexts are capped at max_ctx_tokens (the runs use 32768, the paper's largest context): appends
    are shortened, trailing compose segments dropped;
  * a transfer operation is, with equal probability, a state arriving from elsewhere (import of a
    fresh segment) or a round trip of a live agent (materialize, then import of that buffer); without
    fresh arrivals every context descends from one root and all lengths drift to the cap;
  * compose takes 2-4 distinct live agents and releases them once their merge exists (the merged
    branches are done), so that merging does not only ever grow the population's lengths;
  * fork fan-out k in {1, 2, 4, 8}; new contexts go to the lowest empty slot, else they replace the
    least recently used slot the operator does not use; an operation on an empty system is an import.
"""
from __future__ import annotations

import math

import numpy as np

OOM_BLOCKS = -3
MAX_CTX_TOKENS = 65536
MAX_SEG_TOKENS = 16384
WINDOW_SLACK = 1 << 16  # elements


class ChurnDriver:
    def __init__(self, backend, seed: int, n_slots: int = 64, max_ctx_tokens: int = MAX_CTX_TOKENS,
                 median_tokens: float = 2048.0, max_seg_tokens: int = MAX_SEG_TOKENS, compose_consumes: bool = True):
        self.be = backend
        self.max_ctx_tokens, self.median, self.max_seg = max_ctx_tokens, median_tokens, max_seg_tokens
        self.compose_consumes = compose_consumes
        self.rng = np.random.default_rng(seed)
        self.slots = [None] * n_slots  # each: [ctx, tokens, stamp]
        self.clock = 0
        self.log = []        # (call, args, status)
        self.counts = {}
        self.payload_tokens = 0

    # ------------------------------------------------------------------ bookkeeping
    def _live(self):
        return [i for i, s in enumerate(self.slots) if s is not None]

    def _touch(self, i):
        self.slots[i][2] = self.clock

    def _lru(self, exclude):
        cand = [i for i in self._live() if i not in exclude]
        if not cand:
            return None
        return min(cand, key=lambda i: (self.slots[i][2], self.slots[i][0]))

    def _call(self, name, fn, args):
        st, res = fn()
        self.log.append((name, args, st))
        self.counts[name] = self.counts.get(name, 0) + 1
        return st, res

    def _evict_slot(self, i):
        ctx = self.slots[i][0]
        st, _ = self._call("evict", lambda: self.be.evict([ctx]), (ctx,))
        assert st == 0, st
        self.slots[i] = None

    def _room(self, count, exclude):
        """slot indices for `count` new contexts: empty slots first, then LRU victims (evicted now)."""
        out = [i for i, s in enumerate(self.slots) if s is None][:count]
        while len(out) < count:
            v = self._lru(set(exclude) | set(out))
            if v is None:
                return None
            self._evict_slot(v)
            out.append(v)
        return out

    def _with_pressure(self, name, fn, args, exclude):
        """runs fn; on out-of-blocks evicts LRU agents the operator does not use and retries."""
        while True:
            st, res = self._call(name, fn, args)
            if st != OOM_BLOCKS:
                return st, res
            v = self._lru(exclude)
            if v is None:
                return st, res
            self._evict_slot(v)

    def _seg_len(self):
        n = int(round(float(self.rng.lognormal(math.log(self.median), 0.8))))
        return max(1, min(self.max_seg, n))

    # ------------------------------------------------------------------ operations
    def _import_new(self):
        n = self._seg_len()
        dest = self._room(1, [])
        buf = self.be.window(self.clock, n)
        st, ctx = self._with_pressure("import", lambda: self.be.imp(buf, n), (n,), set(dest))
        if st == 0:
            self.slots[dest[0]] = [ctx, n, self.clock]
            self.payload_tokens += n

    def step(self):
        self.clock += 1
        u = float(self.rng.random())
        live = self._live()
        if not live:
            return self._import_new()
        if u < 0.30:  # append
            i = int(self.rng.choice(live))
            n = min(self._seg_len(), self.max_ctx_tokens - self.slots[i][1])
            if n < 1:
                return
            ctx = self.slots[i][0]
            buf = self.be.window(self.clock, n)
            st, _ = self._with_pressure("append", lambda: self.be.append([ctx], [n], [buf]), (ctx, n), {i})
            if st == 0:
                self.slots[i][1] += n
                self._touch(i)
                self.payload_tokens += n
        elif u < 0.50:  # fork
            i = int(self.rng.choice(live))
            k = int(self.rng.choice([1, 2, 4, 8]))
            dest = self._room(k, [i])
            if dest is None:
                return
            ctx, n = self.slots[i][0], self.slots[i][1]
            st, kids = self._call("fork", lambda: self.be.fork(ctx, k), (ctx, k))
            if st == 0:
                self._touch(i)
                for d, c in zip(dest, kids):
                    self.slots[d] = [c, n, self.clock]
        elif u < 0.70:  # compose
            m = min(int(self.rng.choice([2, 3, 4])), len(live))
            segs = [int(x) for x in self.rng.choice(live, size=m, replace=False)]
            total, keep = 0, []
            for s in segs:
                if total + self.slots[s][1] > self.max_ctx_tokens:
                    break
                keep.append(s)
                total += self.slots[s][1]
            if not keep:
                return
            dest = self._room(1, keep)
            if dest is None:
                return
            handles = [self.slots[s][0] for s in keep]
            st, ctx = self._with_pressure("compose", lambda: self.be.compose(handles, 0), tuple(handles),
                                          set(keep) | set(dest))
            if st == 0:
                for s in keep:
                    self._touch(s)
                self.slots[dest[0]] = [ctx, total, self.clock]
                if self.compose_consumes:  # the merged branches are released once their merge exists
                    for s in keep:
                        self._evict_slot(s)
        elif u < 0.85 and float(self.rng.random()) < 0.5:  # transfer in: a state arrives from elsewhere
            return self._import_new()
        elif u < 0.85:  # transfer round trip: pack, then register the buffer as a new context
            i = int(self.rng.choice(live))
            ctx, n = self.slots[i][0], self.slots[i][1]
            st, buf = self._call("materialize", lambda: self.be.materialize(ctx, 0, n), (ctx, 0, n))
            assert st == 0, st
            self._touch(i)
            dest = self._room(1, [i])
            if dest is None:
                return
            st, c2 = self._with_pressure("import", lambda: self.be.imp(buf, n), (n,), {i} | set(dest))
            if st == 0:
                self.slots[dest[0]] = [c2, n, self.clock]
        else:  # evict the least recently used agent
            v = self._lru(set())
            if v is not None:
                self._evict_slot(v)

    def run(self, n_ops: int, checkpoint_every: int = 0, on_checkpoint=None):
        for i in range(n_ops):
            self.step()
            if checkpoint_every and (i + 1) % checkpoint_every == 0 and on_checkpoint:
                on_checkpoint(i + 1, self)
        return self


def churn_geometry(block_size: int, n_blocks: int, n_layers: int = 32):
    from .configs import Geometry

    return Geometry(n_layers, 8, 128, block_size, 2, n_blocks, 80, MAX_CTX_TOKENS // block_size)


def unbounded_blocks(block_size: int) -> int:
    """pool size for the demand pass: large enough that the trace never runs out of blocks"""
    return 65536 * 16 // block_size
