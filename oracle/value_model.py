"""Value model of the stateful KV operators -- TEST INFRASTRUCTURE, not the product.

The plain definition of what every operator means, with no pool, no blocks and no
reference counts: a context is a finite sequence of tokens and a token is an
opaque identifier.  The paged pool is only a faster representation of this model;
every byte a materialisation returns is defined here.

Passages followed (paper section / algorithm):
  import       Alg. "KV-Materialize" steps 4-6 and Alg. "KV-Transfer" (register received
               blocks): the registered state is the sequence the buffer encodes.
  materialize  Alg. "KV-Transfer" (select blocks by position range): transfer changes
               placement, never logical content (Sec. 3.3).
  fork         Alg. "KV-Fork": k logical children of the same prefix (Sec. 3.3).
  append       Alg. "KV-Resume": continuation tokens extend the state.
  compose      Alg. "Restricted-KV-Merge", concatenation branch: strictly sequential,
               non-overlapping concatenation (Sec. 4.5).
  evict        Alg. "KV-Evict": the logical state disappears.

Context ids follow the same convention as the paged oracle (smallest free slot), so
that one operator list can be replayed on both.
"""
from __future__ import annotations

OK = 0
INVALID_ARG = -1
BAD_CTX = -2
OOM_CTX = -4


class ValueModel:
    """Contexts as Python lists of token identifiers."""

    def __init__(self, max_ctx: int):
        self.max_ctx = max_ctx
        self.ctx: dict[int, list] = {}

    def _free_slots(self):
        return [c for c in range(self.max_ctx) if c not in self.ctx]

    def imp(self, tokens) -> int:
        tokens = list(tokens)
        assert len(tokens) >= 1
        c = self._free_slots()[0]
        self.ctx[c] = tokens
        return c

    def materialize(self, c: int, t0: int | None = None, t1: int | None = None) -> list:
        seq = self.ctx[c]
        t0 = 0 if t0 is None else t0
        t1 = len(seq) if t1 is None else t1
        assert 0 <= t0 < t1 <= len(seq)
        return list(seq[t0:t1])

    def fork(self, parent: int, k: int) -> list[int]:
        assert k >= 1
        slots = self._free_slots()[:k]
        assert len(slots) == k
        for c in slots:
            self.ctx[c] = list(self.ctx[parent])
        return slots

    def append(self, c: int, tokens) -> None:
        tokens = list(tokens)
        assert len(tokens) >= 1
        self.ctx[c] = self.ctx[c] + tokens

    def compose(self, segs) -> int:
        segs = list(segs)
        assert len(segs) >= 1
        out: list = []
        for s in segs:
            out = out + self.ctx[s]
        c = self._free_slots()[0]
        self.ctx[c] = out
        return c

    def evict(self, ctxs) -> None:
        for c in ctxs:
            del self.ctx[c]

    def clone(self) -> "ValueModel":
        v = ValueModel(self.max_ctx)
        v.ctx = {c: list(s) for c, s in self.ctx.items()}
        return v


def encode(tokens, row_of, n_layers: int, row_bytes: int):
    """Transfer-buffer encoding of a token sequence: dense bytes [L][2][n][row].

    ``row_of(token, layer, kv)`` returns the ``row_bytes`` bytes (a ``bytes`` object
    or a uint8 array) of one token's K (kv=0) or V (kv=1) row in one layer.
    """
    import numpy as np

    n = len(tokens)
    out = np.empty((n_layers, 2, n, row_bytes), dtype=np.uint8)
    for l in range(n_layers):
        for kv in range(2):
            for t, tok in enumerate(tokens):
                out[l, kv, t, :] = np.frombuffer(bytes(row_of(tok, l, kv)), dtype=np.uint8)
    return out
