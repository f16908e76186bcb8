"""Shapes and explicit operator lists of the synthetic multi-agent KV workloads.

Pure data producers: a workload is a geometry plus a list of operator records that
any backend (the CPU oracle in the tests, the CUDA library everywhere else) replays
through ``workloads.replay``.  Nothing here computes what an operator does.

The shapes stand in for the paper's shared-prefix fan-out experiments
(root context -> materialize -> fork -> agents -> merge; contexts of 1K-32K tokens,
2-16 agents, Llama-3-8B / Mistral-7B KV shape), whose prompts and weights are not
needed because the path moves opaque bytes.

Operator records (ctx names are symbolic; the replayer binds them to the ids the
backend returns):
    {"op": "import",      "out": name, "n": tokens, "stream": payload stream id}
    {"op": "materialize", "ctx": name, "t0": a, "t1": b, "out_buf": bufname}
    {"op": "import_buf",  "out": name, "buf": bufname}          # import a materialised buffer
    {"op": "fork",        "ctx": name, "k": k, "out": [names]}
    {"op": "append",      "ctxs": [names], "n_new": [...], "streams": [...]}
    {"op": "compose",     "segs": [names], "flags": 0|1, "out": name}
    {"op": "evict",       "ctxs": [names]}
    {"op": "drop_buf",    "buf": bufname}
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

SEED_BASE = 0xA0F10000
COMPOSE_COPY_ALL = 1


@dataclass(frozen=True)
class Geometry:
    n_layers: int
    n_kv_heads: int
    head_dim: int
    block_size: int
    elt_bytes: int
    n_blocks: int
    max_ctx: int
    max_blocks_per_ctx: int

    @property
    def row(self) -> int:  # bytes of one token, one layer, K or V
        return self.n_kv_heads * self.head_dim * self.elt_bytes

    @property
    def run(self) -> int:  # bytes of one block, one layer, K or V
        return self.block_size * self.row

    @property
    def bpt(self) -> int:  # bytes per token over all layers, K and V
        return 2 * self.n_layers * self.row

    @property
    def layer_stride(self) -> int:
        return self.n_blocks * 2 * self.run

    @property
    def pool_bytes(self) -> int:
        return self.n_layers * self.layer_stride

    def nblk(self, tokens: int) -> int:
        return -(-tokens // self.block_size)

    def with_layers(self, n_layers: int) -> "Geometry":
        return replace(self, n_layers=n_layers)


TINY = Geometry(2, 2, 64, 16, 2, 256, 16, 128)
LLAMA8B = Geometry(32, 8, 128, 16, 2, 32768, 64, 4096)
LLAMA70B = Geometry(80, 8, 128, 16, 2, 8192, 32, 8192)


def free_order(seed: int, n_blocks: int) -> np.ndarray:
    """Seeded-permuted ("fragmented") initial free list."""
    return np.random.default_rng(seed).permutation(n_blocks).astype(np.int32)


def fanout_ops(context_tokens: int, n_agents: int, append_tokens: int, *, compose_pair: bool, evict_all: bool,
               roundtrip: bool, batched_append: bool = True):
    """Shared-prefix fan-out: import -> [materialize -> import] -> fork -> append -> [compose] -> [evict].

    With ``roundtrip`` the forked context is the re-imported copy (the "receiver's"
    side of a transfer); the sender's context stays live beside it.
    """
    ops = [{"op": "import", "out": "root", "n": context_tokens, "stream": 1}]
    live = ["root"]
    parent = "root"
    if roundtrip:
        ops += [
            {"op": "materialize", "ctx": "root", "t0": 0, "t1": context_tokens, "out_buf": "xfer"},
            {"op": "import_buf", "out": "recv", "buf": "xfer"},
            {"op": "drop_buf", "buf": "xfer"},
        ]
        live.append("recv")
        parent = "recv"
    else:
        ops.append({"op": "materialize", "ctx": "root", "t0": 0, "t1": context_tokens, "out_buf": "xfer"})
        ops.append({"op": "drop_buf", "buf": "xfer"})
    agents = [f"agent{i}" for i in range(n_agents)]
    ops.append({"op": "fork", "ctx": parent, "k": n_agents, "out": agents})
    live += agents
    if batched_append:
        ops.append({"op": "append", "ctxs": agents, "n_new": [append_tokens] * n_agents,
                    "streams": [2 + i for i in range(n_agents)]})
    else:
        for i, a in enumerate(agents):
            ops.append({"op": "append", "ctxs": [a], "n_new": [append_tokens], "streams": [2 + i]})
    for a in agents:
        ops.append({"op": "materialize", "ctx": a, "t0": 0, "t1": context_tokens + append_tokens, "out_buf": "m_" + a})
        ops.append({"op": "drop_buf", "buf": "m_" + a})
    ops.append({"op": "materialize", "ctx": parent, "t0": 0, "t1": context_tokens, "out_buf": "m_parent"})
    ops.append({"op": "drop_buf", "buf": "m_parent"})
    if compose_pair:
        ops.append({"op": "compose", "segs": agents[:2], "flags": 0, "out": "merged"})
        live.append("merged")
        ops.append({"op": "materialize", "ctx": "merged", "t0": 0, "t1": 2 * (context_tokens + append_tokens),
                    "out_buf": "m_merged"})
        ops.append({"op": "drop_buf", "buf": "m_merged"})
    if evict_all:
        ops.append({"op": "evict", "ctxs": list(live)})
    return ops


def config1(unaligned: bool = False):
    """Tiny pool: 512-token shared context, 4 agents x 64 appended tokens, agents 0+1 composed, all evicted."""
    T = 507 if unaligned else 512
    return TINY, SEED_BASE + 1, fanout_ops(T, 4, 64, compose_pair=True, evict_all=True, roundtrip=False)


def config2(unaligned: bool = False, geometry: Geometry = LLAMA8B, batched_append: bool = True):
    """Llama-3-8B-shaped: 8192-token context, transfer round trip, 16 agents x 512 appended tokens."""
    T = 8187 if unaligned else 8192
    return geometry, SEED_BASE + 2, fanout_ops(T, 16, 512, compose_pair=False, evict_all=False, roundtrip=True,
                                               batched_append=batched_append)


def config4(unaligned: bool = False, geometry: Geometry = LLAMA70B):
    """Llama-3-70B-shaped: 32768-token context, round trip, 8 agents x 1024 appended tokens."""
    T = 32763 if unaligned else 32768
    return geometry, SEED_BASE + 4, fanout_ops(T, 8, 1024, compose_pair=False, evict_all=False, roundtrip=True)


def config3(geometry: Geometry = LLAMA8B, copy_all: bool = False, lo: int = 1024, hi: int = 4096):
    """Composition-heavy: 16 private contexts with non-aligned lengths in [lo, hi], composed in pairs,
    quads, all 16 (tree) and flat (all 16 at once)."""
    seed = SEED_BASE + 3
    rng = np.random.default_rng(seed)
    lens = []
    while len(lens) < 16:
        n = int(rng.integers(lo, hi, endpoint=True))
        if n % geometry.block_size != 0:
            lens.append(n)
    order = rng.permutation(16).tolist()
    ops = []
    for i in order:  # imported in shuffled order: blocks scattered over the permuted pool
        ops.append({"op": "import", "out": f"a{i}", "n": lens[i], "stream": 1 + i})
    fl = COMPOSE_COPY_ALL if copy_all else 0
    for i in range(8):
        ops.append({"op": "compose", "segs": [f"a{2*i}", f"a{2*i+1}"], "flags": fl, "out": f"p{i}", "level": "pairs"})
    for i in range(4):
        ops.append({"op": "compose", "segs": [f"p{2*i}", f"p{2*i+1}"], "flags": fl, "out": f"q{i}", "level": "quads"})
    ops.append({"op": "compose", "segs": ["q0", "q1", "q2", "q3"], "flags": fl, "out": "all_tree", "level": "all16"})
    ops.append({"op": "compose", "segs": [f"a{i}" for i in range(16)], "flags": fl, "out": "all_flat", "level": "flat16"})
    total = sum(lens)
    for name in ["all_tree", "all_flat"]:
        ops.append({"op": "materialize", "ctx": name, "t0": 0, "t1": total, "out_buf": "m_" + name})
        ops.append({"op": "drop_buf", "buf": "m_" + name})
    return geometry, seed, ops, lens


def cow_stress_ops(context_tokens: int = 8187, n_children: int = 1024):
    """One unaligned context forked to many children, then one batched 1-token append: every child
    copies the partial tail block on write."""
    kids = [f"k{i}" for i in range(n_children)]
    return [
        {"op": "import", "out": "root", "n": context_tokens, "stream": 1},
        {"op": "fork", "ctx": "root", "k": n_children, "out": kids},
        {"op": "append", "ctxs": kids, "n_new": [1] * n_children, "streams": [2 + i for i in range(n_children)]},
    ]
