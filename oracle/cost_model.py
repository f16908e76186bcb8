"""Cost model of the state path -- TEST INFRASTRUCTURE, not the product.

The paper's formulas written out in plain Python floats (IEEE double), in the paper's order:

  state_bytes      |KV| = tokens * 2 (K and V) * layers * KV heads * head_dim * element bytes   (Sec. 3.2: a KV state
                   is the K and V blocks of every layer)
  transfer_time    T_transfer = |KV| / BW + delta                                (Sec. 5.4; Exp. 3)
  policy           pi(S) = reuse if the state is local and compatible, transfer if T_transfer < T_prefill, else
                   recompute                                                     (Sec. 4.6; App. C; App. E step 5)
  transfer_time_packed   T_transfer plus a pack at the sender and an unpack at the receiver, each moving 2 |KV|
                   bytes (read + written) at `pack_rate` bytes/s: the term the paper's model leaves out, the one
                   this build measures.  The definition is this build's, not the paper's; it is pinned by
                   hand-computed values (tests/golden/packed_transfer_example.txt) and by the special case of an
                   infinitely fast pack, which must leave the paper's T_transfer.
"""
from __future__ import annotations

REUSE, TRANSFER, RECOMPUTE = 0, 1, 2


def state_bytes(n_layers: int, n_kv_heads: int, head_dim: int, elt_bytes: int, n_tokens: int) -> int:
    return n_tokens * 2 * n_layers * n_kv_heads * head_dim * elt_bytes


def transfer_time(kv_bytes: float, bandwidth: float, latency: float) -> float:
    return float(kv_bytes) / float(bandwidth) + float(latency)


def transfer_time_packed(kv_bytes: float, bandwidth: float, latency: float, pack_rate: float) -> float:
    pack = 2.0 * float(kv_bytes) / float(pack_rate)
    return (pack + transfer_time(kv_bytes, bandwidth, latency)) + pack


def policy(local_and_compatible: bool, t_transfer: float, t_prefill: float) -> int:
    if local_and_compatible:
        return REUSE
    return TRANSFER if t_transfer < t_prefill else RECOMPUTE
