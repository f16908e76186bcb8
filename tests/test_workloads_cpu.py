"""CPU checks of the input generators and of the workload operator lists replayed on the oracle."""
from __future__ import annotations

import numpy as np
import pytest
import torch

from tests.helpers import OracleBackend, ProvenanceBackend, check_conservation, expected_bytes
from workloads import configs, fill
from workloads.replay import replay


def test_fill_is_deterministic_and_looks_gaussian():
    a = fill.fill_np(123, 1, 0, 1 << 18)
    assert np.array_equal(a, fill.fill_np(123, 1, 0, 1 << 18))
    assert np.array_equal(a[1000:2000], fill.fill_np(123, 1, 1000, 1000))
    assert not np.array_equal(a, fill.fill_np(123, 2, 0, 1 << 18))
    assert not np.array_equal(a, fill.fill_np(124, 1, 0, 1 << 18))
    vals = torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).double().numpy()
    assert abs(vals.mean()) < 0.01 and abs(vals.std() - 1.0) < 0.01
    assert abs((np.abs(vals) < 1.0).mean() - 0.6827) < 0.01


def test_quantile_table_is_bf16_round_to_nearest_even():
    q = fill.quantile_table()
    assert q.shape == (65536,) and q.dtype == np.uint16
    from scipy.special import ndtri

    ref = torch.from_numpy(ndtri((np.arange(65536) + 0.5) / 65536.0).astype(np.float32)).to(torch.bfloat16)
    assert np.array_equal(ref.view(torch.int16).numpy().view(np.uint16), q)


@pytest.mark.parametrize("start,count", [(0, 1000), (12345, 70000), ((1 << 35) + 7, 4096)])
def test_fill_torch_matches_fill_np(start, count):
    a = fill.fill_np(77, 3, start, count)
    b = fill.fill_torch(77, 3, start, count, "cpu", chunk=30000).numpy().view(np.uint16)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("unaligned", [False, True])
def test_config1_on_oracle_matches_value_model(unaligned):
    g, seed, ops = configs.config1(unaligned)
    ob = OracleBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks))
    pb = ProvenanceBackend(g)
    cows = 0
    for (i, op, st, res, names), (_, _, st2, res2, names2) in zip(replay(ops, ob, seed), replay(ops, pb, seed)):
        assert st == 0 and st2 == 0, (i, op, st)
        assert names == names2, "context ids must follow the smallest-free-slot rule in both models"
        check_conservation(ob.snapshot(), g.n_blocks, g.block_size)
        if op["op"] == "materialize":
            want = expected_bytes(seed, g, res2)
            assert np.array_equal(res.reshape(want.shape), want), (i, op)
    assert ob.o.stats()["cow_count"] == (4 if unaligned else 0)
    assert sorted(ob.o.free_list().tolist()) == list(range(g.n_blocks))
    if not unaligned:  # literal config: the merge of two block-aligned agents is table-only
        assert ob.o.stats()["peak_live_blocks"] == 32 + 4 * 4


def test_config3_lengths_and_levels():
    g, seed, ops, lens = configs.config3(configs.LLAMA8B)
    assert len(lens) == 16 and all(1024 <= n <= 4096 and n % 16 for n in lens)
    assert sum(1 for o in ops if o["op"] == "compose") == 8 + 4 + 1 + 1


def test_device_side_expected_bytes_equal_the_numpy_ones():
    """The torch routine that regenerates a token sequence's transfer-buffer bytes (used on the GPU to compare
    every layer at full size) against the numpy one, on CPU tensors, with tokens from several payloads and a
    windowed payload."""
    import torch

    from tests.helpers import expected_bytes
    from tests.value_check import expected_plane, token_tensor
    from workloads import fill
    from workloads.configs import Geometry

    g = Geometry(3, 2, 8, 4, 2, 16, 4, 8)
    seed = 77
    tokens = [(1, t, 9, 0) for t in range(2, 9)] + [(5, t, 4, 0) for t in range(4)] + [(1, 0, 9, 0)]
    want = expected_bytes(seed, g, [tk[:3] for tk in tokens])
    q = fill.quantile_table_torch("cpu")
    tt = token_tensor(seed, tokens, "cpu")
    hd = g.row // 2
    for l in range(g.n_layers):
        for kv in range(2):
            got = expected_plane(tt, l, kv, hd, q).numpy().view(np.uint16)
            assert np.array_equal(got.view(np.uint8).reshape(len(tokens), g.row), want[l, kv])
    # a windowed payload: element index shifted by the window's base
    base, n = 40, 6
    tt = token_tensor(seed, [(1, t, n, base) for t in range(n)], "cpu")
    flat = fill.fill_np(seed, 1, base, g.n_layers * 2 * n * hd).reshape(g.n_layers, 2, n, hd)
    for l in range(g.n_layers):
        for kv in range(2):
            assert np.array_equal(expected_plane(tt, l, kv, hd, q).numpy().view(np.uint16), flat[l, kv])
