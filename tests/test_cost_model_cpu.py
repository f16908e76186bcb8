"""Cost model of the state path: the oracle's formulas against what the paper prints, and the library's
host-only functions against the oracle (bit-exact in double precision).  No device is needed."""
from __future__ import annotations

import math
import os

import numpy as np
import pytest

import __graft_entry__ as entry
from oracle import cost_model as cm
from paper_2607_10987_b200 import binding

GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def _read(path):
    out = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=", 1)
            out[k.strip()] = v.strip()
    return out


def test_oracle_transfer_time_reproduces_the_printed_value():
    g = _read(os.path.join(GOLD, "transfer_time_max_context.txt"))
    kv = cm.state_bytes(int(g["n_layers"]), int(g["n_kv_heads"]), int(g["head_dim"]), int(g["elt_bytes"]),
                        int(g["context_tokens"]))
    assert kv == 32640 * 131072
    t = cm.transfer_time(kv, float(g["bandwidth_bytes_per_sec"]), float(g["network_latency_sec"]))
    assert round(t + float(g["resume_overhead_sec"]), int(g["printed_digits"])) == float(g["printed_ttft_sec"])
    # the two terms, separately: a wrong operand order or a dropped term fails one of these
    assert cm.transfer_time(kv, float(g["bandwidth_bytes_per_sec"]), 0.0) == kv / 25e9
    assert cm.transfer_time(0, 1.0, 7.5) == 7.5
    assert cm.transfer_time(10.0, 4.0, 0.25) == 2.75


def test_policy_is_the_strict_comparison_of_the_scheduling_rule():
    assert cm.policy(True, 9.0, 1.0) == cm.REUSE  # local and compatible: reuse, whatever the times
    assert cm.policy(False, 1.0, 2.0) == cm.TRANSFER
    assert cm.policy(False, 2.0, 1.0) == cm.RECOMPUTE
    assert cm.policy(False, 1.0, 1.0) == cm.RECOMPUTE  # "transfer if T_transfer < T_prefill", otherwise recompute


def test_packed_time_against_hand_computed_values():
    g = _read(os.path.join(GOLD, "packed_transfer_example.txt"))
    kv, bw = float(g["kv_bytes"]), float(g["bandwidth_bytes_per_sec"])
    lat, rate = float(g["latency_sec"]), float(g["pack_rate_bytes_per_sec"])
    for f_t, f_p in ((cm.transfer_time, cm.transfer_time_packed),
                     (binding.aaf_kv_transfer_time, binding.aaf_kv_transfer_time_packed)):
        assert f_t(kv, bw, lat) == float(g["t_transfer_sec"])       # exact: powers of two
        assert f_p(kv, bw, lat, rate) == float(g["t_packed_sec"])
        t = f_p(float(g["paper_kv_bytes"]), 25e9, 50e-6, float(g["paper_pack_rate"])) * 1e3
        assert round(t, int(g["paper_t_packed_digits"])) == float(g["paper_t_packed_ms"])
        # halving the pack rate adds exactly one more pack + unpack; an infinitely fast pack leaves T_transfer
        assert f_p(kv, bw, lat, rate / 2) == 5.5
    assert cm.transfer_time_packed(kv, bw, lat, math.inf) == 4.5


def test_packed_time_is_wire_time_plus_a_pack_and_an_unpack():
    kv, bw, lat, rate = 4.0e9, 25e9, 50e-6, 6.4e12
    t = cm.transfer_time_packed(kv, bw, lat, rate)
    assert t == pytest.approx(cm.transfer_time(kv, bw, lat) + 2 * (2 * kv / rate), rel=1e-15)
    assert cm.transfer_time_packed(kv, bw, lat, math.inf) == cm.transfer_time(kv, bw, lat)


def test_library_matches_the_oracle_on_the_papers_network_grid():
    g = _read(os.path.join(GOLD, "exp3_network_grid.txt"))
    for tokens in map(int, g["max_context_tokens"].split()):
        kv = binding.aaf_kv_state_bytes(32, 8, 128, 2, tokens)
        assert kv == cm.state_bytes(32, 8, 128, 2, tokens) == tokens * 131072
        for gbps in map(float, g["bandwidth_gbps"].split()):
            for us in map(float, g["latency_us"].split()):
                bw, lat = gbps * 1e9 / 8.0, us * 1e-6
                assert binding.aaf_kv_transfer_time(kv, bw, lat) == cm.transfer_time(kv, bw, lat)
                for rate in (6.0e12, 6.5e12):
                    assert binding.aaf_kv_transfer_time_packed(kv, bw, lat, rate) == \
                        cm.transfer_time_packed(kv, bw, lat, rate)
    g2 = _read(os.path.join(GOLD, "transfer_time_max_context.txt"))
    t = binding.aaf_kv_transfer_time(binding.aaf_kv_state_bytes(32, 8, 128, 2, 32640), 25e9, 50e-6)
    assert round(t + 1e-4, 3) == float(g2["printed_ttft_sec"])


def test_library_matches_the_oracle_on_random_inputs_and_rejects_bad_ones():
    rng = np.random.default_rng(3)
    for _ in range(2000):
        kv, bw = float(rng.integers(1, 1 << 40)), float(10 ** rng.uniform(8, 12))
        lat, rate = float(10 ** rng.uniform(-6, -3)), float(10 ** rng.uniform(11, 13))
        tp = float(10 ** rng.uniform(-4, 1))
        t = cm.transfer_time(kv, bw, lat)
        assert binding.aaf_kv_transfer_time(kv, bw, lat) == t
        assert binding.aaf_kv_transfer_time_packed(kv, bw, lat, rate) == cm.transfer_time_packed(kv, bw, lat, rate)
        for local in (False, True):
            assert binding.aaf_kv_policy(local, t, tp) == cm.policy(local, t, tp)
    assert binding.aaf_kv_policy(False, 1.0, 1.0) == binding.AAF_POLICY_RECOMPUTE
    assert binding.aaf_kv_policy(False, float("nan"), 1.0) == binding.AAF_POLICY_RECOMPUTE
    assert math.isnan(binding.aaf_kv_transfer_time(-1.0, 1.0, 0.0))
    assert math.isnan(binding.aaf_kv_transfer_time(1.0, 0.0, 0.0))
    assert math.isnan(binding.aaf_kv_transfer_time(1.0, 1.0, -1.0))
    assert math.isnan(binding.aaf_kv_transfer_time_packed(1.0, 1.0, 0.0, 0.0))
    assert binding.aaf_kv_state_bytes(0, 8, 128, 2, 1) == -1
    assert binding.aaf_kv_state_bytes(1 << 30, 1 << 30, 1 << 30, 2, 1 << 40) == -1  # overflow


def test_transfer_never_stops_winning_as_bandwidth_grows():
    """The pattern of the paper's transfer-versus-recompute table (5/8 contexts at 10 Gbps, 8/8 from 25 Gbps on):
    with the other quantities fixed, the set of contexts for which pi(S) = transfer only grows with bandwidth."""
    g = _read(os.path.join(GOLD, "exp3_network_grid.txt"))
    for key in ("beneficial_mistral", "beneficial_llama3"):
        counts = [int(x) for x in g[key].split()]
        assert counts == sorted(counts)
    rng = np.random.default_rng(9)
    bws = [float(x) * 1e9 / 8 for x in g["bandwidth_gbps"].split()]
    for _ in range(300):
        kv, lat, tp = float(rng.integers(1 << 20, 1 << 33)), float(rng.choice([10e-6, 100e-6])), float(10 ** rng.uniform(-3, 1))
        wins = [cm.policy(False, cm.transfer_time(kv, bw, lat), tp) == cm.TRANSFER for bw in bws]
        assert wins == sorted(wins)
        times = [cm.transfer_time(kv, bw, lat) for bw in bws]
        assert times == sorted(times, reverse=True) and all(t > lat for t in times)
