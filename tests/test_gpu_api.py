"""C-ABI behaviour on a device: host-buffer entry points, descriptor compatibility, argument checks,
statistics, engine selection.  Results are compared with the CPU oracle where bytes are involved."""
from __future__ import annotations

import ctypes as C

import numpy as np
import pytest
import torch

from paper_2607_10987_b200 import KVPool, binding
from tests.helpers import GpuBackend, OracleBackend
from workloads import configs, fill
from workloads.configs import Geometry

pytestmark = pytest.mark.gpu

G = Geometry(3, 4, 64, 16, 2, 256, 8, 64)  # row 512 B, run 8 KiB
SEED = 99


def test_host_buffer_forms_match_the_oracle():
    order = configs.free_order(SEED, G.n_blocks)
    gpu = GpuBackend(G, SEED, free_order=order)
    cpu = OracleBackend(G, SEED, free_order=order)
    n = 333
    payload = cpu.payload(SEED, 1, n)  # numpy uint8, full layers
    h_src = torch.from_numpy(payload.copy()).pin_memory()
    staging = torch.empty(n * G.bpt, dtype=torch.uint8, device=gpu.o.device)
    st, c = gpu.o.import_host(h_src, n, staging)
    assert st == 0
    st2, c2 = cpu.imp(payload, n)
    assert (st2, c2) == (0, c)
    assert gpu.snapshot() == cpu.snapshot()
    h_dst = torch.zeros(200 * G.bpt, dtype=torch.uint8).pin_memory()
    assert gpu.o.materialize_host(c, 100, 300, h_dst, staging) == 0
    torch.cuda.synchronize()
    st, want = cpu.materialize(c, 100, 300)
    assert np.array_equal(h_dst.numpy(), want)
    assert np.array_equal(gpu.pool_layers(range(G.n_layers)), cpu.o.pool_view())
    # too small host destination / staging
    small = torch.zeros(16, dtype=torch.uint8).pin_memory()
    assert gpu.o.materialize_host(c, 0, n, small, staging) == binding.AAF_ERR_DST_TOO_SMALL
    assert gpu.o.materialize_host(c, 0, n, h_src, staging[:1024]) == binding.AAF_ERR_DST_TOO_SMALL
    assert gpu.o.import_host(h_src, n, staging[:1024])[0] == binding.AAF_ERR_DST_TOO_SMALL
    assert gpu.snapshot() == cpu.snapshot()


def test_append_from_host_buffers_matches_the_oracle():
    """aaf_kv_append_host: continuation tokens uploaded from pinned host memory, copy-on-write included; two
    calls in a row reuse the same staging buffer (the second upload must wait for the first scatter)."""
    order = configs.free_order(SEED, G.n_blocks)
    gpu = GpuBackend(G, SEED, free_order=order)
    cpu = OracleBackend(G, SEED, free_order=order)
    n = 203  # 203 = 12 * 16 + 11: the tail block holds 11 rows and is shared after the fork
    for be in (gpu, cpu):
        st, root = be.imp(be.payload(SEED, 1, n), n)
        assert (st, root) == (0, 0)
        st, kids = be.fork(root, 3)
        assert st == 0 and kids == [1, 2, 3]
    staging = torch.empty(64 * G.bpt, dtype=torch.uint8, device=gpu.o.device)
    for rnd, n_new in enumerate(([7, 21, 1], [16, 5, 30])):
        payloads = [cpu.payload(SEED, 10 * rnd + 2 + i, k) for i, k in enumerate(n_new)]
        hosts = [torch.from_numpy(p.copy()).pin_memory() for p in payloads]
        assert gpu.o.append_host(kids, n_new, hosts, staging) == 0
        assert cpu.append(kids, n_new, payloads)[0] == 0
        assert gpu.snapshot() == cpu.snapshot()
    torch.cuda.synchronize()
    assert np.array_equal(gpu.pool_layers(range(G.n_layers)), cpu.o.pool_view())
    assert gpu.o.stats()["cow_count"] == cpu.o.stats()["cow_count"] == 3
    # argument checks: staging too small, a dead handle, a null host pointer
    hosts = [torch.zeros(G.bpt, dtype=torch.uint8).pin_memory() for _ in range(3)]
    assert gpu.o.append_host(kids, [1, 1, 1], hosts, staging[: 2 * G.bpt]) == binding.AAF_ERR_DST_TOO_SMALL
    assert gpu.o.append_host([7], [1], hosts[:1], staging) == binding.AAF_ERR_BAD_CTX
    assert gpu.snapshot() == cpu.snapshot() and gpu.o.sync_status() == 0


def test_incompatible_descriptor_is_refused_and_changes_nothing():
    gpu = GpuBackend(G, SEED)
    buf = gpu.payload(SEED, 1, 40)
    before = gpu.snapshot()
    for field, value in (("model_id", 7), ("config_hash", 7), ("n_layers", 2), ("head_dim", 32), ("elt_bytes", 4)):
        d = gpu.o.xfer_desc(40)
        setattr(d, field, value)
        assert gpu.o.imp(buf, 40, desc=d)[0] == binding.AAF_ERR_INCOMPAT, field
    d = gpu.o.xfer_desc(0)
    assert gpu.o.imp(buf, 0, desc=d)[0] == binding.AAF_ERR_INVALID_ARG
    assert gpu.snapshot() == before
    # the descriptor materialize fills in is accepted back by import (transfer round trip, positions carried)
    st, c = gpu.o.imp(buf, 40)
    out = torch.empty(30 * G.bpt, dtype=torch.uint8, device=gpu.o.device)
    xd = binding.aaf_kv_xfer_desc()
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert binding.aaf_kv_materialize(gpu.o.h, c, 5, 35, out.data_ptr(), out.numel(), C.byref(xd), stream) == 0
    assert (xd.pos_start, xd.n_tokens, xd.n_layers) == (5, 30, G.n_layers)
    assert gpu.o.imp(out, 30, desc=xd)[0] == 0


def test_pointer_and_range_checks():
    gpu = GpuBackend(G, SEED)
    buf = gpu.payload(SEED, 1, 40)
    st, c = gpu.o.imp(buf, 40)
    out = torch.empty(40 * G.bpt + 64, dtype=torch.uint8, device=gpu.o.device)
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    mis = out.data_ptr() + 8
    assert binding.aaf_kv_materialize(gpu.o.h, c, 0, 40, mis, 40 * G.bpt, None, stream) == binding.AAF_ERR_INVALID_ARG
    assert binding.aaf_kv_materialize(gpu.o.h, c, 0, 40, out.data_ptr(), 40 * G.bpt - 1, None, stream) == \
        binding.AAF_ERR_DST_TOO_SMALL
    assert gpu.o.materialize(c, 0, 41)[0] == binding.AAF_ERR_INVALID_ARG
    assert gpu.o.materialize(c, 7, 7)[0] == binding.AAF_ERR_INVALID_ARG
    assert gpu.o.materialize(5, 0, 1)[0] == binding.AAF_ERR_BAD_CTX
    d = gpu.o.xfer_desc(40)
    out_ctx = C.c_int32(-1)
    assert binding.aaf_kv_import(gpu.o.h, buf.data_ptr() + 4, C.byref(d), C.byref(out_ctx), stream) == \
        binding.AAF_ERR_INVALID_ARG
    assert gpu.o.set_copy_engine(9) == binding.AAF_ERR_INVALID_ARG
    assert gpu.o.fork(c, 0)[0] == binding.AAF_ERR_INVALID_ARG
    assert gpu.o.fork(c, 5000)[0] == binding.AAF_ERR_TOO_MANY
    assert gpu.o.sync_status() == 0


def test_out_of_blocks_is_exact_after_evictions_the_host_did_not_count():
    """The host only keeps a lower bound of the free count (evict does not raise it); a request the
    bound cannot prove must be decided against the device's real count, not refused."""
    g = Geometry(1, 1, 8, 4, 2, 16, 8, 16)
    gpu = GpuBackend(g, SEED)
    cpu = OracleBackend(g, SEED)
    mk = lambda be, s, n: be.payload(SEED, s, n)
    for be in (gpu, cpu):
        assert be.imp(mk(be, 1, 40), 40) == (0, 0)       # 10 blocks
        assert be.imp(mk(be, 2, 18), 18) == (0, 1)       # 5 blocks (tail half full) -> 1 free
        assert be.imp(mk(be, 3, 8), 8)[0] == binding.AAF_ERR_OOM_BLOCKS
        assert be.evict([0])[0] == 0                     # 11 free, the host's bound still says 1
        assert be.imp(mk(be, 4, 44), 44) == (0, 0)       # exactly 11 blocks: must succeed
        assert be.imp(mk(be, 5, 1), 1)[0] == binding.AAF_ERR_OOM_BLOCKS
        # append whose worst case (COW + 1) does not fit but whose real need (in place, 0 new blocks) does
        assert be.fork(1, 1) == (0, [2])
        assert be.evict([2])[0] == 0                     # tail of ctx 1 is unshared again
        assert be.append([1], [2], [mk(be, 6, 2)])[0] == 0  # 18 -> 20 tokens in place: the real need is 0 blocks
        assert be.append([1], [1], [mk(be, 7, 1)])[0] == binding.AAF_ERR_OOM_BLOCKS  # would need a 6th block
    assert gpu.snapshot() == cpu.snapshot()
    assert np.array_equal(gpu.pool_layers([0]), cpu.o.pool_view())


def test_stats_and_launch_counters():
    gpu = GpuBackend(G, SEED)
    gpu.o.set_timing(True)
    st, c = gpu.o.imp(gpu.payload(SEED, 1, 100), 100)
    gpu.o.materialize(c, 0, 100)
    kids = gpu.o.fork(c, 2)[1]
    gpu.o.append([kids[0]], [5], [gpu.payload(SEED, 2, 5)])
    s = gpu.o.stats()
    assert s["copy_launches"] == {"materialize": 1, "import": 1, "append": 1, "compose": 0}
    assert s["timed_launches"] == s["copy_launches"]
    assert all(v > 0 for k, v in s["copy_ms"].items() if k != "compose")
    assert s["meta_launches"] == 4 and s["cow_count"] == 1 and s["live_ctx"] == 3
    assert s["payload_bytes"] == (100 + 100 + 5 + 100 % 16) * G.bpt
    assert s["live_blocks"] == 7 + 1 and s["free_blocks"] == G.n_blocks - 8


def test_bounded_wait_expires_with_a_status_and_the_pool_keeps_working():
    """Failure detection without a fault: a device-side wait that nothing will ever satisfy gives up after
    its limit, records AAF_ERR_TIMEOUT, and the next operators run normally."""
    gpu = GpuBackend(G, SEED)
    cpu = OracleBackend(G, SEED)
    pay = lambda be: be.payload(SEED, 1, 50)
    assert gpu.imp(pay(gpu), 50) == cpu.imp(pay(cpu), 50) == (0, 0)
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert binding.aaf_kv_debug_expire_wait(gpu.o.h, 2_000_000, stream) == 0  # about a millisecond
    assert gpu.o.sync_status() == binding.AAF_ERR_TIMEOUT
    assert gpu.o.sync_status() == 0, "the status is sticky until read, then cleared"
    assert binding.aaf_kv_debug_expire_wait(gpu.o.h, 0, stream) == binding.AAF_ERR_INVALID_ARG
    for be in (gpu, cpu):
        assert be.fork(0, 2)[0] == 0
        assert be.append([1], [7], [be.payload(SEED, 2, 7)])[0] == 0
    st, got = gpu.materialize(1, 0, 57)
    st2, want = cpu.materialize(1, 0, 57)
    assert st == st2 == 0
    assert np.array_equal(gpu.buf_layers(got, 57, range(G.n_layers)).reshape(-1), want)
    assert gpu.snapshot() == cpu.snapshot() and gpu.o.sync_status() == 0


@pytest.mark.parametrize("chunk_tokens", [16, 32, 160, 4096])
def test_chunked_host_transfer_is_byte_identical_and_flags_every_chunk(chunk_tokens):
    order = configs.free_order(SEED, G.n_blocks)
    gpu = GpuBackend(G, SEED, free_order=order)
    cpu = OracleBackend(G, SEED, free_order=order)
    n = 333
    payload = cpu.payload(SEED, 1, n)
    h_src = torch.from_numpy(payload.copy()).pin_memory()
    staging = torch.empty(n * G.bpt, dtype=torch.uint8, device=gpu.o.device)
    # chunked import: H2D of chunk c+1 overlaps the scatter of chunk c
    st, c = gpu.o.import_host_chunked(h_src, n, staging, chunk_tokens)
    assert (st, c) == (0, 0) and cpu.imp(payload, n) == (0, 0)
    assert gpu.snapshot() == cpu.snapshot()
    assert np.array_equal(gpu.pool_layers(range(G.n_layers)), cpu.o.pool_view())
    # chunked materialize of an unaligned range, one completion flag per chunk
    t0, t1 = 37, 300
    h_dst = torch.zeros((t1 - t0) * G.bpt, dtype=torch.uint8).pin_memory()
    flags = torch.full((64,), 7, dtype=torch.int32).pin_memory()
    st, n_chunks = gpu.o.materialize_host_chunked(c, t0, t1, h_dst, staging, chunk_tokens, flags)
    assert st == 0
    blocks = (t1 - 1) // 16 - t0 // 16 + 1
    assert n_chunks == -(-blocks // (chunk_tokens // 16))
    torch.cuda.synchronize()
    assert flags[:n_chunks].tolist() == [1] * n_chunks and flags[n_chunks:].tolist() == [7] * (64 - n_chunks)
    assert np.array_equal(h_dst.numpy(), cpu.materialize(c, t0, t1)[1])
    # argument checks
    assert gpu.o.materialize_host_chunked(c, t0, t1, h_dst, staging, 24, flags)[0] == binding.AAF_ERR_INVALID_ARG
    assert gpu.o.materialize_host_chunked(c, t0, t1, h_dst, staging, 16, flags[:3])[0] == binding.AAF_ERR_DST_TOO_SMALL
    assert gpu.o.import_host_chunked(h_src, n, staging, 0)[0] == binding.AAF_ERR_INVALID_ARG
    assert gpu.snapshot() == cpu.snapshot() and gpu.o.sync_status() == 0


def test_calls_on_alternating_streams_do_not_overlap_their_copy_launches():
    """Data-independent operators of one pool issued to two streams without any ordering by the caller: the
    library serialises their copy launches (they share the pool's work counter), so every byte still arrives."""
    g = Geometry(4, 8, 128, 16, 2, 1024, 32, 64)  # 2 KiB rows, 32 KiB runs: the bulk engine
    order = configs.free_order(SEED, g.n_blocks)
    gpu = GpuBackend(g, SEED, free_order=order, init_fill=False)
    cpu = OracleBackend(g, SEED, free_order=order, init_fill=False)
    gpu.o.pool.zero_()
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(gpu.o.device), torch.cuda.Stream(gpu.o.device)]
    lens = [600 + 37 * i for i in range(12)]
    bufs = [gpu.payload(SEED, 1 + i, n) for i, n in enumerate(lens)]
    torch.cuda.synchronize()
    for i, n in enumerate(lens):
        with torch.cuda.stream(streams[i % 2]):
            st, c = gpu.imp(bufs[i], n)
        assert (st, c) == (0, i)
        assert cpu.imp(cpu.payload(SEED, 1 + i, n), n) == (0, i)
    torch.cuda.synchronize()
    assert gpu.snapshot() == cpu.snapshot()
    assert np.array_equal(gpu.pool_layers(range(g.n_layers)), cpu.o.pool_view())
    assert gpu.o.sync_status() == 0


def test_a_pool_marked_unusable_refuses_every_operator_and_changes_nothing():
    """The documented exception to "an error changes nothing": after a CUDA failure inside an operator the pool
    refuses all further work.  The state is entered here through the test hook, without any failure."""
    gpu = GpuBackend(G, SEED)
    o = gpu.o
    buf = gpu.payload(SEED, 1, 40)
    st, c = o.imp(buf, 40)
    assert st == 0
    before = gpu.snapshot()
    assert binding.aaf_kv_debug_mark_unusable(o.h) == 0
    out = torch.empty(40 * G.bpt, dtype=torch.uint8, device=o.device)
    host = torch.empty(40 * G.bpt, dtype=torch.uint8).pin_memory()
    E = binding.AAF_ERR_CUDA
    assert o.materialize(c, 0, 40, out=out)[0] == E and o.imp(buf, 40)[0] == E and o.fork(c, 1)[0] == E
    assert o.append([c], [40], [buf])[0] == E and o.compose([c, c])[0] == E and o.evict([c])[0] == E
    assert o.compose_batch([[c], [c]])[0] == E and o.materialize_batch([c], [0], [40], [out]) == E
    assert o.import_batch([buf], [40])[0] == E and o.append_host([c], [40], [host], out) == E
    assert o.materialize_host(c, 0, 40, host, out) == E and o.import_host(host, 40, out)[0] == E
    assert o.materialize_host_chunked(c, 0, 40, host, out, 16)[0] == E and o.import_host_chunked(host, 40, out, 16)[0] == E
    assert o.evict_to_budget(0.0, 0.0, 1.0, 0)[0] == E
    assert gpu.snapshot() == before and o.sync_status() == 0  # introspection still answers; nothing changed
    o.close()


def test_two_pools_of_different_geometry_interleaved():
    """Launch shapes and scratch are per pool: two pools with different rows, block sizes and engines,
    used alternately on the same stream, each stay bit-exact against their own oracle."""
    ga = Geometry(2, 8, 128, 16, 2, 128, 8, 64)   # 2 KiB rows, 32 KiB runs
    gb = Geometry(3, 1, 8, 5, 2, 160, 8, 64)      # 16-byte rows, 80-byte runs
    pairs = []
    for g, seed, engine in ((ga, 11, 0), (gb, 12, 0)):
        order = configs.free_order(seed, g.n_blocks)
        pairs.append((g, seed, GpuBackend(g, seed, free_order=order, engine=engine),
                      OracleBackend(g, seed, free_order=order)))
    script = [("imp", 70), ("fork", 2), ("append", 9), ("compose", None), ("mat", None), ("evict", None), ("imp", 33)]
    for step, arg in script:
        for g, seed, gpu, cpu in pairs:  # alternate pools at every operator
            for be in (gpu, cpu):
                if step == "imp":
                    assert be.imp(be.payload(seed, 1 + arg, arg), arg)[0] == 0
                elif step == "fork":
                    assert be.fork(0, arg)[0] == 0
                elif step == "append":
                    assert be.append([1, 2], [arg, arg + 1], [be.payload(seed, 5, arg), be.payload(seed, 6, arg + 1)])[0] == 0
                elif step == "compose":
                    assert be.compose([1, 0, 2], 0)[0] == 0
                elif step == "evict":
                    assert be.evict([0, 2])[0] == 0
            if step == "mat":
                n = cpu.o.ctx_len(3)
                sg, bg = gpu.materialize(3, 0, n)
                sc, bc = cpu.materialize(3, 0, n)
                assert sg == sc == 0
                assert np.array_equal(gpu.buf_layers(bg, n, range(g.n_layers)).reshape(-1), bc)
    for g, seed, gpu, cpu in pairs:
        assert gpu.snapshot() == cpu.snapshot()
        assert np.array_equal(gpu.pool_layers(range(g.n_layers)), cpu.o.pool_view())
        assert gpu.o.sync_status() == 0


def test_bench_prints_one_json_line_with_the_contract_keys():
    import json
    import os
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--workload", "tiny", "--steps", "5",
                          "--warmup", "3"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert k in d, k
    assert d["n_gpus"] == 1 and d["steps"] == 5 and d["warmup"] == 3 and d["scaling"] == "weak"
    assert d["vs_baseline"] is None and d["dtype"] == "u8" and d["data"] == "synthetic" and "workload" in d["config"]
    assert d["gpu_launches"] == 5 * 12
    assert set(d["e2e"]) >= {"value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"}
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert set(d["cpu_baseline"]) >= {"value", "unit", "cores", "kind", "sample"} and d["cpu_baseline"]["kind"] == "oracle"
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert d["repeats"] >= 1 and d["timed_seconds"] > 0 and "traffic_source" in r
    assert set(d["e2e"]) >= {"pcie_floor_ms_per_step", "frac_of_pcie_floor", "api"}


def test_default_bench_line_carries_the_other_full_size_workloads():
    """The headline run also measures the 70B-shaped step, the composition levels and the copy-on-write stress and
    attaches them as roofline.per_workload (short timed regions here; the keys and the sanity of the figures)."""
    import json
    import os
    import subprocess
    import sys

    free_b, _ = torch.cuda.mem_get_info()
    if free_b < (80 << 30):
        pytest.skip("not enough free device memory for the full-size pools")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--steps", "3", "--warmup", "3",
                          "--min-seconds", "0.05", "--no-e2e", "--no-cpu-baseline"], capture_output=True, text=True,
                         timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads([l for l in out.stdout.splitlines() if l.strip()][-1])
    assert d["config"]["n_blocks"] == 32768 and d["gpu_launches"] == 3 * 12
    pw = d["roofline"]["per_workload"]
    assert set(pw) == {"70b", "compose_pairs", "compose_quads", "compose_all16", "compose_flat16", "cow", "cow_70b",
                       "suffix_pack_loop", "suffix_pack_batch", "suffix_unpack_loop", "suffix_unpack_batch"}
    for name, rec in pw.items():
        assert set(rec) >= {"achieved", "frac", "algorithmic_bytes_per_launch", "mean_launch_ms", "launches"}, name
        assert 0.5 < rec["frac"] < 1.2 and rec["launches"] > 0, (name, rec["frac"])
        assert abs(rec["achieved"] - rec["frac"] * d["roofline"]["peak"]) < 1e-6 * rec["achieved"]
    assert "frac_of_measured_peak" not in pw["cow"] and pw["cow"]["counted_read_plus_written_GBps"] > pw["cow"]["achieved"]
