#!/usr/bin/env python
"""Benchmark of the paged-KV operator path on B200 (one JSON line on stdout).

A step is one pass of the whole operator path over one batch of synthetic input, on the
Llama-3-8B-shaped workload (32 layers, 8 KV heads, head_dim 128, block 16, bf16; pool of 32768
blocks with a seeded-permuted free list), in its unaligned variant so that copy-on-write and the
re-packing compose really copy:

    import 8187-token context -> materialize to a transfer buffer -> import that buffer ->
    fork to 16 agents -> one batched append of 16 x 512 tokens (each agent copies the shared
    partial tail on write) -> compose(agent0, agent1) -> evict everything

metric  = KV bytes moved (read + written) per second, whole job, inputs resident in HBM.
e2e     = the same step with the step's inputs copied from pinned host memory and the
          materialised transfer buffer copied back to the host inside the timed region.
roofline= the copy kernel (the one kernel every operator's bytes go through): algorithmic bytes
          per launch / its mean launch time from CUDA events recorded by the library on the
          launching stream, against the measured HBM copy peak.  roofline.per_workload carries
          the same figures for the other full-size workloads, measured in the same run after the
          headline step: the Llama-3-70B-shaped step, the composition levels (pairs / quads /
          all 16) and the copy-on-write stress (1024 children of one unaligned context).
cpu_baseline = the CPU oracle (plain single-threaded C) timed on a bounded sample of the same step.

The timed region is `--steps` steps between a barrier + synchronize on both sides; it is repeated
(`repeats` in the JSON line) until at least a second of device time has been measured, and the
reported time per step is the mean over all repeats.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 8b|70b|tiny]
N > 1 runs independent replicas (the path has no exchange step): launch with torch.distributed.run.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from workloads import configs, fill  # noqa: E402

METRIC = "kv_bytes_moved_GBps"
UNIT = "GB/s"

# DRAM traffic of a copy launch, modelled from a one-pass capture of the two DRAM byte counters: reads equal the
# algorithmic bytes read; writes fall short of the algorithmic bytes written by the dirty lines that are still in
# the L2 when the kernel ends (a fixed residue per launch, independent of the launch size)
L2_DIRTY_RESIDUE_BYTES = 48e6


def workload(name: str):
    if name == "8b":
        g = configs.LLAMA8B
        return dict(name="llama3-8b-shaped KV, 8187-token context, 16 agents x 512 tokens, unaligned (COW)", g=g,
                    seed=configs.SEED_BASE + 2, T=8187, agents=16, n_new=512)
    if name == "8b-aligned":  # the literal block-aligned variant: no copy-on-write, the compose is table-only
        g = configs.LLAMA8B
        return dict(name="llama3-8b-shaped KV, 8192-token context, 16 agents x 512 tokens, block-aligned", g=g,
                    seed=configs.SEED_BASE + 2, T=8192, agents=16, n_new=512)
    if name == "70b":
        g = configs.LLAMA70B
        return dict(name="llama3-70b-shaped KV, 32763-token context, 8 agents x 1024 tokens, unaligned (COW)", g=g,
                    seed=configs.SEED_BASE + 4, T=32763, agents=8, n_new=1024)
    if name == "8b-small":  # same rows and runs as "8b" on a pool small enough for a full ncu capture
        g = configs.Geometry(32, 8, 128, 16, 2, 2048, 16, 512)
        return dict(name="llama3-8b-shaped KV rows, 2043-token context, 4 agents x 128 tokens, 2048-block pool", g=g,
                    seed=configs.SEED_BASE + 2, T=2043, agents=4, n_new=128)
    if name == "tiny":
        g = configs.TINY
        return dict(name="tiny pool, 507-token context, 4 agents x 64 tokens", g=g, seed=configs.SEED_BASE + 1,
                    T=507, agents=4, n_new=64)
    raise SystemExit(f"unknown workload {name}")


def step_config(w, n_blocks, engine):
    """`config` of the JSON line: the same dict on both arms (the closed-form byte count needs no device)."""
    g = w["g"]
    moved = 2 * sum(class_tokens(g, w["T"], w["agents"], w["n_new"]).values()) * g.bpt
    return {"workload": w["name"], "n_blocks": n_blocks, "pool_GiB": g.n_layers * n_blocks * 2 * g.run / 2**30,
            "l2_policy": ("inputs_exceed_l2 (each operator streams %.1f GiB or more)" % (w["T"] * g.bpt / 2**30)
                          if w["T"] * g.bpt > (256 << 20) else "none: smaller than the L2, a test shape, not a bench line"),
            "parallelism": "replicas only",
            "engine": engine, "moved_GB_per_step": moved / 1e9}


def class_tokens(g, T, agents, n_new):
    """Tokens each operator class copies in one step (closed form of the step above)."""
    r = T % g.block_size
    la = T + n_new  # length of an agent after the append
    rem = la % g.block_size
    return {"materialize": T, "import": 2 * T, "append": agents * (n_new + r), "compose": (rem + la) if rem else 0}


def step_ops(backend, root_buf, agent_bufs, T, agents, n_new, staging):
    """One pass of the whole path on any backend with the KVPool method names. Returns #operators."""
    st, root = backend.imp(root_buf, T)
    assert st == 0, st
    st, xfer = backend.materialize(root, 0, T, staging) if staging is not None else backend.materialize(root, 0, T)
    assert st == 0, st
    st, recv = backend.imp(xfer, T)
    assert st == 0, st
    st, kids = backend.fork(recv, agents)
    assert st == 0, st
    st, _ = backend.append(kids, [n_new] * agents, agent_bufs)
    assert st == 0, st
    st, merged = backend.compose(kids[:2], 0)
    assert st == 0, st
    st, _ = backend.evict([root, recv] + kids + [merged])
    assert st == 0, st
    return 7


# ------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: str):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        self.f.close()
        os.unlink(self.f.name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------- CPU oracle arm
def oracle_rate(w, layers_sample: int, budget_s: float, max_steps: int, warm_steps: int = 1):
    """Times the CPU oracle, as it stands, on the same step restricted to `layers_sample` layers."""
    from oracle import paged

    g = w["g"]
    paged.build()
    o = paged.PagedOracle(layers_sample, g.n_kv_heads, g.head_dim, g.block_size, g.elt_bytes, g.n_blocks, g.max_ctx,
                          g.max_blocks_per_ctx, configs.free_order(w["seed"], g.n_blocks))
    per_layer = lambda n: 2 * n * g.row // 2
    root = np.concatenate([fill.fill_np(w["seed"], 1, l * per_layer(w["T"]), per_layer(w["T"]))
                           for l in range(layers_sample)]).view(np.uint8)
    bufs = [np.concatenate([fill.fill_np(w["seed"], 2 + i, l * per_layer(w["n_new"]), per_layer(w["n_new"]))
                            for l in range(layers_sample)]).view(np.uint8) for i in range(w["agents"])]

    class B:  # adapter: the oracle's materialize allocates its own output
        imp, fork, append, evict = o.imp, o.fork, o.append, o.evict
        compose = staticmethod(lambda segs, fl: o.compose(segs, fl))
        materialize = staticmethod(lambda c, a, b: o.materialize(c, a, b))

    for _ in range(max(warm_steps, 1)):  # warm-up (page faults of the pool)
        step_ops(B, root, bufs, w["T"], w["agents"], w["n_new"], None)
    rows0 = o.stats()["rows_copied"]
    t0 = time.perf_counter()
    steps = 0
    while steps < max_steps and (steps == 0 or time.perf_counter() - t0 < budget_s):
        step_ops(B, root, bufs, w["T"], w["agents"], w["n_new"], None)
        steps += 1
    dt = time.perf_counter() - t0
    moved = 2 * (o.stats()["rows_copied"] - rows0) * g.row
    return moved / dt / 1e9, steps, dt, 7 * steps / dt


def reference_arm(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    layers = 2 if w["g"].n_layers > 2 else w["g"].n_layers
    # `steps` timed passes, each a bounded sample of the workload (a subset of the layers)
    warm = max(args.warmup, 3)
    gbps, steps, dt, ops_s = oracle_rate(w, layers, budget_s=1e9, max_steps=max(args.steps, 1), warm_steps=warm)
    cores = 1
    sample = f"{layers} of {w['g'].n_layers} layers of the step, {steps} passes, single thread"
    line = {
        "impl": "reference", "metric": METRIC, "value": gbps, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": step_config(w, w["g"].n_blocks, args.engine),
        "cpu_baseline": {"value": gbps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "ops_per_s": ops_s,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------- shared helpers
def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback"


def kernel_record(bytes_rw, copy_ms, launches, peak):
    """Roofline figures of the copy kernel over a set of launches: bytes_rw = algorithmic bytes read + written."""
    if launches == 0 or copy_ms <= 0:
        return None
    ach = bytes_rw / (copy_ms * 1e-3) / 1e9
    per_launch = bytes_rw / launches
    return {"achieved": ach, "unit": "GB/s", "frac": ach / peak, "frac_of_nominal_8TBps": ach / 8000.0,
            "algorithmic_bytes_per_launch": per_launch, "mean_launch_ms": copy_ms / launches, "launches": launches,
            "traffic": max(per_launch - L2_DIRTY_RESIDUE_BYTES, per_launch / 2),
            "traffic_source": "modelled: algorithmic bytes minus the dirty-L2 residue of a one-pass DRAM-counter capture"}


def timed_ops(pool, fn, meta=False):
    """Runs fn with the library's kernel timing on; returns (ms on the stream, per-class kernel ms, per-class
    launches, bytes one way).  meta=True: fn is a metadata-only operator, which runs on the library's own stream;
    the host then waits for both of the library's streams before the closing event, so ms is the call's wall time."""
    import torch

    s0 = pool.stats()
    pool.set_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    fn()
    if meta:
        pool.sync_status()
    e1.record()
    torch.cuda.synchronize()
    pool.set_timing(False)
    s1 = pool.stats()
    dms = {k: s1["copy_ms"][k] - s0["copy_ms"][k] for k in s1["copy_ms"]}
    dl = {k: s1["timed_launches"][k] - s0["timed_launches"][k] for k in s1["timed_launches"]}
    return e0.elapsed_time(e1), dms, dl, s1["payload_bytes"] - s0["payload_bytes"]


def cow_stress(args, peak, steps, warmup, n_layers=32):
    """Copy-on-write stress: one unaligned 8187-token context forked to 1024 children, one batched 1-token append,
    so 1024 children each copy the 11 valid rows of the shared partial tail block.  All children read the same
    11 source rows (they stay in the L2), so the DRAM side of this kernel is its writes.  n_layers = 32: the
    8B-shaped rows; 80: the 70B-shaped ones."""
    from tests.gpu_backend import GpuBackend

    g = configs.Geometry(n_layers, 8, 128, 16, 2, 2048 if n_layers > 32 else 4096, 1100, 1024)
    seed = configs.SEED_BASE + 6
    be = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), engine=args.engine, init_fill=False,
                    max_batch=1024)
    T, kids_n = 8187, 1024
    root_buf = be.payload(seed, 1, T)
    eight = [be.payload(seed, 2 + i, 1) for i in range(8)]
    one = [eight[i % 8] for i in range(kids_n)]
    acc = {"append_ms": 0.0, "append_bytes": 0, "launches": 0, "fork_ms": 0.0, "evict_ms": 0.0}
    for it in range(warmup + steps):
        st, root = be.imp(root_buf, T)
        res = {}
        ms_f, _, _, _ = timed_ops(be.o, lambda: res.update(r=be.fork(root, kids_n)), meta=True)
        kids = res["r"][1]
        ms_a, dms, dl, b = timed_ops(be.o, lambda: res.update(a=be.append(kids, [1] * kids_n, one)[0]))
        assert res["a"] == 0
        ms_e, _, _, _ = timed_ops(be.o, lambda: res.update(e=(be.evict(kids)[0], be.evict([root])[0])), meta=True)
        assert res["r"][0] == 0 and res["e"] == (0, 0), res
        if it >= warmup:
            acc["append_ms"] += dms["append"]; acc["append_bytes"] += b; acc["launches"] += dl["append"]
            acc["fork_ms"] += ms_f; acc["evict_ms"] += ms_e
    assert be.o.sync_status() == 0 and be.o.stats()["cow_count"] == kids_n * (warmup + steps)
    # the same at the fan-out of the workload configs (16 agents at the 8B shape, 8 at the 70B shape): a copy of a
    # few tens of MiB, i.e. a latency figure: kernel time and time of the whole call on an idle stream
    few = 16 if n_layers <= 32 else 8
    lat = {"kernel_ms": 0.0, "call_ms": 0.0}
    for it in range(warmup + steps):
        st, root = be.imp(root_buf, T)
        st, kids = be.fork(root, few)
        ms_a, dms, dl, b = timed_ops(be.o, lambda: be.append(kids, [1] * few, one[:few]))
        be.evict(kids + [root])
        if it >= warmup:
            lat["kernel_ms"] += dms["append"] / steps; lat["call_ms"] += ms_a / steps
    lat.update({"agents": few, "bytes_copied_MiB": b / 2**20})
    rec = kernel_record(2 * acc["append_bytes"], acc["append_ms"], acc["launches"], peak)
    written = acc["append_bytes"] / (acc["append_ms"] * 1e-3) / 1e9
    # the counted rate (read + written) exceeds the DRAM peak because the reads are L2 hits: the figure to hold
    # against the HBM roofline is the write side
    rec.update({"counted_read_plus_written_GBps": rec.pop("achieved"), "achieved": written, "frac": written / peak,
                "frac_of_nominal_8TBps": written / 8000.0, "traffic": rec["algorithmic_bytes_per_launch"] / 2,
                "traffic_source": "modelled: the bytes written (the 11 shared source rows are read from the L2)",
                "note": "achieved = bytes written per second (DRAM side); the 1024 children read the same 11 rows",
                "children": kids_n, "rows_copied_per_child": T % g.block_size, "n_layers": n_layers,
                "fork_1024_ms": acc["fork_ms"] / steps, "evict_1024_plus_1_ctx_ms": acc["evict_ms"] / steps,
                "first_append_of_the_config_fanout": lat})
    del be
    return rec


def suffix_transfers(args, peak, steps, warmup):
    """Partial transfers (Sec. 5.4: only the subset of a state that a consumer needs is sent): 16 agents share an
    8187-token prefix that the receiver already holds, so only each agent's 512-token continuation is packed, and
    unpacked at the other end.  Sixteen 64 MiB transfers, issued one call each and as ONE batched call."""
    import torch

    from tests.gpu_backend import GpuBackend

    g = configs.Geometry(32, 8, 128, 16, 2, 8192, 64, 1024)
    seed, T, agents, n_new = configs.SEED_BASE + 2, 8187, 16, 512
    be = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), engine=args.engine, init_fill=False)
    pool = be.o
    st, root = be.imp(be.payload(seed, 1, T), T)
    st, kids = be.fork(root, agents)
    assert be.append(kids, [n_new] * agents, [be.payload(seed, 2 + i, n_new) for i in range(agents)])[0] == 0
    bufs = [torch.empty(n_new * g.bpt, dtype=torch.uint8, device=pool.device) for _ in range(agents)]
    acc = {k: {"ms": 0.0, "kernel_ms": 0.0, "bytes": 0, "launches": 0} for k in
           ("pack_loop", "pack_batch", "unpack_loop", "unpack_batch")}

    def note(key, r):
        ms, dms, dl, b = r
        a = acc[key]
        a["ms"] += ms; a["kernel_ms"] += sum(dms.values()); a["bytes"] += b; a["launches"] += sum(dl.values())

    for it in range(warmup + steps):
        res = {}
        r1 = timed_ops(pool, lambda: [pool.materialize(k, T, T + n_new, out=b) for k, b in zip(kids, bufs)])
        r2 = timed_ops(pool, lambda: res.update(m=pool.materialize_batch(kids, [T] * agents, [T + n_new] * agents, bufs)))
        assert res["m"] == 0
        got = []
        r3 = timed_ops(pool, lambda: got.extend(pool.imp(b, n_new)[1] for b in bufs))
        pool.evict(got)
        r4 = timed_ops(pool, lambda: res.update(i=pool.import_batch(bufs, [n_new] * agents)))
        assert res["i"][0] == 0
        pool.evict(res["i"][1])
        if it >= warmup:
            for key, r in (("pack_loop", r1), ("pack_batch", r2), ("unpack_loop", r3), ("unpack_batch", r4)):
                note(key, r)
    assert pool.sync_status() == 0
    out = {"transfers": agents, "tokens_each": n_new, "bytes_each_MiB": n_new * g.bpt / 2**20}
    for key, a in acc.items():
        rec = kernel_record(2 * a["bytes"], a["kernel_ms"], a["launches"], peak)
        rec.update({"launches_per_pass": a["launches"] / steps,
                    "whole_pass_GBps": 2 * a["bytes"] / (a["ms"] * 1e-3) / 1e9,
                    "whole_pass_note": "events around the 16 calls (or the one batched call), host latency included"})
        out[key] = rec
    del be
    torch.cuda.empty_cache()
    return out


def compose_levels(args, peak, steps, warmup, copy_all=False):
    """Composition workload: 16 contexts of 1024..4096 tokens (none block-aligned) composed in pairs, quads, all 16
    (tree) and flat.  Per level: the copy kernel's rate from the library's events, and the level's throughput with
    all of the level's composes issued back to back (CUDA events around the level, no per-kernel events)."""
    import torch

    from tests.gpu_backend import GpuBackend

    g, seed, ops, lens = configs.config3(configs.LLAMA8B, copy_all=copy_all)
    free_b, _ = torch.cuda.mem_get_info()
    while g.pool_bytes + (6 << 30) > free_b and g.n_blocks > 8192:
        g = configs.Geometry(g.n_layers, g.n_kv_heads, g.head_dim, g.block_size, g.elt_bytes, g.n_blocks // 2,
                             g.max_ctx, g.max_blocks_per_ctx)
    be = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), engine=args.engine, init_fill=False)
    names = {}
    for o in (o for o in ops if o["op"] == "import"):
        st, c = be.imp(be.payload(seed, o["stream"], o["n"]), o["n"])
        assert st == 0
        names[o["out"]] = c
    by_level = {}
    for o in (o for o in ops if o["op"] == "compose"):
        by_level.setdefault(o["level"], []).append(o)
    acc = {k: {"ms": 0.0, "kernel_ms": 0.0, "launches": 0, "bytes": 0, "ops": 0, "b2b_ms": 0.0, "b2b_bytes": 0,
               "bat_ms": 0.0, "bat_kernel_ms": 0.0, "bat_bytes": 0, "bat_launches": 0}
           for k in by_level}

    def run_level(level, made):
        for o in by_level[level]:
            st, c = be.compose([names[x] for x in o["segs"]], o["flags"])
            assert st == 0
            names[o["out"]] = c
            made.append(c)

    def run_level_batched(level, made):  # the whole level as ONE call: one planner launch, one copy launch
        st, outs = be.o.compose_batch([[names[x] for x in o["segs"]] for o in by_level[level]],
                                      by_level[level][0]["flags"])
        assert st == 0
        for o, c in zip(by_level[level], outs):
            names[o["out"]] = c
        made += outs

    for it in range(warmup + 3 * steps):
        made = []
        kernel_pass = it < warmup + steps  # first the per-kernel events, then the back-to-back levels, then batches
        batched_pass = it >= warmup + 2 * steps
        for level in by_level:
            if batched_pass:
                ms, dms, dl, b = timed_ops(be.o, lambda: run_level_batched(level, made))
                a = acc[level]
                a["bat_ms"] += ms; a["bat_kernel_ms"] += dms["compose"]; a["bat_bytes"] += b; a["bat_launches"] += dl["compose"]
            elif kernel_pass:
                ms, dms, dl, b = timed_ops(be.o, lambda: run_level(level, made))
                if it >= warmup:
                    a = acc[level]
                    a["ms"] += ms; a["kernel_ms"] += dms["compose"]; a["launches"] += dl["compose"]; a["bytes"] += b
                    a["ops"] += len(by_level[level])
            else:
                b0 = be.o.stats()["payload_bytes"]
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record()
                run_level(level, made)
                e1.record()
                torch.cuda.synchronize()
                acc[level]["b2b_ms"] += e0.elapsed_time(e1)
                acc[level]["b2b_bytes"] += be.o.stats()["payload_bytes"] - b0
        be.evict(made)
    assert be.o.sync_status() == 0
    out = {}
    for level, a in acc.items():
        rec = kernel_record(2 * a["bytes"], a["kernel_ms"], a["launches"], peak)
        lvl = 2 * a["b2b_bytes"] / (a["b2b_ms"] * 1e-3) / 1e9
        rec.update({"composes_per_level": len(by_level[level]), "copied_GB_per_compose": a["bytes"] / a["ops"] / 1e9,
                    "level_GBps": lvl, "level_frac": lvl / peak, "level_ms": a["b2b_ms"] / steps,
                    "level_note": "the level's composes issued back to back, events around the level",
                    "batched_level_GBps": 2 * a["bat_bytes"] / (a["bat_ms"] * 1e-3) / 1e9,
                    "batched_kernel_GBps": 2 * a["bat_bytes"] / (a["bat_kernel_ms"] * 1e-3) / 1e9,
                    "batched_kernel_frac": 2 * a["bat_bytes"] / (a["bat_kernel_ms"] * 1e-3) / 1e9 / peak,
                    "batched_launches_per_level": a["bat_launches"] / steps,
                    "batched_note": "the whole level as one aaf_kv_compose_batch call: one copy launch"})
        out[level] = rec
    del be
    torch.cuda.empty_cache()
    return out


# ------------------------------------------------------------------------------------------- other workloads
def extra_report(args):
    """Reports for the workloads that are parity cases rather than the headline step: the copy-on-write
    stress, the composition levels, metadata-only operators, host transfers and the churn trace.  One JSON line
    each, kernel GB/s from the library's CUDA events, bytes from the library's device-side byte counter."""
    import torch

    from paper_2607_10987_b200 import binding
    from tests.gpu_backend import GpuBackend
    from workloads import churn

    binding.load()
    assert torch.cuda.is_available()
    dev = torch.device("cuda", 0)
    peak, _ = hbm_peak()
    out = {"workload": args.workload, "engine": args.engine, "peak_GBps": peak}
    timed = lambda pool, fn, meta=False: (lambda r: (r[0], r[1], r[3]))(timed_ops(pool, fn, meta))

    if args.workload == "cow":
        out.update(cow_stress(args, peak, args.steps, args.warmup))
        out["llama70b_rows"] = cow_stress(args, peak, args.steps, args.warmup, n_layers=80)
    elif args.workload == "suffix":
        out.update(suffix_transfers(args, peak, args.steps, args.warmup))
    elif args.workload == "compose":
        out["share"] = compose_levels(args, peak, args.steps, args.warmup, copy_all=False)
        out["copy_all"] = compose_levels(args, peak, args.steps, args.warmup, copy_all=True)
    elif args.workload == "costmodel":
        # Transfer time of the paper's largest state over its network grid (Sec. 5.4: |KV| / BW + delta; Exp. 3:
        # 10-400 Gbps, 10 / 100 us), with the pack / unpack term measured here beside it, and the decision
        # pi(S) = transfer iff T_transfer < T_prefill for a range of assumed prefill times (the paper's measured
        # prefill times are not available).
        g = configs.Geometry(32, 8, 128, 16, 2, 8192, 8, 4096)
        seed, T = configs.SEED_BASE + 2, 32640
        be = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), engine=args.engine, init_fill=False,
                        staging_tokens=T)
        buf = be.payload(seed, 1, T)
        acc = {"materialize": [0.0, 0], "import": [0.0, 0]}
        for it in range(args.warmup + args.steps):
            res = {}
            _, dms, dl, _ = timed_ops(be.o, lambda: res.update(c=be.imp(buf, T)))
            _, dms2, dl2, _ = timed_ops(be.o, lambda: res.update(m=be.materialize(res["c"][1], 0, T)))
            assert res["c"][0] == 0 and res["m"][0] == 0
            be.evict([res["c"][1]])
            if it >= args.warmup:
                acc["import"][0] += dms["import"]; acc["import"][1] += dl["import"]
                acc["materialize"][0] += dms2["materialize"]; acc["materialize"][1] += dl2["materialize"]
        kv = binding.aaf_kv_state_bytes(g.n_layers, g.n_kv_heads, g.head_dim, g.elt_bytes, T)
        pack = 2 * kv * acc["materialize"][1] / (acc["materialize"][0] * 1e-3)   # bytes read + written per second
        unpack = 2 * kv * acc["import"][1] / (acc["import"][0] * 1e-3)
        rate = 2.0 / (1.0 / pack + 1.0 / unpack)  # one rate for pack and unpack together
        rows = []
        links = [(f"{gb} Gbps", gb * 1e9 / 8) for gb in (10, 25, 100, 200, 400)] + [("NVLink 5, 900 GB/s", 900e9)]
        for name, bw in links:
            for lat in (10e-6, 100e-6):
                wire = binding.aaf_kv_transfer_time(kv, bw, lat)
                full = binding.aaf_kv_transfer_time_packed(kv, bw, lat, rate)
                rows.append({"link": name, "latency_us": lat * 1e6, "T_transfer_ms": wire * 1e3,
                             "T_with_pack_unpack_ms": full * 1e3, "pack_unpack_share": (full - wire) / full,
                             "transfer_wins_if_prefill_exceeds_ms": full * 1e3,
                             "policy_at_prefill_1s": binding.aaf_kv_policy(False, full, 1.0),
                             "policy_at_prefill_100ms": binding.aaf_kv_policy(False, full, 0.1)})
        out.update({"state_tokens": T, "state_bytes": kv, "pack_GBps_read_plus_written": pack / 1e9,
                    "unpack_GBps_read_plus_written": unpack / 1e9, "pack_ms": 2 * kv / pack * 1e3,
                    "unpack_ms": 2 * kv / unpack * 1e3, "policy_codes": {"reuse": 0, "transfer": 1, "recompute": 2},
                    "rows": rows})
    elif args.workload == "meta":
        # metadata-only operators: rate of back-to-back calls (host launch + device execution), against the
        # rate of back-to-back launches of a trivial kernel on the same stream (the launch floor)
        g = configs.Geometry(32, 8, 128, 16, 2, 4096, 64, 2048)
        seed = configs.SEED_BASE + 2
        be = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), engine=args.engine, init_fill=False)
        T = 8192
        st, root = be.imp(be.payload(seed, 1, T), T)
        assert st == 0
        K = 200 * max(args.steps, 1)

        def rate(fn, calls_per_iter):
            for _ in range(20):
                fn()
            be.o.sync_status()
            t0 = time.perf_counter()
            for _ in range(K):
                fn()
            be.o.sync_status()  # synchronises both of the library's streams
            dt = time.perf_counter() - t0
            return {"calls_per_s": calls_per_iter * K / dt, "us_per_call": 1e6 * dt / (calls_per_iter * K)}

        def fork_evict():
            st, kids = be.fork(root, 16)
            assert st == 0
            assert be.evict(kids)[0] == 0

        def fork1_evict():
            st, kids = be.fork(root, 1)
            assert st == 0
            assert be.evict(kids)[0] == 0

        def compose_evict():  # block-aligned segments: the merge only builds a table (1024 shared entries)
            st, z = be.compose([root, root], 0)
            assert st == 0
            assert be.evict([z])[0] == 0

        one = torch.zeros(1, device=dev)

        def floor():
            one.add_(1.0)

        def breakdown(fn, wait):
            """one call at a time: time inside the call (host side: validation, launch, bookkeeping, binding) and
            time until the device has finished it"""
            host, total = [], []
            for _ in range(300):
                wait()
                t0 = time.perf_counter_ns()
                fn()
                t1 = time.perf_counter_ns()
                wait()
                t2 = time.perf_counter_ns()
                host.append(t1 - t0); total.append(t2 - t0)
            host.sort(); total.sort()
            return {"host_call_us_median": host[len(host) // 2] / 1e3, "call_plus_wait_us_median": total[len(total) // 2] / 1e3}

        kid = []

        def fork1():
            kid[:] = be.fork(root, 1)[1]

        def evict1():
            be.evict(kid)

        def fork_then_evict():  # keeps the handle count constant across iterations
            fork1(); evict1()

        out.update({"context_blocks": T // 16,
                    "fork16_then_evict16 (8192 + 8192 entries)": rate(fork_evict, 2),
                    "fork1_then_evict1 (512 + 512 entries)": rate(fork1_evict, 2),
                    "table_only_compose_then_evict (1024 entries)": rate(compose_evict, 2),
                    "launch_floor_trivial_torch_kernel": rate(floor, 1),
                    "one_call_at_a_time": {
                        "fork1_plus_evict1 (two calls)": breakdown(fork_then_evict, torch.cuda.synchronize),
                        "trivial_torch_kernel": breakdown(floor, torch.cuda.synchronize)}})
    elif args.workload == "transfer":
        # pack / unpack against host memory: one shot versus chunked with per-chunk completion flags
        g, seed, T = configs.LLAMA8B, configs.SEED_BASE + 2, 8187
        g = configs.Geometry(g.n_layers, g.n_kv_heads, g.head_dim, g.block_size, g.elt_bytes, 4096, 8, 1024)
        be = GpuBackend(g, seed, free_order=configs.free_order(seed, g.n_blocks), engine=args.engine, init_fill=False)
        pool = be.o
        h_src = torch.empty(T * g.bpt, dtype=torch.uint8).pin_memory()
        h_src.copy_(be.payload(seed, 1, T))
        h_dst = torch.empty(T * g.bpt, dtype=torch.uint8).pin_memory()
        staging = torch.empty(T * g.bpt, dtype=torch.uint8, device=dev)
        flags = torch.zeros(1024, dtype=torch.int32).pin_memory()
        fl = flags.numpy()
        st, c = pool.import_host(h_src, T, staging)
        assert st == 0
        rep = {}
        for chunk in (0, 512, 1024, 2048):
            first, total, imp = [], [], []
            for it in range(args.warmup + args.steps):
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                if chunk:
                    st, nch = pool.materialize_host_chunked(c, 0, T, h_dst, staging, chunk, flags)
                    assert st == 0
                    while fl[0] == 0:
                        pass
                    t_first = time.perf_counter() - t0
                else:
                    assert pool.materialize_host(c, 0, T, h_dst, staging) == 0
                    t_first = None
                torch.cuda.synchronize()
                t_total = time.perf_counter() - t0
                t1 = time.perf_counter()
                st, c2 = pool.import_host_chunked(h_dst, T, staging, chunk) if chunk else pool.import_host(h_dst, T, staging)
                assert st == 0
                torch.cuda.synchronize()
                t_imp = time.perf_counter() - t1
                pool.evict([c2])
                if it >= args.warmup:
                    total.append(t_total); imp.append(t_imp)
                    if t_first is not None:
                        first.append(t_first)
            rep["one_shot" if not chunk else f"chunk_{chunk}_tokens"] = {
                "materialize_to_host_ms": 1e3 * sum(total) / len(total),
                "first_chunk_on_host_ms": (1e3 * sum(first) / len(first)) if first else None,
                "import_from_host_ms": 1e3 * sum(imp) / len(imp)}
        assert torch.equal(h_dst, h_src)
        out.update({"context_tokens": T, "bytes_each_way_GB": T * g.bpt / 1e9, "modes": rep})
    else:  # churn
        bs, cap, seed = args.block_size, 32768, configs.SEED_BASE + 5
        small = lambda nb: configs.Geometry(1, 1, 8, bs, 2, nb, 80, cap // bs)
        be0 = GpuBackend(small(64 * cap // bs), seed, init_fill=False, staging_tokens=cap)
        d0 = churn.ChurnDriver(be0, seed, max_ctx_tokens=cap).run(10000)
        assert all(st == 0 for _, _, st in d0.log)
        demand = be0.o.stats()["peak_live_blocks"]
        del be0, d0
        nb = int(0.75 * demand)
        g = configs.Geometry(32, 8, 128, bs, 2, nb, 80, cap // bs)
        free_b, _ = torch.cuda.mem_get_info(dev)
        if g.pool_bytes + (12 << 30) > free_b:
            out.update({"skipped": "pool of %.1f GiB does not fit" % (g.pool_bytes / 2**30)})
        else:
            be = GpuBackend(g, seed, free_order=configs.free_order(seed, nb), engine=args.engine, init_fill=False,
                            staging_tokens=cap)
            be.window(0, 1)
            d = churn.ChurnDriver(be, seed, max_ctx_tokens=cap)
            t0 = time.perf_counter()
            ms, dms, b = timed(be.o, lambda: d.run(10000))
            wall = time.perf_counter() - t0
            assert be.o.sync_status() == 0
            calls = len(d.log)
            kms = sum(dms.values())
            # columnar catalog export of the final state (two kernels), timed with events over 20 repeats
            be.o.export_catalog()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(20):
                cols = be.o.export_catalog()
            e1.record()
            torch.cuda.synchronize()
            out.update({"catalog_export": {"states": int(cols["state_id"].numel()),
                                           "block_rows": int(cols["block_id"].numel()),
                                           "ms_per_export_including_buffer_allocation": e0.elapsed_time(e1) / 20}})
            # scored eviction (Alg. KV-Evict on the device): halve the live blocks by LRU score
            live0 = be.o.stats()["live_blocks"]
            t1 = time.perf_counter()
            st_e, victims = be.o.evict_to_budget(0.0, 0.0, 1.0, live0 // 2)
            t_evict = time.perf_counter() - t1
            assert st_e == 0
            out.update({"evict_to_budget": {"live_blocks_before": live0, "budget": live0 // 2, "victims": len(victims),
                                            "live_blocks_after": be.o.stats()["live_blocks"],
                                            "call_ms_including_sync": 1e3 * t_evict}})
            out.update({"block_size": bs, "demand_blocks": demand, "n_blocks": nb, "pool_GiB": g.pool_bytes / 2**30,
                        "library_calls": calls, "calls_by_kind": d.counts,
                        "oom_answers": sum(1 for _, _, st in d.log if st == churn.OOM_BLOCKS),
                        "moved_TB": 2 * b / 1e12, "stream_ms": ms, "wall_s": wall, "ops_per_s": 10000 / wall,
                        "calls_per_s": calls / wall, "GBps_whole_trace": 2 * b / wall / 1e9,
                        "copy_kernel_GBps": 2 * b / (kms * 1e-3) / 1e9, "peak_live_blocks": be.o.stats()["peak_live_blocks"],
                        "cow_count": be.o.stats()["cow_count"]})
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------- GPU arm
class Cluster:
    """Control plane of an N-replica run: barrier and max-over-ranks of a time.  No data-path collective."""

    def __init__(self, torch, dist, dev, world, backend):
        self.torch, self.dist, self.dev, self.world, self.backend = torch, dist, dev, world, backend

    def _sync(self):
        if self.torch.cuda.is_available():  # (the host-only self-test of this class runs without a device)
            self.torch.cuda.synchronize()

    def barrier(self):
        self._sync()
        if self.world > 1:
            self.dist.barrier()
            self._sync()

    def max_ms(self, ms):
        if self.world > 1:
            t = self.torch.tensor([ms], device=self.dev if self.backend == "nccl" else "cpu")
            self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    def run(self, steps, fn):
        """Exactly `steps` calls of fn between a barrier + synchronize on both sides; device time, max over ranks."""
        self.barrier()
        e0, e1 = self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        self.barrier()
        return self.max_ms(e0.elapsed_time(e1))


def measure_step(w, args, cl, dev_index, steps, warmup, min_seconds, clocks_for_rank0, do_e2e):
    """The fan-out step of workload `w` on a full-size pool: device-resident throughput, per-class kernel rates,
    and (optionally) the end-to-end form with host buffers.  Returns a dict of raw results."""
    import torch

    from paper_2607_10987_b200 import KVPool

    dev = torch.device("cuda", dev_index)
    g, seed, T, agents, n_new = w["g"], w["seed"], w["T"], w["agents"], w["n_new"]
    free_b, _total = torch.cuda.mem_get_info(dev)
    n_blocks = g.n_blocks
    need = lambda nb: g.n_layers * nb * 2 * g.run + 4 * T * g.bpt + (8 << 30)
    # blocks one step holds at its peak: sender's and receiver's context, every agent's continuation and COW block,
    # the merged pair
    step_blocks = 2 * g.nblk(T) + agents * (g.nblk(T + n_new) - g.nblk(T) + 1) + g.nblk(2 * (T + n_new)) + 64
    while need(n_blocks) > free_b and n_blocks // 2 >= step_blocks:
        n_blocks //= 2  # recorded in config.n_blocks when the device lacks memory for the full pool
    if need(n_blocks) > free_b:
        raise RuntimeError(f"{w['name']}: needs {need(n_blocks) / 2**30:.0f} GiB of device memory, "
                           f"{free_b / 2**30:.0f} GiB are free")
    pool = KVPool(g.n_layers, g.n_kv_heads, g.head_dim, g.block_size, g.elt_bytes, n_blocks, g.max_ctx,
                  g.max_blocks_per_ctx, free_order=configs.free_order(seed, n_blocks), device=dev_index)
    pool.set_copy_engine(args.engine)
    elems = lambda n: g.n_layers * 2 * n * g.row // 2
    root_buf = fill.fill_torch(seed, 1, 0, elems(T), dev).view(torch.uint8)
    agent_bufs = [fill.fill_torch(seed, 2 + i, 0, elems(n_new), dev).view(torch.uint8) for i in range(agents)]
    staging = torch.empty(T * g.bpt, dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()
    dev_step = lambda: step_ops(pool, root_buf, agent_bufs, T, agents, n_new, staging)

    # ---- device-resident measurement: `repeats` timed regions of exactly `steps` steps each
    ms_warm = cl.run(max(warmup, 1), dev_step) / max(warmup, 1)
    repeats = max(1, min(400, int(np.ceil(1.15 * min_seconds * 1e3 / max(ms_warm * steps, 1e-3)))))
    s0 = pool.stats()
    pool.set_timing(True)
    sampler = None
    if clocks_for_rank0:
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        smi_id = vis.split(",")[dev_index].strip() if vis and dev_index < len(vis.split(",")) else str(dev_index)
        sampler = ClockSampler(smi_id)
    region_ms = [cl.run(steps, dev_step) for _ in range(repeats)]
    clocks = sampler.stop() if sampler else None
    pool.set_timing(False)
    s1 = pool.stats()
    assert pool.sync_status() == 0
    total_steps = steps * repeats
    ms = sum(region_ms)
    moved_per_step = 2 * (s1["payload_bytes"] - s0["payload_bytes"]) / total_steps  # read + written
    copy_launches = sum(s1["copy_launches"].values()) - sum(s0["copy_launches"].values())
    meta_launches = s1["meta_launches"] - s0["meta_launches"]
    copy_ms = sum(s1["copy_ms"].values()) - sum(s0["copy_ms"].values())
    assert sum(s1["timed_launches"].values()) - sum(s0["timed_launches"].values()) == copy_launches
    ct = class_tokens(g, T, agents, n_new)
    assert 2 * sum(ct.values()) * g.bpt == moved_per_step, (ct, moved_per_step)
    per_class = {}
    for k, toks in ct.items():
        dms = s1["copy_ms"][k] - s0["copy_ms"][k]
        per_class[k] = (2 * toks * g.bpt * total_steps / (dms * 1e-3) / 1e9) if dms > 0 else None
    res = {"name": w["name"], "n_blocks": n_blocks, "pool_GiB": g.n_layers * n_blocks * 2 * g.run / 2**30,
           "ms_per_step": ms / total_steps, "repeats": repeats, "region_ms": region_ms,
           "moved_per_step": moved_per_step, "value_per_replica": moved_per_step * total_steps / (ms * 1e-3) / 1e9,
           "copy_launches": copy_launches, "meta_launches": meta_launches, "copy_ms": copy_ms,
           "per_class": per_class, "clocks": clocks, "launches_per_region": (copy_launches + meta_launches) // repeats,
           "e2e": None}

    # ---- end to end: every input of the step comes from pinned host memory through the library's host-buffer
    # calls, and the materialised transfer buffer goes back to the host, all inside the timed region
    if do_e2e:
        h_root = torch.empty(T * g.bpt, dtype=torch.uint8).pin_memory()
        h_agents = [torch.empty(n_new * g.bpt, dtype=torch.uint8).pin_memory() for _ in range(agents)]
        h_out = torch.empty(T * g.bpt, dtype=torch.uint8).pin_memory()
        h_root.copy_(root_buf)
        for h, d in zip(h_agents, agent_bufs):
            h.copy_(d)
        d_root = torch.empty_like(root_buf)
        d_agents = torch.empty(agents * n_new * g.bpt, dtype=torch.uint8, device=dev)
        chunk = 1024 if T >= 4096 else max(g.block_size, (T // 4) // g.block_size * g.block_size)

        def e2e_step():
            st, root = pool.import_host_chunked(h_root, T, d_root, chunk)  # H2D chunk c+1 overlaps the scatter of chunk c
            assert st == 0, st
            st, _ = pool.materialize_host_chunked(root, 0, T, h_out, staging, chunk)  # gather c+1 overlaps D2H of c
            assert st == 0, st
            st, recv = pool.imp(staging, T)
            assert st == 0, st
            st, kids = pool.fork(recv, agents)
            assert st == 0, st
            st = pool.append_host(kids, [n_new] * agents, h_agents, d_agents)  # H2D of the continuation tokens + scatter
            assert st == 0, st
            st, merged = pool.compose(kids[:2], 0)
            assert st == 0, st
            st, _ = pool.evict([root, recv] + kids + [merged])
            assert st == 0, st

        k_e2e = max(3, min(steps, 10))
        cl.run(1, e2e_step)
        ms_e2e = cl.run(k_e2e, e2e_step)
        assert torch.equal(h_out, h_root), "end-to-end round trip changed the payload"
        h2d, d2h = (T + agents * n_new) * g.bpt, T * g.bpt

        # what PCIe allows for this step: plain copies of the same pinned buffers, each direction alone and both at
        # once (the directions slow each other down).  A step must upload h2d bytes and download d2h bytes; in
        # steady state the download of one step overlaps uploads of the same and the next step.
        def copy_ms(pairs):
            evs = []
            torch.cuda.synchronize()
            for dst, src in pairs:
                strm = torch.cuda.Stream(dev)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                with torch.cuda.stream(strm):
                    e0.record(strm)
                    dst.copy_(src, non_blocking=True)
                    e1.record(strm)
                evs.append((e0, e1))
            torch.cuda.synchronize()
            return [a.elapsed_time(b) for a, b in evs]

        copy_ms([(d_root, h_root)])
        up = h_root.numel() / copy_ms([(d_root, h_root)])[0] / 1e6
        down = h_out.numel() / copy_ms([(h_out, staging)])[0] / 1e6
        both = copy_ms([(d_root, h_root), (h_out, staging)])
        up2, down2 = h_root.numel() / both[0] / 1e6, h_out.numel() / both[1] / 1e6
        t_overlap = d2h / down2 / 1e6                      # ms with both directions busy
        rest_up = max(h2d - t_overlap * up2 * 1e6, 0.0)    # upload bytes left for the time the download is idle
        floor_ms = t_overlap + rest_up / up / 1e6
        res["e2e"] = {"value_per_replica": moved_per_step * k_e2e / (ms_e2e * 1e-3) / 1e9, "unit": UNIT,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / k_e2e,
                      "steps": k_e2e, "pcie_GBps_each_way": [h2d / (ms_e2e / k_e2e * 1e-3) / 1e9,
                                                              d2h / (ms_e2e / k_e2e * 1e-3) / 1e9],
                      "api": "aaf_kv_import_host_chunked, aaf_kv_materialize_host_chunked, aaf_kv_append_host",
                      "pcie_probe_GBps": {"h2d_alone": up, "d2h_alone": down, "h2d_with_d2h": up2, "d2h_with_h2d": down2},
                      "pcie_floor_ms_per_step": floor_ms, "frac_of_pcie_floor": floor_ms / (ms_e2e / k_e2e)}
    pool.close()
    del pool, root_buf, agent_bufs, staging
    torch.cuda.empty_cache()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b", choices=["8b", "8b-aligned", "70b", "8b-small", "tiny", "cow", "compose",
                                                         "churn", "transfer", "meta", "costmodel", "suffix"])
    ap.add_argument("--block-size", type=int, default=16, help="churn workload only: 8, 16, 32 or 64")
    ap.add_argument("--engine", type=int, default=0, help="0 auto, 1 vector LD/ST per CTA, 2 cp.async.bulk, 3 vector LD/ST per warp")
    ap.add_argument("--min-seconds", type=float, default=1.0, help="repeat the timed region until this much device time is measured")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip roofline.per_workload (70B step, compose levels, COW stress)")
    args = ap.parse_args()
    if args.workload in ("cow", "compose", "churn", "transfer", "meta", "costmodel", "suffix"):
        return extra_report(args)
    w = workload(args.workload)
    if args.impl == "reference":
        reference_arm(args, w)
        return

    import torch
    import torch.distributed as dist

    from paper_2607_10987_b200 import binding

    binding.load()  # fails loudly if the CUDA library is missing: there is no fallback
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    dev_index = local_rank % torch.cuda.device_count()  # one rank per GPU; the modulo only matters in self-tests
    torch.cuda.set_device(dev_index)
    dev = torch.device("cuda", dev_index)
    backend = os.environ.get("AAFKV_BENCH_DIST_BACKEND", "nccl")  # control plane only: barrier + max of the time
    if world > 1:
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=dev)
        else:
            dist.init_process_group(backend)
    cl = Cluster(torch, dist, dev, world, backend)
    peak, peak_src = hbm_peak()

    r = measure_step(w, args, cl, dev_index, args.steps, max(args.warmup, 3), args.min_seconds, rank == 0,
                     not args.no_e2e)
    g = w["g"]
    total_steps = args.steps * r["repeats"]
    roofline = {"bound": "hbm", "kernel": "copy engine (aafkv::copy_bulk_kernel; copy_warp_kernel for small pieces)"}
    roofline.update(kernel_record(r["moved_per_step"] * total_steps, r["copy_ms"], r["copy_launches"], peak))
    roofline.update({"peak": peak, "peak_source": peak_src, "per_class_GBps": r["per_class"]})

    # ---- the other full-size workloads of the throughput target, same run, same library
    if args.workload == "8b" and not args.no_extra:
        single = Cluster(torch, dist, dev, 1, backend)  # replicas do not wait for each other here
        pw = {}
        k = max(3, min(args.steps, 10))

        def step70():
            r70 = measure_step(workload("70b"), args, single, dev_index, k, 3, args.min_seconds, False, False)
            rec = kernel_record(r70["moved_per_step"] * k * r70["repeats"], r70["copy_ms"], r70["copy_launches"], peak)
            rec.update({"workload": r70["name"], "whole_step_GBps": r70["value_per_replica"],
                        "ms_per_step": r70["ms_per_step"], "repeats": r70["repeats"], "pool_GiB": r70["pool_GiB"],
                        "per_class_GBps": r70["per_class"]})
            return {"70b": rec}

        parts = (step70,
                 lambda: {"compose_" + n: lv for n, lv in compose_levels(args, peak, k, 2, copy_all=False).items()},
                 lambda: {"cow": cow_stress(args, peak, k, 2)},
                 lambda: {"cow_70b": cow_stress(args, peak, k, 2, n_layers=80)},
                 lambda: {"suffix_" + n: rec for n, rec in suffix_transfers(args, peak, k, 2).items()
                          if isinstance(rec, dict)})
        for part in parts:  # a sub-workload that cannot run here (device memory) must not cost the headline line
            try:
                pw.update(part())
            except (RuntimeError, AssertionError) as exc:
                pw.setdefault("skipped", []).append(f"{type(exc).__name__}: {str(exc)[:200]}")
                torch.cuda.empty_cache()
        roofline["per_workload"] = pw

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu_baseline = None
    if not args.no_cpu_baseline:
        layers = 2 if g.n_layers > 2 else g.n_layers
        gbps, steps_c, dt, _ = oracle_rate(w, layers, budget_s=12.0, max_steps=2000)
        cpu_baseline = {"value": gbps, "unit": UNIT, "cores": 1, "kind": "oracle",
                        "sample": f"{layers} of {g.n_layers} layers of the same step, {steps_c} passes in {dt:.1f} s, "
                                  f"single thread of {len(os.sched_getaffinity(0))} available cores"}
    e2e = r["e2e"]
    if e2e is not None:
        e2e = dict(e2e)
        e2e["value"] = world * e2e.pop("value_per_replica")
    line = {
        "metric": METRIC, "value": world * r["value_per_replica"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "repeats": r["repeats"], "timed_seconds": sum(r["region_ms"]) / 1e3,
        "config": step_config(w, r["n_blocks"], args.engine),
        "ops_per_s": world * 7 * total_steps / (sum(r["region_ms"]) * 1e-3),
        "gpu_launches": r["launches_per_region"],
        "clocks": r["clocks"], "e2e": e2e, "roofline": roofline, "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
