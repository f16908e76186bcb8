"""ctypes wrapper around the sequential paged-pool oracle -- TEST INFRASTRUCTURE.

``build()`` compiles ``kv_paged_oracle.c`` with gcc into ``libkvoracle.so`` next to
it; ``PagedOracle`` exposes the operators on numpy buffers.  Nothing here touches
the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kv_paged_oracle.c")
_LIB = os.path.join(_HERE, "libkvoracle.so")

OK, INVALID_ARG, BAD_CTX, OOM_BLOCKS, OOM_CTX, TOO_LONG, DST_TOO_SMALL = 0, -1, -2, -3, -4, -5, -7
COMPOSE_COPY_ALL = 1
STATE_COLUMNS = ("state_id", "n_tokens", "reuse", "last_access", "origin", "parent", "born", "parent_born")

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (plain gcc -O2, one translation unit)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-Wall", "-Wextra", "-fPIC", "-shared", _SRC, "-o", _LIB]
        )
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64, u32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32
        p32, p64 = C.POINTER(C.c_int32), C.POINTER(C.c_int64)
        L.kvo_create.restype = vp
        L.kvo_create.argtypes = [i32] * 8 + [p32]
        L.kvo_destroy.argtypes = [vp]
        L.kvo_destroy.restype = None
        L.kvo_clone.restype = vp
        L.kvo_clone.argtypes = [vp]
        L.kvo_pool_bytes.restype = vp
        L.kvo_pool_bytes.argtypes = [vp]
        L.kvo_pool_nbytes.restype = i64
        L.kvo_pool_nbytes.argtypes = [vp]
        L.kvo_import.argtypes = [vp, vp, i64, p32]
        L.kvo_materialize.argtypes = [vp, i32, i64, i64, vp, i64]
        L.kvo_fork.argtypes = [vp, i32, i32, p32]
        L.kvo_append.argtypes = [vp, i32, p32, p32, C.POINTER(vp)]
        L.kvo_compose.argtypes = [vp, i32, p32, u32, p32]
        L.kvo_evict.argtypes = [vp, i32, p32]
        L.kvo_ctx_len.argtypes = [vp, i32, p64]
        L.kvo_get_table.argtypes = [vp, i32, p32, i32, p32]
        L.kvo_get_refcounts.argtypes = [vp, p32]
        L.kvo_get_free_list.argtypes = [vp, p32, p32]
        L.kvo_stats.argtypes = [vp, p64]
        L.kvo_evict_to_budget.argtypes = [vp, C.c_double, C.c_double, C.c_double, i64, p32, i32, p32]
        L.kvo_get_catalog.argtypes = [vp, p64, p64, p64]
        L.kvo_export_catalog.argtypes = [vp, p32, p64, p64, p64, p32, p32, p64, p64, p32, p32, p64, p64, p32, p64, p32, p32]
        _lib = L
    return _lib


def _i32arr(v):
    a = np.ascontiguousarray(np.asarray(v, dtype=np.int32))
    return a, a.ctypes.data_as(C.POINTER(C.c_int32))


class PagedOracle:
    """Sequential paged KV pool on the CPU.  Methods return (status, result)."""

    def __init__(self, L, H, D, BS, E, NB, max_ctx, max_blk, free_order=None, _handle=None):
        self.L, self.H, self.D, self.BS, self.E, self.NB = L, H, D, BS, E, NB
        self.max_ctx, self.max_blk = max_ctx, max_blk
        self.row = H * D * E
        self.bpt = 2 * L * self.row
        if _handle is not None:
            self.h = _handle
            return
        fo = None
        if free_order is not None:
            fo_arr, fo = _i32arr(free_order)
            assert sorted(fo_arr.tolist()) == list(range(NB)), "free_order must be a permutation"
        self.h = lib().kvo_create(L, H, D, BS, E, NB, max_ctx, max_blk, fo)
        if not self.h:
            raise MemoryError("kvo_create failed")

    def close(self):
        if self.h:
            lib().kvo_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def clone(self) -> "PagedOracle":
        h = lib().kvo_clone(self.h)
        return PagedOracle(self.L, self.H, self.D, self.BS, self.E, self.NB, self.max_ctx, self.max_blk, _handle=h)

    # -- pool image -------------------------------------------------------
    def pool_view(self) -> np.ndarray:
        """uint8 view [L, NB, 2, BS, row] of the oracle's own pool memory (no copy)."""
        n = lib().kvo_pool_nbytes(self.h)
        buf = (C.c_uint8 * n).from_address(lib().kvo_pool_bytes(self.h))
        return np.frombuffer(buf, dtype=np.uint8).reshape(self.L, self.NB, 2, self.BS, self.row)

    # -- operators --------------------------------------------------------
    def imp(self, buf: np.ndarray, n: int):
        buf = np.ascontiguousarray(buf).view(np.uint8).reshape(-1)
        assert buf.size == n * self.bpt, (buf.size, n, self.bpt)
        out = C.c_int32(-1)
        st = lib().kvo_import(self.h, buf.ctypes.data, n, C.byref(out))
        return st, (out.value if st == OK else None)

    def materialize(self, c: int, t0: int, t1: int, dst_bytes: int | None = None):
        n = max(t1 - t0, 0)
        nbytes = n * self.bpt if dst_bytes is None else dst_bytes
        dst = np.zeros(max(nbytes, 1), dtype=np.uint8)
        st = lib().kvo_materialize(self.h, c, t0, t1, dst.ctypes.data, nbytes)
        return st, (dst[: n * self.bpt] if st == OK else None)

    def fork(self, parent: int, k: int):
        out = np.full(max(k, 1), -1, dtype=np.int32)
        st = lib().kvo_fork(self.h, parent, k, out.ctypes.data_as(C.POINTER(C.c_int32)))
        return st, (out[:k].tolist() if st == OK else None)

    def append(self, ctxs, n_new, srcs):
        n = len(ctxs)
        _, cp = _i32arr(ctxs)
        _, npn = _i32arr(n_new)
        keep = [np.ascontiguousarray(s).view(np.uint8).reshape(-1) for s in srcs]
        for s, nn in zip(keep, n_new):
            assert s.size == nn * self.bpt
        ptrs = (C.c_void_p * max(n, 1))(*[s.ctypes.data for s in keep])
        st = lib().kvo_append(self.h, n, cp, npn, ptrs)
        return st, None

    def compose(self, segs, flags: int = 0):
        _, sp = _i32arr(segs)
        out = C.c_int32(-1)
        st = lib().kvo_compose(self.h, len(segs), sp, flags, C.byref(out))
        return st, (out.value if st == OK else None)

    def evict(self, ctxs):
        _, cp = _i32arr(ctxs)
        st = lib().kvo_evict(self.h, len(ctxs), cp)
        return st, None

    def evict_to_budget(self, alpha, beta, gamma, budget_blocks):
        out = np.full(self.max_ctx, -1, dtype=np.int32)
        nv = C.c_int32(0)
        st = lib().kvo_evict_to_budget(self.h, alpha, beta, gamma, budget_blocks,
                                       out.ctypes.data_as(C.POINTER(C.c_int32)), self.max_ctx, C.byref(nv))
        return st, (out[: nv.value].tolist() if st == OK else None)

    def catalog(self):
        clock = C.c_int64(0)
        reuse = np.empty(self.max_ctx, dtype=np.int64)
        last = np.empty(self.max_ctx, dtype=np.int64)
        lib().kvo_get_catalog(self.h, C.byref(clock), reuse.ctypes.data_as(C.POINTER(C.c_int64)),
                              last.ctypes.data_as(C.POINTER(C.c_int64)))
        return {"clock": clock.value, "reuse": reuse.tolist(), "last_access": last.tolist()}

    def export_catalog(self) -> dict:
        """Columnar catalog: dict of numpy columns (see kvo_export_catalog)."""
        cap_rows = self.max_ctx * self.max_blk
        i32 = lambda n: np.zeros(n, dtype=np.int32)
        i64 = lambda n: np.zeros(n, dtype=np.int64)
        cols = {"state_id": i32(self.max_ctx), "n_tokens": i64(self.max_ctx), "reuse": i64(self.max_ctx),
                "last_access": i64(self.max_ctx), "origin": i32(self.max_ctx), "parent": i32(self.max_ctx),
                "born": i64(self.max_ctx), "parent_born": i64(self.max_ctx),
                "block_offsets": i32(self.max_ctx + 1), "block_id": i32(cap_rows),
                "pos_begin": i64(cap_rows), "pos_end": i64(cap_rows), "refcount": i32(cap_rows),
                "address": i64(cap_rows)}
        ns, nr = C.c_int32(0), C.c_int32(0)
        P32, P64 = C.POINTER(C.c_int32), C.POINTER(C.c_int64)
        ptr = lambda k: cols[k].ctypes.data_as(P32 if cols[k].dtype == np.int32 else P64)
        lib().kvo_export_catalog(self.h, ptr("state_id"), ptr("n_tokens"), ptr("reuse"), ptr("last_access"),
                                 ptr("origin"), ptr("parent"), ptr("born"), ptr("parent_born"), ptr("block_offsets"), ptr("block_id"), ptr("pos_begin"), ptr("pos_end"),
                                 ptr("refcount"), ptr("address"), C.byref(ns), C.byref(nr))
        out = {}
        for k, v in cols.items():
            n = ns.value + 1 if k == "block_offsets" else (ns.value if k in STATE_COLUMNS else nr.value)
            out[k] = v[:n].copy()
        return out

    # -- introspection ----------------------------------------------------
    def ctx_len(self, c: int):
        v = C.c_int64(-1)
        st = lib().kvo_ctx_len(self.h, c, C.byref(v))
        return v.value if st == OK else None

    def table(self, c: int):
        out = np.empty(self.max_blk, dtype=np.int32)
        nb = C.c_int32(0)
        st = lib().kvo_get_table(self.h, c, out.ctypes.data_as(C.POINTER(C.c_int32)), self.max_blk, C.byref(nb))
        assert st == OK, st
        return out[: nb.value].copy()

    def refcounts(self):
        out = np.empty(self.NB, dtype=np.int32)
        lib().kvo_get_refcounts(self.h, out.ctypes.data_as(C.POINTER(C.c_int32)))
        return out

    def free_list(self):
        out = np.empty(self.NB, dtype=np.int32)
        nf = C.c_int32(0)
        lib().kvo_get_free_list(self.h, out.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(nf))
        return out[: nf.value].copy()

    def stats(self):
        out = np.zeros(6, dtype=np.int64)
        lib().kvo_stats(self.h, out.ctypes.data_as(C.POINTER(C.c_int64)))
        keys = ["free_blocks", "live_blocks", "peak_live_blocks", "live_ctx", "cow_count", "rows_copied"]
        return dict(zip(keys, out.tolist()))

    def live_ctxs(self):
        return [c for c in range(self.max_ctx) if self.ctx_len(c) is not None]
