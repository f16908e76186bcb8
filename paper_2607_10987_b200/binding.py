"""ctypes binding of libaafkv.so: the same entry points as include/aaf_kv.h, argument
marshalling only.  Every step of the path runs in the library's kernels; there is no Python
or CPU fallback, and loading fails loudly if the shared library is missing.

``KVPool`` is a convenience holder: it lets PyTorch allocate the pool, the workspace and
transfer buffers (PyTorch is used for device memory and streams only) and forwards to the
C entry points with the current stream.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libaafkv.so")

AAF_KV_ABI_VERSION = 1
AAF_OK = 0
AAF_ERR_INVALID_ARG, AAF_ERR_BAD_CTX, AAF_ERR_OOM_BLOCKS, AAF_ERR_OOM_CTX = -1, -2, -3, -4
AAF_ERR_TOO_LONG, AAF_ERR_INCOMPAT, AAF_ERR_DST_TOO_SMALL, AAF_ERR_CUDA = -5, -6, -7, -8
AAF_ERR_CORRUPT, AAF_ERR_TIMEOUT, AAF_ERR_TOO_MANY, AAF_ERR_SCRATCH_LIMIT = -9, -10, -11, -12
AAF_NOALLOC_MAX_BLOCKS = 4096
AAF_COMPOSE_SHARE, AAF_COMPOSE_COPY_ALL = 0, 1
AAF_POLICY_REUSE, AAF_POLICY_TRANSFER, AAF_POLICY_RECOMPUTE = 0, 1, 2
AAF_ENGINE_AUTO, AAF_ENGINE_VEC, AAF_ENGINE_BULK, AAF_ENGINE_WARP = 0, 1, 2, 3
AAF_OP_MATERIALIZE, AAF_OP_IMPORT, AAF_OP_APPEND, AAF_OP_COMPOSE, AAF_OP_CLASSES = 0, 1, 2, 3, 4
OP_NAMES = ("materialize", "import", "append", "compose")


class aaf_kv_pool_desc(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("abi_version", C.c_uint32),
        ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("block_size", C.c_int32),
        ("elt_bytes", C.c_int32), ("n_blocks", C.c_int32), ("max_ctx", C.c_int32),
        ("max_blocks_per_ctx", C.c_int32), ("max_batch", C.c_int32), ("device", C.c_int32),
        ("pool_base", C.c_void_p), ("layer_stride_bytes", C.c_size_t),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("free_order", C.POINTER(C.c_int32)),
        ("model_id", C.c_uint64), ("config_hash", C.c_uint64),
    ]


class aaf_kv_xfer_desc(C.Structure):
    _fields_ = [
        ("model_id", C.c_uint64), ("config_hash", C.c_uint64),
        ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("elt_bytes", C.c_int32),
        ("pos_start", C.c_int64), ("n_tokens", C.c_int64),
    ]


class aaf_kv_stats(C.Structure):
    _fields_ = [
        ("free_blocks", C.c_int64), ("live_blocks", C.c_int64), ("peak_live_blocks", C.c_int64),
        ("live_ctx", C.c_int64), ("cow_count", C.c_int64), ("payload_bytes", C.c_int64),
        ("copy_launches", C.c_int64 * AAF_OP_CLASSES), ("meta_launches", C.c_int64),
        ("copy_ms", C.c_double * AAF_OP_CLASSES), ("timed_launches", C.c_int64 * AAF_OP_CLASSES),
    ]


class aaf_kv_catalog_cols(C.Structure):
    _fields_ = [("state_id", C.c_void_p), ("n_tokens", C.c_void_p), ("reuse", C.c_void_p), ("last_access", C.c_void_p),
                ("origin", C.c_void_p), ("parent", C.c_void_p), ("born", C.c_void_p), ("parent_born", C.c_void_p),
                ("block_offsets", C.c_void_p), ("block_id", C.c_void_p), ("pos_begin", C.c_void_p),
                ("pos_end", C.c_void_p), ("refcount", C.c_void_p), ("address", C.c_void_p)]


# every symbol include/aaf_kv.h declares: name -> (restype, argtypes)
_vp, _i32, _i64, _u32, _sz = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_size_t
_p32 = C.POINTER(C.c_int32)
SYMBOLS = {
    "aaf_kv_pool_workspace_bytes": (_sz, [C.POINTER(aaf_kv_pool_desc)]),
    "aaf_kv_pool_create": (C.c_int, [C.POINTER(aaf_kv_pool_desc), C.POINTER(_vp)]),
    "aaf_kv_pool_destroy": (C.c_int, [_vp]),
    "aaf_kv_materialize": (C.c_int, [_vp, _i32, _i64, _i64, _vp, _sz, C.POINTER(aaf_kv_xfer_desc), _vp]),
    "aaf_kv_import": (C.c_int, [_vp, _vp, C.POINTER(aaf_kv_xfer_desc), _p32, _vp]),
    "aaf_kv_materialize_batch": (C.c_int, [_vp, _i32, _p32, C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_vp),
                                           C.POINTER(_sz), C.POINTER(aaf_kv_xfer_desc), _vp]),
    "aaf_kv_import_batch": (C.c_int, [_vp, _i32, C.POINTER(_vp), C.POINTER(aaf_kv_xfer_desc), _p32, _vp]),
    "aaf_kv_fork": (C.c_int, [_vp, _i32, _i32, _p32, _vp]),
    "aaf_kv_append": (C.c_int, [_vp, _i32, _p32, _p32, C.POINTER(_vp), _vp]),
    "aaf_kv_compose": (C.c_int, [_vp, _i32, _p32, _u32, _p32, _vp]),
    "aaf_kv_compose_batch": (C.c_int, [_vp, _i32, _p32, _p32, _u32, _p32, _vp]),
    "aaf_kv_evict": (C.c_int, [_vp, _i32, _p32, _vp]),
    "aaf_kv_materialize_host": (C.c_int, [_vp, _i32, _i64, _i64, _vp, _sz, _vp, _sz, C.POINTER(aaf_kv_xfer_desc), _vp]),
    "aaf_kv_import_host": (C.c_int, [_vp, _vp, C.POINTER(aaf_kv_xfer_desc), _vp, _sz, _p32, _vp]),
    "aaf_kv_append_host": (C.c_int, [_vp, _i32, _p32, _p32, C.POINTER(_vp), _vp, _sz, _vp]),
    "aaf_kv_materialize_host_chunked": (C.c_int, [_vp, _i32, _i64, _i64, _vp, _sz, _vp, _sz, _i32, C.POINTER(C.c_uint32),
                                                  _i32, _p32, C.POINTER(aaf_kv_xfer_desc), _vp]),
    "aaf_kv_import_host_chunked": (C.c_int, [_vp, _vp, C.POINTER(aaf_kv_xfer_desc), _vp, _sz, _i32, _p32, _vp]),
    "aaf_kv_evict_to_budget": (C.c_int, [_vp, C.c_double, C.c_double, C.c_double, _i64, _p32, _i32, _p32, _vp]),
    "aaf_kv_catalog_rows": (C.c_int, [_vp, _p32, C.POINTER(_i64)]),
    "aaf_kv_export_catalog": (C.c_int, [_vp, C.POINTER(aaf_kv_catalog_cols), _vp]),
    "aaf_kv_get_catalog": (C.c_int, [_vp, C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64)]),
    "aaf_kv_ctx_len": (C.c_int, [_vp, _i32, C.POINTER(_i64)]),
    "aaf_kv_get_table": (C.c_int, [_vp, _i32, _p32, _i32, _p32]),
    "aaf_kv_get_refcounts": (C.c_int, [_vp, _p32]),
    "aaf_kv_get_free_list": (C.c_int, [_vp, _p32, _p32]),
    "aaf_kv_pool_stats": (C.c_int, [_vp, C.POINTER(aaf_kv_stats)]),
    "aaf_kv_sync_status": (C.c_int, [_vp]),
    "aaf_kv_set_copy_engine": (C.c_int, [_vp, C.c_int]),
    "aaf_kv_set_timing": (C.c_int, [_vp, C.c_int]),
    "aaf_kv_materialize_noalloc": (C.c_int, [_vp, _sz, _i32, _i32, _i32, _i32, _i32, _i32, _p32, _i32, _i64, _i64, _vp,
                                             _sz, _vp]),
    "aaf_kv_state_bytes": (C.c_int64, [_i32, _i32, _i32, _i32, _i64]),
    "aaf_kv_transfer_time": (C.c_double, [C.c_double, C.c_double, C.c_double]),
    "aaf_kv_transfer_time_packed": (C.c_double, [C.c_double, C.c_double, C.c_double, C.c_double]),
    "aaf_kv_policy": (C.c_int, [C.c_int, C.c_double, C.c_double]),
    "aaf_kv_debug_expire_wait": (C.c_int, [_vp, C.c_uint64, _vp]),
    "aaf_kv_debug_mark_unusable": (C.c_int, [_vp]),
    "aaf_kv_strerror": (C.c_char_p, [C.c_int]),
}

_lib = None


def load():
    """Loads libaafkv.so (raises if it has not been built: there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2607_10987_b200._build` "
                "(nvcc, sm_100a). There is no CPU or PyTorch fallback for the KV operators."
            )
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _fn(name):
    return getattr(load(), name)


# thin same-name wrappers ---------------------------------------------------------------------
def aaf_kv_pool_workspace_bytes(desc): return _fn("aaf_kv_pool_workspace_bytes")(C.byref(desc))
def aaf_kv_pool_create(desc, out): return _fn("aaf_kv_pool_create")(C.byref(desc), C.byref(out))
def aaf_kv_pool_destroy(pool): return _fn("aaf_kv_pool_destroy")(pool)
def aaf_kv_materialize(pool, ctx, t0, t1, dst, dst_bytes, out_desc, stream):
    return _fn("aaf_kv_materialize")(pool, ctx, t0, t1, dst, dst_bytes, out_desc, stream)
def aaf_kv_import(pool, src, desc, out_ctx, stream): return _fn("aaf_kv_import")(pool, src, desc, out_ctx, stream)
def aaf_kv_materialize_batch(pool, n, ctxs, t0, t1, dsts, dst_bytes, out_descs, stream):
    return _fn("aaf_kv_materialize_batch")(pool, n, ctxs, t0, t1, dsts, dst_bytes, out_descs, stream)
def aaf_kv_import_batch(pool, n, srcs, descs, out_ctxs, stream):
    return _fn("aaf_kv_import_batch")(pool, n, srcs, descs, out_ctxs, stream)
def aaf_kv_fork(pool, parent, k, out_children, stream): return _fn("aaf_kv_fork")(pool, parent, k, out_children, stream)
def aaf_kv_append(pool, n, ctxs, n_new, srcs, stream): return _fn("aaf_kv_append")(pool, n, ctxs, n_new, srcs, stream)
def aaf_kv_compose(pool, m, segs, flags, out_ctx, stream): return _fn("aaf_kv_compose")(pool, m, segs, flags, out_ctx, stream)
def aaf_kv_compose_batch(pool, n_out, seg_off, segs, flags, out_ctxs, stream):
    return _fn("aaf_kv_compose_batch")(pool, n_out, seg_off, segs, flags, out_ctxs, stream)
def aaf_kv_evict(pool, n, ctxs, stream): return _fn("aaf_kv_evict")(pool, n, ctxs, stream)
def aaf_kv_materialize_host(pool, ctx, t0, t1, dst_host, dst_bytes, staging, staging_bytes, out_desc, stream):
    return _fn("aaf_kv_materialize_host")(pool, ctx, t0, t1, dst_host, dst_bytes, staging, staging_bytes, out_desc, stream)
def aaf_kv_import_host(pool, src_host, desc, staging, staging_bytes, out_ctx, stream):
    return _fn("aaf_kv_import_host")(pool, src_host, desc, staging, staging_bytes, out_ctx, stream)
def aaf_kv_append_host(pool, n, ctxs, n_new, srcs_host, staging, staging_bytes, stream):
    return _fn("aaf_kv_append_host")(pool, n, ctxs, n_new, srcs_host, staging, staging_bytes, stream)
def aaf_kv_materialize_host_chunked(pool, ctx, t0, t1, dst_host, dst_bytes, staging, staging_bytes, chunk_tokens,
                                    done_flags, flags_cap, n_chunks_out, out_desc, stream):
    return _fn("aaf_kv_materialize_host_chunked")(pool, ctx, t0, t1, dst_host, dst_bytes, staging, staging_bytes,
                                                  chunk_tokens, done_flags, flags_cap, n_chunks_out, out_desc, stream)
def aaf_kv_import_host_chunked(pool, src_host, desc, staging, staging_bytes, chunk_tokens, out_ctx, stream):
    return _fn("aaf_kv_import_host_chunked")(pool, src_host, desc, staging, staging_bytes, chunk_tokens, out_ctx, stream)
def aaf_kv_evict_to_budget(pool, alpha, beta, gamma, budget, out_victims, cap, n_victims, stream):
    return _fn("aaf_kv_evict_to_budget")(pool, alpha, beta, gamma, budget, out_victims, cap, n_victims, stream)
def aaf_kv_catalog_rows(pool, n_states, n_rows): return _fn("aaf_kv_catalog_rows")(pool, n_states, n_rows)
def aaf_kv_export_catalog(pool, cols, stream): return _fn("aaf_kv_export_catalog")(pool, cols, stream)
def aaf_kv_get_catalog(pool, clock, reuse, last): return _fn("aaf_kv_get_catalog")(pool, clock, reuse, last)
def aaf_kv_ctx_len(pool, ctx, out): return _fn("aaf_kv_ctx_len")(pool, ctx, out)
def aaf_kv_get_table(pool, ctx, out, cap, n_blocks): return _fn("aaf_kv_get_table")(pool, ctx, out, cap, n_blocks)
def aaf_kv_get_refcounts(pool, out): return _fn("aaf_kv_get_refcounts")(pool, out)
def aaf_kv_get_free_list(pool, out, n_free): return _fn("aaf_kv_get_free_list")(pool, out, n_free)
def aaf_kv_pool_stats(pool, out): return _fn("aaf_kv_pool_stats")(pool, out)
def aaf_kv_sync_status(pool): return _fn("aaf_kv_sync_status")(pool)
def aaf_kv_set_copy_engine(pool, engine): return _fn("aaf_kv_set_copy_engine")(pool, engine)
def aaf_kv_set_timing(pool, enable): return _fn("aaf_kv_set_timing")(pool, enable)
def aaf_kv_materialize_noalloc(pool_base, layer_stride, n_layers, n_kv_heads, head_dim, block_size, elt_bytes, n_blocks,
                               block_table_host, n_table_blocks, t0, t1, dst, dst_bytes, stream):
    """Gather without any allocation (see include/aaf_kv.h): for callers that may not call cudaMalloc.
    block_table_host is a ctypes int32 array / pointer in host memory."""
    return _fn("aaf_kv_materialize_noalloc")(pool_base, layer_stride, n_layers, n_kv_heads, head_dim, block_size,
                                             elt_bytes, n_blocks, block_table_host, n_table_blocks, t0, t1, dst,
                                             dst_bytes, stream)
def aaf_kv_state_bytes(n_layers, n_kv_heads, head_dim, elt_bytes, n_tokens):
    return _fn("aaf_kv_state_bytes")(n_layers, n_kv_heads, head_dim, elt_bytes, n_tokens)
def aaf_kv_transfer_time(kv_bytes, bandwidth, latency): return _fn("aaf_kv_transfer_time")(kv_bytes, bandwidth, latency)
def aaf_kv_transfer_time_packed(kv_bytes, bandwidth, latency, pack_rate):
    return _fn("aaf_kv_transfer_time_packed")(kv_bytes, bandwidth, latency, pack_rate)
def aaf_kv_policy(local_and_compatible, t_transfer, t_prefill):
    return _fn("aaf_kv_policy")(1 if local_and_compatible else 0, t_transfer, t_prefill)
def aaf_kv_debug_expire_wait(pool, limit_cycles, stream): return _fn("aaf_kv_debug_expire_wait")(pool, limit_cycles, stream)
def aaf_kv_debug_mark_unusable(pool): return _fn("aaf_kv_debug_mark_unusable")(pool)
def aaf_kv_strerror(status): return _fn("aaf_kv_strerror")(status).decode()


def make_desc(n_layers, n_kv_heads, head_dim, block_size, elt_bytes, n_blocks, max_ctx, max_blocks_per_ctx,
              max_batch=0, device=0, model_id=0, config_hash=0) -> aaf_kv_pool_desc:
    d = aaf_kv_pool_desc()
    d.struct_size = C.sizeof(aaf_kv_pool_desc)
    d.abi_version = AAF_KV_ABI_VERSION
    d.n_layers, d.n_kv_heads, d.head_dim, d.block_size, d.elt_bytes = n_layers, n_kv_heads, head_dim, block_size, elt_bytes
    d.n_blocks, d.max_ctx, d.max_blocks_per_ctx, d.max_batch, d.device = n_blocks, max_ctx, max_blocks_per_ctx, max_batch, device
    d.model_id, d.config_hash = model_id, config_hash
    return d


class KVPool:
    """Holds the torch-allocated memory of one pool and forwards to the C ABI.

    Methods return (status, result); nothing is computed on the Python side.
    """

    def __init__(self, n_layers, n_kv_heads, head_dim, block_size, elt_bytes, n_blocks, max_ctx,
                 max_blocks_per_ctx, free_order=None, max_batch=0, device=0, model_id=1, config_hash=1,
                 pool_tensor=None):
        import numpy as np
        import torch

        self.torch = torch
        self.device = torch.device("cuda", device)
        self.L, self.H, self.D, self.BS, self.E, self.NB = n_layers, n_kv_heads, head_dim, block_size, elt_bytes, n_blocks
        self.max_ctx, self.max_blk = max_ctx, max_blocks_per_ctx
        self.row = n_kv_heads * head_dim * elt_bytes
        self.run = block_size * self.row
        self.bpt = 2 * n_layers * self.row
        self.layer_stride = n_blocks * 2 * self.run
        d = make_desc(n_layers, n_kv_heads, head_dim, block_size, elt_bytes, n_blocks, max_ctx, max_blocks_per_ctx,
                      max_batch, device, model_id, config_hash)
        ws_bytes = aaf_kv_pool_workspace_bytes(d)
        if ws_bytes == 0:
            raise ValueError("invalid pool geometry")
        if pool_tensor is None:
            pool_tensor = torch.empty(n_layers * self.layer_stride, dtype=torch.uint8, device=self.device)
        assert pool_tensor.numel() * pool_tensor.element_size() >= n_layers * self.layer_stride
        self.pool = pool_tensor
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
        d.pool_base, d.layer_stride_bytes = self.pool.data_ptr(), self.layer_stride
        d.workspace, d.workspace_bytes = self.workspace.data_ptr(), ws_bytes
        self._fo = None
        if free_order is not None:
            self._fo = np.ascontiguousarray(np.asarray(free_order, dtype=np.int32))
            d.free_order = self._fo.ctypes.data_as(_p32)
        self.desc = d
        self.h = C.c_void_p()
        st = aaf_kv_pool_create(d, self.h)
        if st != AAF_OK:
            raise RuntimeError(f"aaf_kv_pool_create failed: {aaf_kv_strerror(st)}")

    # ------------------------------------------------------------------ helpers
    def _stream(self):
        return C.c_void_p(self.torch.cuda.current_stream(self.device).cuda_stream)

    def xfer_desc(self, n_tokens, pos_start=0) -> aaf_kv_xfer_desc:
        x = aaf_kv_xfer_desc()
        x.model_id, x.config_hash = self.desc.model_id, self.desc.config_hash
        x.n_layers, x.n_kv_heads, x.head_dim, x.elt_bytes = self.L, self.H, self.D, self.E
        x.pos_start, x.n_tokens = pos_start, n_tokens
        return x

    def close(self):
        if getattr(self, "h", None) and self.h.value:
            aaf_kv_pool_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ operators
    def materialize(self, ctx, t0, t1, out=None):
        n = max(t1 - t0, 0)
        if out is None:
            out = self.torch.empty(max(n * self.bpt, 16), dtype=self.torch.uint8, device=self.device)
        xd = aaf_kv_xfer_desc()
        st = aaf_kv_materialize(self.h, ctx, t0, t1, out.data_ptr(), out.numel() * out.element_size(), C.byref(xd),
                                self._stream())
        return st, (out if st == AAF_OK else None)

    def imp(self, buf, n, desc=None):
        xd = desc if desc is not None else self.xfer_desc(n)
        out = C.c_int32(-1)
        st = aaf_kv_import(self.h, buf.data_ptr(), C.byref(xd), C.byref(out), self._stream())
        return st, (out.value if st == AAF_OK else None)

    def materialize_batch(self, ctxs, t0s, t1s, outs):
        """outs: one device tensor per entry.  Returns the status."""
        n = len(ctxs)
        a = (C.c_int32 * max(n, 1))(*ctxs)
        b0 = (C.c_int64 * max(n, 1))(*t0s)
        b1 = (C.c_int64 * max(n, 1))(*t1s)
        ptrs = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in outs])
        sizes = (C.c_size_t * max(n, 1))(*[t.numel() * t.element_size() for t in outs])
        return aaf_kv_materialize_batch(self.h, n, a, b0, b1, ptrs, sizes, None, self._stream())

    def import_batch(self, bufs, ns):
        """bufs: one device transfer buffer per entry, ns: its token count.  Returns (status, [handles])."""
        n = len(bufs)
        ptrs = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in bufs])
        descs = (aaf_kv_xfer_desc * max(n, 1))(*[self.xfer_desc(k) for k in ns])
        out = (C.c_int32 * max(n, 1))()
        st = aaf_kv_import_batch(self.h, n, ptrs, descs, out, self._stream())
        return st, (list(out[:n]) if st == AAF_OK else None)

    def fork(self, parent, k):
        out = (C.c_int32 * max(k, 1))()
        st = aaf_kv_fork(self.h, parent, k, out, self._stream())
        return st, (list(out[:k]) if st == AAF_OK else None)

    def append(self, ctxs, n_new, bufs):
        n = len(ctxs)
        a = (C.c_int32 * max(n, 1))(*ctxs)
        b = (C.c_int32 * max(n, 1))(*n_new)
        ptrs = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in bufs])
        return aaf_kv_append(self.h, n, a, b, ptrs, self._stream()), None

    def append_host(self, ctxs, n_new, host_bufs, staging):
        """host_bufs: one (pinned) host tensor per entry; staging: device scratch for all of them."""
        n = len(ctxs)
        a = (C.c_int32 * max(n, 1))(*ctxs)
        b = (C.c_int32 * max(n, 1))(*n_new)
        ptrs = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in host_bufs])
        return aaf_kv_append_host(self.h, n, a, b, ptrs, staging.data_ptr(), staging.numel() * staging.element_size(),
                                  self._stream())

    def compose(self, segs, flags=0):
        m = len(segs)
        a = (C.c_int32 * max(m, 1))(*segs)
        out = C.c_int32(-1)
        st = aaf_kv_compose(self.h, m, a, flags, C.byref(out), self._stream())
        return st, (out.value if st == AAF_OK else None)

    def compose_batch(self, seg_lists, flags=0):
        """seg_lists: one list of segment handles per merge; returns (status, [result handles])."""
        n_out = len(seg_lists)
        offs, flat = [0], []
        for segs in seg_lists:
            flat += list(segs)
            offs.append(len(flat))
        a = (C.c_int32 * (n_out + 1))(*offs)
        b = (C.c_int32 * max(len(flat), 1))(*flat)
        out = (C.c_int32 * max(n_out, 1))()
        st = aaf_kv_compose_batch(self.h, n_out, a, b, flags, out, self._stream())
        return st, (list(out[:n_out]) if st == AAF_OK else None)

    def evict(self, ctxs):
        n = len(ctxs)
        a = (C.c_int32 * max(n, 1))(*ctxs)
        return aaf_kv_evict(self.h, n, a, self._stream()), None

    def materialize_host(self, ctx, t0, t1, dst_host, staging):
        return aaf_kv_materialize_host(self.h, ctx, t0, t1, dst_host.data_ptr(),
                                       dst_host.numel() * dst_host.element_size(), staging.data_ptr(),
                                       staging.numel() * staging.element_size(), None, self._stream())

    def import_host(self, src_host, n, staging):
        xd = self.xfer_desc(n)
        out = C.c_int32(-1)
        st = aaf_kv_import_host(self.h, src_host.data_ptr(), C.byref(xd), staging.data_ptr(),
                                staging.numel() * staging.element_size(), C.byref(out), self._stream())
        return st, (out.value if st == AAF_OK else None)

    def evict_to_budget(self, alpha, beta, gamma, budget_blocks):
        out = (C.c_int32 * self.max_ctx)()
        nv = C.c_int32(0)
        st = aaf_kv_evict_to_budget(self.h, alpha, beta, gamma, budget_blocks, out, self.max_ctx, C.byref(nv),
                                    self._stream())
        return st, (list(out[: nv.value]) if st == AAF_OK else None)

    def catalog(self):
        import numpy as np

        clock = C.c_int64(0)
        reuse = np.empty(self.max_ctx, dtype=np.int64)
        last = np.empty(self.max_ctx, dtype=np.int64)
        st = aaf_kv_get_catalog(self.h, C.byref(clock), reuse.ctypes.data_as(C.POINTER(C.c_int64)),
                                last.ctypes.data_as(C.POINTER(C.c_int64)))
        if st != AAF_OK:
            raise RuntimeError(aaf_kv_strerror(st))
        return {"clock": clock.value, "reuse": reuse.tolist(), "last_access": last.tolist()}

    def export_catalog(self) -> dict:
        """Runs the columnar export into torch-allocated device buffers; returns the columns as torch tensors
        (still on the device) trimmed to their row counts."""
        torch = self.torch
        ns, nr = C.c_int32(0), C.c_int64(0)
        aaf_kv_catalog_rows(self.h, C.byref(ns), C.byref(nr))
        i32 = lambda n: torch.empty(max(n, 1), dtype=torch.int32, device=self.device)
        i64 = lambda n: torch.empty(max(n, 1), dtype=torch.int64, device=self.device)
        t = {"state_id": i32(ns.value), "n_tokens": i64(ns.value), "reuse": i64(ns.value), "last_access": i64(ns.value),
             "origin": i32(ns.value), "parent": i32(ns.value), "born": i64(ns.value), "parent_born": i64(ns.value),
             "block_offsets": i32(ns.value + 1), "block_id": i32(nr.value), "pos_begin": i64(nr.value),
             "pos_end": i64(nr.value), "refcount": i32(nr.value), "address": i64(nr.value)}
        cols = aaf_kv_catalog_cols(**{k: v.data_ptr() for k, v in t.items()})
        st = aaf_kv_export_catalog(self.h, C.byref(cols), self._stream())
        if st != AAF_OK:
            raise RuntimeError(aaf_kv_strerror(st))
        n_of = lambda k: ns.value + 1 if k == "block_offsets" else (
            ns.value if k in ("state_id", "n_tokens", "reuse", "last_access", "origin", "parent", "born",
                              "parent_born") else nr.value)
        return {k: v[: n_of(k)] for k, v in t.items()}

    def materialize_host_chunked(self, ctx, t0, t1, dst_host, staging, chunk_tokens, flags=None):
        """flags: pinned torch int32 tensor receiving one completion flag per chunk (or None)."""
        nch = C.c_int32(0)
        fptr = C.cast(flags.data_ptr(), C.POINTER(C.c_uint32)) if flags is not None else None
        st = aaf_kv_materialize_host_chunked(self.h, ctx, t0, t1, dst_host.data_ptr(),
                                             dst_host.numel() * dst_host.element_size(), staging.data_ptr(),
                                             staging.numel() * staging.element_size(), chunk_tokens, fptr,
                                             flags.numel() if flags is not None else 0, C.byref(nch), None,
                                             self._stream())
        return st, nch.value

    def import_host_chunked(self, src_host, n, staging, chunk_tokens):
        xd = self.xfer_desc(n)
        out = C.c_int32(-1)
        st = aaf_kv_import_host_chunked(self.h, src_host.data_ptr(), C.byref(xd), staging.data_ptr(),
                                        staging.numel() * staging.element_size(), chunk_tokens, C.byref(out),
                                        self._stream())
        return st, (out.value if st == AAF_OK else None)

    # ------------------------------------------------------------------ introspection
    def ctx_len(self, ctx):
        v = C.c_int64(-1)
        return v.value if aaf_kv_ctx_len(self.h, ctx, C.byref(v)) == AAF_OK else None

    def table(self, ctx):
        import numpy as np

        out = np.empty(self.max_blk, dtype=np.int32)
        nb = C.c_int32(0)
        st = aaf_kv_get_table(self.h, ctx, out.ctypes.data_as(_p32), self.max_blk, C.byref(nb))
        if st != AAF_OK:
            raise RuntimeError(aaf_kv_strerror(st))
        return out[: nb.value].copy()

    def refcounts(self):
        import numpy as np

        out = np.empty(self.NB, dtype=np.int32)
        st = aaf_kv_get_refcounts(self.h, out.ctypes.data_as(_p32))
        if st != AAF_OK:
            raise RuntimeError(aaf_kv_strerror(st))
        return out

    def free_list(self):
        import numpy as np

        out = np.empty(self.NB, dtype=np.int32)
        nf = C.c_int32(0)
        st = aaf_kv_get_free_list(self.h, out.ctypes.data_as(_p32), C.byref(nf))
        if st != AAF_OK:
            raise RuntimeError(aaf_kv_strerror(st))
        return out[: nf.value].copy()

    def live_ctxs(self):
        return [c for c in range(self.max_ctx) if self.ctx_len(c) is not None]

    def stats(self) -> dict:
        s = aaf_kv_stats()
        st = aaf_kv_pool_stats(self.h, C.byref(s))
        if st != AAF_OK:
            raise RuntimeError(aaf_kv_strerror(st))
        d = {k: getattr(s, k) for k in ("free_blocks", "live_blocks", "peak_live_blocks", "live_ctx", "cow_count",
                                        "payload_bytes", "meta_launches")}
        d["copy_launches"] = dict(zip(OP_NAMES, list(s.copy_launches)))
        d["copy_ms"] = dict(zip(OP_NAMES, list(s.copy_ms)))
        d["timed_launches"] = dict(zip(OP_NAMES, list(s.timed_launches)))
        return d

    def sync_status(self):
        return aaf_kv_sync_status(self.h)

    def set_copy_engine(self, engine):
        return aaf_kv_set_copy_engine(self.h, engine)

    def set_timing(self, enable):
        return aaf_kv_set_timing(self.h, 1 if enable else 0)
