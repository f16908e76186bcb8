/*
 * aaf_kv.h -- C ABI of the B200 paged-KV operator library (libaafkv.so).
 *
 * The library implements the block-granular data movement behind the stateful KV
 * operators of AAFLOW+ (arxiv 2607.10987): a paged KV pool whose contexts are block
 * tables, with a device-resident free ring and reference-count table, and copy
 * kernels for every path that moves KV bytes.
 *
 * Geometry and layouts (all sizes in bytes unless noted)
 *   row   = n_kv_heads * head_dim * elt_bytes     one token, one layer, K or V
 *   run   = block_size * row                      one block, one layer, K or V
 *   bpt   = 2 * n_layers * row                    one token, all layers, K and V
 *   pool  : device memory, layer l at pool_base + l * layer_stride_bytes, each layer
 *           laid out [n_blocks][2 (K,V)][block_size][n_kv_heads][head_dim]; one block id
 *           names the same slot range in every layer (Sec. 3.2: blocks b_j = (K_j, V_j,
 *           layer, position range, device); Sec. 5.3: fixed-size block partitioning)
 *   transfer buffer : dense [n_layers][2][n_tokens][n_kv_heads][head_dim], no header; the
 *           metadata travels separately in an aaf_kv_xfer_desc (Sec. 5.4: raw tensor
 *           buffers, metadata descriptors sent apart)
 *   context: a block table (int32 block ids) plus a token count; token p lives in block
 *           table[p / block_size], slot p % block_size (Sec. 5.3: the mapping
 *           (state_id, block_id) -> (device, address))
 *   refcount[b] = number of block-table entries that name block b (App. A.2, metadata
 *           catalog: "refcount"); 0 <=> b is on the free ring
 *
 * Conventions the paper leaves open (stated so that results are reproducible):
 *   allocation takes the oldest entries of the FIFO free ring in order; a block whose
 *   refcount reaches 0 is pushed at the ring's tail, in (context, table position) order
 *   of the evicting call; a new context gets the smallest free handle; no operator
 *   writes a slot outside the tokens it stores; a failing call changes no state.
 *
 * Ownership: the caller owns ALL device memory (pool, workspace, transfer buffers) and
 * keeps it valid while the pool object lives / until the stream has run the call.  The
 * library allocates host memory only (the pool object, a pinned argument ring, events).
 *
 * Ordering: calls on one pool are applied in call order and must be issued to one stream
 * (or the caller orders streams itself; the library additionally makes the copy launches of a pool
 * run one after the other when consecutive calls name different streams, because they share a work
 * counter in the pool's control block).  Data calls are asynchronous.  Every kernel that
 * touches payload bytes (pool rows, transfer buffers) runs on the `stream` argument, so the
 * caller's own work on that stream is ordered against them as usual.  Kernels that touch only
 * the library's metadata (block tables, reference counts, the ring, copy descriptors) run on a
 * library-owned stream that the library orders against `stream` with events; metadata is
 * visible only through the introspection calls, which synchronise both.  Not thread-safe
 * per pool.  Pointers marked (device) must be device pointers, 16-byte aligned; row must
 * be a multiple of 16.  Pointers marked (host) are ordinary host pointers read or
 * written before the call returns.
 *
 * Errors: every call returns 0 (AAF_OK) or a negative aaf_status.  Everything the host
 * can know is checked before anything is launched, so an error return means no state
 * changed -- with one exception: AAF_ERR_CUDA from an operator means that a CUDA runtime
 * call failed, possibly after a metadata kernel had already been enqueued, so the host's
 * view of the pool can no longer be trusted.  The pool is then unusable: every later
 * operator call on it returns AAF_ERR_CUDA, and the only useful call left is
 * aaf_kv_pool_destroy.  Conditions only the device can see (a corrupted ring or
 * reference count, a bounded wait that gave up) never trap: they set a sticky status
 * word that aaf_kv_sync_status returns and clears.
 */
#ifndef AAF_KV_H
#define AAF_KV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AAF_KV_ABI_VERSION 1u

typedef enum aaf_status {
    AAF_OK = 0,
    AAF_ERR_INVALID_ARG = -1,   /* null / misaligned pointer, bad range, k < 1, duplicate ctx in a batch ... */
    AAF_ERR_BAD_CTX = -2,       /* handle is not a live context                                             */
    AAF_ERR_OOM_BLOCKS = -3,    /* not enough free blocks (exact: decided against the device's free count)  */
    AAF_ERR_OOM_CTX = -4,       /* no free context handle                                                   */
    AAF_ERR_TOO_LONG = -5,      /* result would exceed max_blocks_per_ctx                                   */
    AAF_ERR_INCOMPAT = -6,      /* descriptor does not match the pool (Compat predicate, Sec. 3.2)          */
    AAF_ERR_DST_TOO_SMALL = -7,
    AAF_ERR_CUDA = -8,          /* a CUDA runtime call failed (no usable device, launch error ...)          */
    AAF_ERR_CORRUPT = -9,       /* device found the ring / a reference count inconsistent                   */
    AAF_ERR_TIMEOUT = -10,      /* a bounded device-side wait gave up                                       */
    AAF_ERR_TOO_MANY = -11,     /* batch larger than max_batch                                              */
    AAF_ERR_SCRATCH_LIMIT = -12 /* request larger than the built-in scratch of aaf_kv_materialize_noalloc   */
} aaf_status;

typedef struct aaf_kv_pool aaf_kv_pool; /* opaque host object */
typedef int32_t aaf_ctx_t;              /* context handle: slot index >= 0 */

/* M and Theta of the KV state object S_KV = (M, Theta, B, Pi, Lambda, Gamma) (Sec. 3.2), the
 * pool geometry, capacities and the caller-owned memory the pool lives in. */
typedef struct aaf_kv_pool_desc {
    uint32_t struct_size;        /* sizeof(aaf_kv_pool_desc)                                  */
    uint32_t abi_version;        /* AAF_KV_ABI_VERSION                                        */
    int32_t n_layers, n_kv_heads, head_dim, block_size, elt_bytes;
    int32_t n_blocks;            /* blocks per layer in the pool                              */
    int32_t max_ctx;             /* context handles 0 .. max_ctx-1                            */
    int32_t max_blocks_per_ctx;  /* longest block table                                       */
    int32_t max_batch;           /* largest n / m / k of a batched call (0 -> 1024)           */
    int32_t device;              /* CUDA device ordinal that owns pool_base and workspace     */
    void *pool_base;             /* (device) >= n_layers * layer_stride_bytes bytes           */
    size_t layer_stride_bytes;   /* >= n_blocks * 2 * run, multiple of 16                     */
    void *workspace;             /* (device) >= aaf_kv_pool_workspace_bytes(desc) bytes, 256-byte aligned */
    size_t workspace_bytes;
    const int32_t *free_order;   /* (host) permutation of [0, n_blocks) = initial ring, or NULL = identity */
    uint64_t model_id;           /* M      : compared by the Compat predicate                 */
    uint64_t config_hash;        /* Theta  : compared by the Compat predicate                 */
} aaf_kv_pool_desc;

/* Stand-in for the metadata descriptor that travels beside a transfer buffer (Sec. 5.4; Alg.
 * "KV-Transfer": the descriptor is sent, then the raw buffers).  Host memory. */
typedef struct aaf_kv_xfer_desc {
    uint64_t model_id, config_hash;
    int32_t n_layers, n_kv_heads, head_dim, elt_bytes;
    int64_t pos_start;           /* Pi: position of the buffer's first token in its source context */
    int64_t n_tokens;
} aaf_kv_xfer_desc;

#define AAF_COMPOSE_SHARE 0u     /* aligned segments share their full blocks by reference        */
#define AAF_COMPOSE_COPY_ALL 1u  /* merge policy mu that forbids aliasing: everything is copied  */

/* copy engines (aaf_kv_set_copy_engine) */
#define AAF_ENGINE_AUTO 0        /* the library picks                                                     */
#define AAF_ENGINE_VEC 1         /* 16-byte vector loads/stores through registers                         */
#define AAF_ENGINE_BULK 2        /* cp.async.bulk global->shared->global with mbarrier completion         */
#define AAF_ENGINE_WARP 3        /* 16-byte vector copies scheduled per warp (best for small / ragged pieces) */

/* operator classes that move payload (index into the per-class arrays of aaf_kv_stats) */
#define AAF_OP_MATERIALIZE 0
#define AAF_OP_IMPORT 1
#define AAF_OP_APPEND 2
#define AAF_OP_COMPOSE 3
#define AAF_OP_CLASSES 4

typedef struct aaf_kv_stats {
    int64_t free_blocks, live_blocks;
    int64_t peak_live_blocks;              /* Mem_KV = max_t sum ||KV_i(t)|| in blocks (Sec. 6.2)          */
    int64_t live_ctx;
    int64_t cow_count;                     /* partial tail blocks copied on write so far                   */
    int64_t payload_bytes;                 /* bytes read (= bytes written) by the copy kernels so far      */
    int64_t copy_launches[AAF_OP_CLASSES]; /* copy-kernel launches per operator class                      */
    int64_t meta_launches;                 /* metadata (plan / fork / evict) kernel launches               */
    double copy_ms[AAF_OP_CLASSES];        /* device time of the copy kernels per class, CUDA events on the
                                              launching stream; only accumulated while timing is enabled   */
    int64_t timed_launches[AAF_OP_CLASSES];
} aaf_kv_stats;

/* Workspace size for a geometry (pool_base / workspace / free_order fields are ignored).
 * Returns 0 if the descriptor is invalid. */
size_t aaf_kv_pool_workspace_bytes(const aaf_kv_pool_desc *desc);

/* Pool creation: all reference counts 0, free ring = free_order, no context.  Writes the
 * workspace on the device (synchronous).  The pool bytes themselves are not touched.
 * Errors: INVALID_ARG (bad geometry, row not a multiple of 16, misaligned pointers, workspace
 * too small, free_order not a permutation), CUDA. */
int aaf_kv_pool_create(const aaf_kv_pool_desc *desc, aaf_kv_pool **out);
int aaf_kv_pool_destroy(aaf_kv_pool *pool);

/* materialize -- Alg. "KV-Transfer" (select the blocks of a position range, hand raw buffers to
 * the transport), Sec. 5.4 (block granularity, prefix subsets).  Gathers tokens
 * [tok_begin, tok_end) of ctx through its block table into the dense transfer buffer
 * dst_dev (device, >= (tok_end - tok_begin) * bpt bytes): dst[l][kv][t - tok_begin] =
 * pool[l][table[t / BS]][kv][t % BS].  Pure read of the pool.  out_desc (host, may be NULL)
 * receives the descriptor.  Errors: BAD_CTX, INVALID_ARG (range, pointer), DST_TOO_SMALL. */
int aaf_kv_materialize(aaf_kv_pool *pool, aaf_ctx_t ctx, int64_t tok_begin, int64_t tok_end, void *dst_dev,
                       size_t dst_bytes, aaf_kv_xfer_desc *out_desc, void *stream);

/* import -- Alg. "KV-Materialize" steps 4-6 (partition layer-wise K/V into blocks, register them)
 * and Alg. "KV-Transfer" (register received blocks).  Scatters the desc->n_tokens tokens of
 * src_dev (device) into ceil(n / BS) blocks taken from the free ring in order, each with
 * refcount 1; *out_ctx (host) receives the new handle.  Only the slots of stored tokens are
 * written.  Errors: INCOMPAT, INVALID_ARG, TOO_LONG, OOM_CTX, OOM_BLOCKS. */
int aaf_kv_import(aaf_kv_pool *pool, const void *src_dev, const aaf_kv_xfer_desc *desc, aaf_ctx_t *out_ctx,
                  void *stream);

/* materialize / import, batched -- n independent transfers packed (unpacked) by one planner launch and ONE copy
 * launch (Alg. "KV-Transfer": block selection by position range for several states at once; Sec. 5.4: only the
 * subset a consumer needs is sent, so transfers are often short suffixes, whose copies are too small to reach the
 * HBM rate one launch each).  When it succeeds the result is exactly that of the for-loop over i of
 * aaf_kv_materialize(ctxs[i], tok_begin[i], tok_end[i], dst_dev[i], dst_bytes[i]) or of
 * aaf_kv_import(src_dev[i], &descs[i]): the same handles (the n smallest free ones, in order), the same blocks
 * (import i takes its blocks behind those of the imports before it), the same catalog stamps.  A context may
 * appear in several entries of a materialize batch; destination buffers must not overlap.  All-or-nothing.
 * All arrays are host arrays of n entries; out_descs may be NULL.  Errors: as the single forms, OOM_CTX /
 * OOM_BLOCKS / TOO_MANY counted over the whole batch. */
int aaf_kv_materialize_batch(aaf_kv_pool *pool, int32_t n, const aaf_ctx_t *ctxs, const int64_t *tok_begin,
                             const int64_t *tok_end, void *const *dst_dev, const size_t *dst_bytes,
                             aaf_kv_xfer_desc *out_descs, void *stream);
int aaf_kv_import_batch(aaf_kv_pool *pool, int32_t n, const void *const *src_dev, const aaf_kv_xfer_desc *descs,
                        aaf_ctx_t *out_ctxs, void *stream);

/* fork -- Alg. "KV-Fork": k children alias the parent's blocks (table copied, refcount += 1 per
 * entry per child); nothing is copied, no block allocated (Sec. 3.3).  out_children (host, k
 * entries) receives the k smallest free handles in order.  Errors: BAD_CTX, INVALID_ARG, OOM_CTX,
 * TOO_MANY. */
int aaf_kv_fork(aaf_kv_pool *pool, aaf_ctx_t parent, int32_t k, aaf_ctx_t *out_children, void *stream);

/* append -- Alg. "KV-Resume" (register continuation KV) with copy-on-write on divergence
 * (Sec. 3.3; App. A.2).  For i < n: context ctxs[i] grows by n_new[i] tokens read from
 * src_dev[i] (device, transfer layout [L][2][n_new[i]][H][D]).  If the context's partial tail
 * block is shared, its valid rows are first copied into a fresh block and the old one is
 * released.  The batch equals the for-loop over i; it is all-or-nothing.  ctxs, n_new, src_dev
 * are host arrays.  Errors: BAD_CTX, INVALID_ARG (n_new < 1, duplicate ctx), TOO_LONG,
 * OOM_BLOCKS, TOO_MANY. */
int aaf_kv_append(aaf_kv_pool *pool, int32_t n, const aaf_ctx_t *ctxs, const int32_t *n_new,
                  const void *const *src_dev, void *stream);

/* compose -- Alg. "Restricted-KV-Merge", concatenation branch (Sec. 4.5): the new context is
 * segs[0] || segs[1] || ... || segs[m-1], bytes verbatim.  A segment that starts on a block
 * boundary shares its full blocks (and, if it is the last one, its partial tail) by reference;
 * everything behind the first partial tail is re-packed into fresh blocks.  With
 * AAF_COMPOSE_COPY_ALL nothing is shared.  Sources stay live; repeats allowed.  segs is a host
 * array; *out_ctx (host).  Errors: BAD_CTX, INVALID_ARG, TOO_LONG, OOM_CTX, OOM_BLOCKS, TOO_MANY. */
int aaf_kv_compose(aaf_kv_pool *pool, int32_t m, const aaf_ctx_t *segs, uint32_t flags, aaf_ctx_t *out_ctx,
                   void *stream);

/* compose, batched -- n_out independent merges (Alg. "Restricted-KV-Merge", concatenation branch) in one call:
 * merge i concatenates segs[seg_off[i] .. seg_off[i + 1]) (seg_off has n_out + 1 entries, seg_off[0] = 0, every
 * merge at least one segment).  When it succeeds the result is exactly that of the for-loop of aaf_kv_compose
 * over i -- the same handles (the n_out smallest free ones, in order), the same block tables (each merge takes its
 * fresh blocks behind those of the merges before it), the same catalog stamps -- but with one planner launch and
 * ONE copy launch for all merges, so that a level of small merges (the agents of a workflow merged in pairs)
 * does not pay the launch ramp per merge.  Segments must be live before the call (a result of the same batch
 * cannot be a segment).  The batch is all-or-nothing: any error leaves every merge undone.  seg_off, segs host;
 * out_ctxs (host, n_out entries).  Errors: as aaf_kv_compose; OOM_CTX / OOM_BLOCKS / TOO_MANY count the whole batch. */
int aaf_kv_compose_batch(aaf_kv_pool *pool, int32_t n_out, const int32_t *seg_off, const aaf_ctx_t *segs,
                         uint32_t flags, aaf_ctx_t *out_ctxs, void *stream);

/* evict -- Alg. "KV-Evict", release step: every block-table entry of every listed context drops
 * one reference; blocks that reach 0 return to the ring's tail in (context, table position)
 * order; the handles become free.  Victim selection is the caller's policy.  ctxs is a host
 * array.  Errors: BAD_CTX, INVALID_ARG (duplicate), TOO_MANY. */
int aaf_kv_evict(aaf_kv_pool *pool, int32_t n, const aaf_ctx_t *ctxs, void *stream);

/* evict to a budget -- Alg. "KV-Evict", the whole loop, selected on the device.  For every live
 * context score(S) = alpha * reuse(S) - beta * size(S) - gamma * age(S): reuse = number of times S
 * was read by materialize, fork or compose (per occurrence); size = its block-table length; age =
 * logical clock of this call - clock of the last call that read, wrote or created S (the clock counts
 * successful state-touching calls).  Scores are taken once, in double precision, one rounding per
 * operation.  While the live blocks (n_blocks - free) exceed budget_blocks, the context with the
 * lowest score (ties: smallest handle) is evicted by the release rule of aaf_kv_evict.  Shared
 * blocks survive while another context references them.  out_victims (host, cap >= number of live
 * contexts) receives the evicted handles in order, *n_victims their count.  The call waits for the
 * metadata kernels issued so far, not for copies still running on `stream` (the host needs the victims).  alpha = beta = 0, gamma > 0 is LRU.
 * Errors: INVALID_ARG (negative budget, non-finite weight, cap too small), CUDA. */
int aaf_kv_evict_to_budget(aaf_kv_pool *pool, double alpha, double beta, double gamma, int64_t budget_blocks,
                           aaf_ctx_t *out_victims, int32_t cap, int32_t *n_victims, void *stream);

/* Host-buffer forms of the transfer pack / unpack (the device end of Sec. 5.4's transport when
 * the peer is host memory).  staging_dev (device, >= n * bpt bytes) is caller-owned scratch.
 * materialize_host gathers into staging_dev and copies it to dst_host; import_host copies
 * src_host to staging_dev and scatters it.  Both enqueue on `stream`; host buffers must stay
 * valid until the stream has run the call (use pinned memory for asynchronous copies). */
int aaf_kv_materialize_host(aaf_kv_pool *pool, aaf_ctx_t ctx, int64_t tok_begin, int64_t tok_end, void *dst_host,
                            size_t dst_bytes, void *staging_dev, size_t staging_bytes, aaf_kv_xfer_desc *out_desc,
                            void *stream);
int aaf_kv_import_host(aaf_kv_pool *pool, const void *src_host, const aaf_kv_xfer_desc *desc, void *staging_dev,
                       size_t staging_bytes, aaf_ctx_t *out_ctx, void *stream);

/* append with the continuation tokens in HOST memory -- Alg. "KV-Resume" (register continuation KV)
 * fed from the transport's host end (Sec. 5.4).  Same result as aaf_kv_append, but src_host[i] (host,
 * transfer layout [L][2][n_new[i]][H][D]; pinned memory for a truly asynchronous copy) is first
 * uploaded into staging_dev (device, caller-owned scratch, >= sum(n_new) * bpt bytes, 16-byte
 * aligned), entry after entry, on a library-owned copy stream; the scatter on `stream` waits for the
 * upload.  The upload does NOT wait for work already queued on `stream`, except for the scatter of
 * the previous aaf_kv_append_host of this pool: staging_dev must be scratch that nothing else has in
 * use, so that the upload can overlap whatever `stream` is still doing (e.g. a transfer buffer on its
 * way back to the host).  Host buffers and staging_dev must stay untouched until `stream` has run
 * the call.  Errors as aaf_kv_append, plus DST_TOO_SMALL for a staging buffer that is too small;
 * after an error the contents of staging_dev are undefined. */
int aaf_kv_append_host(aaf_kv_pool *pool, int32_t n, const aaf_ctx_t *ctxs, const int32_t *n_new,
                       const void *const *src_host, void *staging_dev, size_t staging_bytes, void *stream);

/* Chunked, overlapped forms of the host transfer (Sec. 5.4: the transport overlaps communication
 * with computation, and consumers may start as blocks arrive).  The token range is cut into chunks
 * of chunk_tokens tokens (a multiple of block_size, counted from the block that holds tok_begin);
 * while one chunk crosses PCIe on a library-owned copy stream, the kernel for the next chunk runs on
 * `stream`.  Results are byte-identical to the unchunked forms.
 *   materialize: done_flags_host (host, pinned recommended, may be NULL; flags_cap entries) receives
 *   one completion flag per chunk: the library zeroes the flags, and flag c becomes 1, in stream
 *   order, after chunk c's bytes have landed in dst_host, so a consumer (a network sender) can poll
 *   and forward chunk c while later chunks are still being packed.  Chunk c covers the columns of
 *   blocks [c * chunk_tokens / BS, ...) of the range in every (layer, K/V) plane of dst_host.
 *   *n_chunks_out (host, may be NULL) receives the number of chunks.  `stream` is complete only
 *   when the last chunk has landed.
 *   import: blocks are allocated up front; chunk c is scattered as soon as it has arrived.  The upload
 *   runs on the library's upload stream (uploads of this pool arrive in call order) and does NOT wait for
 *   work already queued on `stream`, except for the scatter of the previous aaf_kv_import_host_chunked:
 *   staging_dev must be scratch that nothing else has in use.
 * Errors as for the unchunked forms, plus INVALID_ARG for a chunk_tokens that is not a positive
 * multiple of block_size and DST_TOO_SMALL for too few flags. */
int aaf_kv_materialize_host_chunked(aaf_kv_pool *pool, aaf_ctx_t ctx, int64_t tok_begin, int64_t tok_end,
                                    void *dst_host, size_t dst_bytes, void *staging_dev, size_t staging_bytes,
                                    int32_t chunk_tokens, uint32_t *done_flags_host, int32_t flags_cap,
                                    int32_t *n_chunks_out, aaf_kv_xfer_desc *out_desc, void *stream);
int aaf_kv_import_host_chunked(aaf_kv_pool *pool, const void *src_host, const aaf_kv_xfer_desc *desc,
                               void *staging_dev, size_t staging_bytes, int32_t chunk_tokens, aaf_ctx_t *out_ctx,
                               void *stream);

/* Introspection (metadata catalog of App. A.2).  These synchronise the library's metadata stream and
 * the stream of the most recent call. */
int aaf_kv_ctx_len(aaf_kv_pool *pool, aaf_ctx_t ctx, int64_t *n_tokens);
int aaf_kv_get_table(aaf_kv_pool *pool, aaf_ctx_t ctx, int32_t *host_out, int32_t cap, int32_t *n_blocks);
int aaf_kv_get_refcounts(aaf_kv_pool *pool, int32_t *host_out /* n_blocks entries */);
int aaf_kv_get_free_list(aaf_kv_pool *pool, int32_t *host_out /* n_blocks entries */, int32_t *n_free);
/* Columnar export of the metadata catalog (App. A.2, catalog fields; Sec. 5.3: metadata kept in a
 * columnar, zero-copy encoding).  All columns are DEVICE buffers the caller owns; they are written
 * by metadata kernels that `stream` is made to wait for, and are laid out like Arrow primitive arrays
 * and list offsets, so a consumer on `stream` can wrap them without conversion.
 *   state rows, one per live context in ascending handle order (capacity max_ctx):
 *     state_id int32, n_tokens int64, reuse int64, last_access int64,
 *     lineage (Lambda of Sec. 3.2): origin int32 (AAF_ORIGIN_*), parent int32 (the fork parent or the
 *     first merged segment, -1 for none), born int64 (clock of the creating call), parent_born int64
 *     (creation clock of that parent: handles are reused, (handle, born) names a state for good),
 *     block_offsets int32[n_states + 1]: list offsets into the block rows (exclusive prefix sum of
 *     the block-table lengths; capacity max_ctx + 1)
 *   block rows, one per block-table entry (capacity = n_block_rows of aaf_kv_catalog_rows):
 *     block_id int32, pos_begin / pos_end int64 (token range within the context), refcount int32,
 *     address int64 (byte offset of the block's layer-0 K run from pool_base; layer l and V follow
 *     by + l * layer_stride_bytes and + run).
 * model_id / config_hash (M, Theta) are pool-wide and live in the pool descriptor; device and owner
 * are the caller's tags.  aaf_kv_catalog_rows answers from the host mirror (no sync). */
#define AAF_ORIGIN_BUFFER 1 /* registered from a transfer buffer: prefill output or received state */
#define AAF_ORIGIN_FORK 2
#define AAF_ORIGIN_MERGE 3
typedef struct aaf_kv_catalog_cols {
    int32_t *state_id;
    int64_t *n_tokens, *reuse, *last_access;
    int32_t *origin, *parent;
    int64_t *born, *parent_born;
    int32_t *block_offsets;
    int32_t *block_id;
    int64_t *pos_begin, *pos_end;
    int32_t *refcount;
    int64_t *address;
} aaf_kv_catalog_cols;
int aaf_kv_catalog_rows(aaf_kv_pool *pool, int32_t *n_states, int64_t *n_block_rows);
int aaf_kv_export_catalog(aaf_kv_pool *pool, const aaf_kv_catalog_cols *cols_dev, void *stream);

/* Catalog counters per handle (max_ctx entries each; -1 for a free handle) and the logical clock. */
int aaf_kv_get_catalog(aaf_kv_pool *pool, int64_t *clock, int64_t *reuse_out, int64_t *last_access_out);
int aaf_kv_pool_stats(aaf_kv_pool *pool, aaf_kv_stats *out);
/* Returns the sticky device status (AAF_OK, AAF_ERR_CORRUPT or AAF_ERR_TIMEOUT) and clears it. */
int aaf_kv_sync_status(aaf_kv_pool *pool);

/* Tuning and measurement knobs. */
int aaf_kv_set_copy_engine(aaf_kv_pool *pool, int engine);  /* AAF_ENGINE_* */
int aaf_kv_set_timing(aaf_kv_pool *pool, int enable);       /* bracket copy kernels with CUDA events */

/* Cost model of the state path (host-only arithmetic; no device is touched, no pool is needed).
 *   aaf_kv_state_bytes   |KV| of n_tokens tokens: n_tokens * 2 * n_layers * n_kv_heads * head_dim * elt_bytes
 *                        (K and V blocks of every layer, Sec. 3.2); -1 if an argument is not positive or the
 *                        product overflows.
 *   aaf_kv_transfer_time T_transfer = |KV| / BW + delta (Sec. 5.4; Exp. 3: KV bytes / bandwidth + latency),
 *                        evaluated in double precision as one division and one addition, in that order.
 *                        Returns a NaN for kv_bytes < 0, bandwidth <= 0 or latency < 0.
 *   aaf_kv_transfer_time_packed  the same plus the term the paper's model leaves out: packing the state into
 *                        a transfer buffer at the sender and unpacking it at the receiver (aaf_kv_materialize /
 *                        aaf_kv_import), each moving 2 |KV| bytes (read + written) at pack_rate bytes per second
 *                        (read + written, as the library's benchmark reports it):
 *                        T = 2 |KV| / pack_rate + (|KV| / BW + delta) + 2 |KV| / pack_rate, summed left to right.
 *                        This is the un-overlapped upper bound; the chunked forms overlap packing with the wire.
 *   aaf_kv_policy        the scheduling rule pi(S) (Sec. 4.6; App. C; App. E step 5): AAF_POLICY_REUSE if the
 *                        state is local and compatible, else AAF_POLICY_TRANSFER iff t_transfer < t_prefill
 *                        (strictly), else AAF_POLICY_RECOMPUTE.  A NaN time compares false: recompute. */
#define AAF_POLICY_REUSE 0
#define AAF_POLICY_TRANSFER 1
#define AAF_POLICY_RECOMPUTE 2
int64_t aaf_kv_state_bytes(int32_t n_layers, int32_t n_kv_heads, int32_t head_dim, int32_t elt_bytes, int64_t n_tokens);
double aaf_kv_transfer_time(double kv_bytes, double bandwidth_bytes_per_s, double latency_s);
double aaf_kv_transfer_time_packed(double kv_bytes, double bandwidth_bytes_per_s, double latency_s,
                                   double pack_rate_bytes_per_s);
int aaf_kv_policy(int local_and_compatible, double t_transfer_s, double t_prefill_s);

/* Gather for callers that cannot allocate -- the paper has no counterpart; this is a library
 * convenience.  Same result as aaf_kv_materialize (dst[l][kv][t - tok_begin] =
 * pool[l][table[t / BS]][kv][t % BS] for t in [tok_begin, tok_end)), but it needs no pool object and
 * no workspace: the caller passes the pool memory and geometry as plain values and the context's
 * block table as a HOST array (n_table_blocks entries, e.g. from aaf_kv_get_table), and the scratch
 * the gather needs lives in a fixed array inside the library.  It is meant for callers that must
 * not call cudaMalloc: a process whose GPU memory is already fully committed to its own pool, a
 * latency-critical path that cannot take an allocation's device-wide synchronisation, or a plug-in
 * that is only ever handed pointers.  The call allocates nothing, on the device or in pinned host
 * memory, and frees nothing.
 *   - Limit: the token range may touch at most AAF_NOALLOC_MAX_BLOCKS blocks; a larger request
 *     returns AAF_ERR_SCRATCH_LIMIT and does nothing (split the range).
 *   - The first call on a device looks up the device address of the built-in array (with the
 *     calling thread's current device, which must be the one that owns the memory); make that
 *     first call before any stream capture begins.
 *   - All calls on a device share the one array, which keeps the previous call's contents; each
 *     call clears or overwrites what it reads.  Two calls that overlap on the GPU (different
 *     streams, or host threads racing) corrupt each other: keep them on one stream or order them.
 *   - pool_base_dev, dst_dev: memory of the current device, 16-byte aligned.  block_table_host: host
 *     memory; its entries are checked before the call returns and uploaded by an asynchronous copy on
 *     `stream`, so the array must stay unchanged until the stream has run the call (a pageable array
 *     happens to be read before return; a pinned one is not).
 * Errors: INVALID_ARG (pointers, memory of another device, geometry, range, a table entry outside
 * [0, n_blocks)), DST_TOO_SMALL, SCRATCH_LIMIT, CUDA. */
#define AAF_NOALLOC_MAX_BLOCKS 4096
int aaf_kv_materialize_noalloc(const void *pool_base_dev, size_t layer_stride_bytes, int32_t n_layers,
                               int32_t n_kv_heads, int32_t head_dim, int32_t block_size, int32_t elt_bytes,
                               int32_t n_blocks, const int32_t *block_table_host, int32_t n_table_blocks,
                               int64_t tok_begin, int64_t tok_end, void *dst_dev, size_t dst_bytes, void *stream);

/* Test hook for the failure path of the device-side waits (no paper counterpart).  Every wait in the
 * library's kernels is bounded: when its limit expires the kernel records AAF_ERR_TIMEOUT in the
 * sticky status word and returns, so the context stays usable.  This call launches a one-thread
 * kernel that waits, for at most limit_cycles SM clock cycles (1 .. 2^31), on a barrier nothing ever
 * signals, so that a test can watch the limit expire: aaf_kv_sync_status then returns
 * AAF_ERR_TIMEOUT once, and the pool keeps working.  Nothing faults, traps or hangs. */
int aaf_kv_debug_expire_wait(aaf_kv_pool *pool, uint64_t limit_cycles, void *stream);

/* Test hook for the error contract (no paper counterpart): puts the pool into the state that a CUDA runtime failure
 * inside an operator leaves it in, without any failure.  Every later operator call then returns AAF_ERR_CUDA and
 * changes nothing; introspection and aaf_kv_pool_destroy keep working. */
int aaf_kv_debug_mark_unusable(aaf_kv_pool *pool);

const char *aaf_kv_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* AAF_KV_H */
