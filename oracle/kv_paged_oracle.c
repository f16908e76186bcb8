/*
 * kv_paged_oracle.c -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
 *
 * A plain, sequential, single-threaded CPU model of the paged KV pool behind the
 * paper's stateful KV operators.  It exists only so that the CUDA library can be
 * checked against something that can be read and verified by eye.  Only the test
 * suite, the smoke check and the CPU-baseline leg of the benchmark may load it.
 * It shares no code with the CUDA library and never calls it.
 *
 * What it models (paper passages each function follows are cited at the function):
 *   - KV state B = {b_j}: fixed-size blocks of K and V rows (Sec. 3.2 "KV State
 *     Object"; Sec. 5.3 "KV-State Manager": fixed-size block partitioning).
 *   - mapping (state_id, block_id) -> address (Sec. 5.3): a per-context block table.
 *   - refcount = number of logical states sharing a block (metadata catalog table,
 *     App. A.2), kept here as "number of block-table entries that name the block".
 *
 * Physical conventions the paper leaves open (allocation order, free order, context
 * ids, share-vs-copy rule of the merge) are fixed as follows.  The paper cannot pin
 * them; they are pinned by two worked examples derived by hand from these rules
 * (tests/golden/worked_example_w1.txt and _w2.txt: tables, block contents, reference
 * counts and the order of the free list, including the order in which one evicting
 * call frees several blocks), while every materialised byte is pinned by the value
 * model (oracle/value_model.py) and the invariants in the tests:
 *   pool    : bytes [L][NB][2][BS][row], row = H*D*E bytes (one token, one layer, K or V)
 *   buffer  : transfer layout [L][2][n][row], dense, no header
 *   ring    : FIFO of free block ids; alloc takes ring[head++ mod NB],
 *             release pushes ring[tail++ mod NB] when a refcount reaches 0
 *   ctx ids : smallest free slot index
 *   an operator never writes a slot outside the tokens it stores
 *   a failing operator changes no state
 *
 * Every data copy below is one memcpy of one row (one token, one layer, K or V):
 * no blocking, no fusion, no reordering beyond the loops written out.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum {
    KVO_OK = 0,
    KVO_INVALID_ARG = -1,
    KVO_BAD_CTX = -2,
    KVO_OOM_BLOCKS = -3,
    KVO_OOM_CTX = -4,
    KVO_TOO_LONG = -5,
    KVO_DST_TOO_SMALL = -7
};

#define KVO_COMPOSE_COPY_ALL 1u

typedef struct kvo_pool {
    int32_t L, H, D, BS, E, NB, max_ctx, max_blk;
    int64_t row;          /* bytes of one row                         */
    uint8_t *pool;        /* [L][NB][2][BS][row]                      */
    int32_t *refcount;    /* [NB]                                     */
    int32_t *ring;        /* [NB] free ring                           */
    uint64_t head, tail;  /* free count = tail - head                 */
    int32_t *table;       /* [max_ctx][max_blk]                       */
    int64_t *len;         /* [max_ctx] tokens; -1 = slot is free      */
    int64_t *reuse;       /* [max_ctx] times the state was read by fork / materialize / compose   */
    int64_t *last_access; /* [max_ctx] logical clock of the last operator that used the state     */
    int64_t clock;        /* logical clock: number of successful state-touching operators so far  */
    /* lineage Lambda (Sec. 3.2: how a state was produced; App. A.2 catalog field "lineage") */
    int32_t *origin;      /* [max_ctx] 1 = registered from a buffer (prefill / transfer), 2 = fork, 3 = merge */
    int32_t *parent;      /* [max_ctx] handle the state descends from (fork parent, first merged segment), -1 = none */
    int64_t *born;        /* [max_ctx] clock of the operator that created the state               */
    int64_t *parent_born; /* [max_ctx] creation clock of that parent: (handle, born) names a state for good */
    int64_t peak_live;    /* max over time of NB - free (Mem_KV in blocks, Sec. 6.2) */
    int64_t cow_count;    /* copy-on-write events so far              */
    int64_t rows_copied;  /* rows moved by memcpy so far              */
} kvo_pool;

/* ---------------------------------------------------------------- helpers */

static int64_t nblk(const kvo_pool *p, int64_t tokens) { return (tokens + p->BS - 1) / p->BS; }
static int64_t free_blocks(const kvo_pool *p) { return (int64_t)(p->tail - p->head); }
static int32_t *tbl(const kvo_pool *p, int32_t c) { return p->table + (int64_t)c * p->max_blk; }
static int live(const kvo_pool *p, int32_t c) { return c >= 0 && c < p->max_ctx && p->len[c] >= 0; }

/* address of pool row (layer l, block b, K/V kv, slot s) */
static uint8_t *pool_row(const kvo_pool *p, int l, int32_t b, int kv, int s) {
    return p->pool + ((((int64_t)l * p->NB + b) * 2 + kv) * p->BS + s) * p->row;
}
/* address of row (layer l, K/V kv, token t) of an n-token transfer buffer */
static uint8_t *buf_row(const void *buf, int64_t n, const kvo_pool *p, int l, int kv, int64_t t) {
    return (uint8_t *)buf + (((int64_t)l * 2 + kv) * n + t) * p->row;
}

static void note_live(kvo_pool *p) {
    int64_t lv = p->NB - free_blocks(p);
    if (lv > p->peak_live) p->peak_live = lv;
}

/* take the oldest free block; it becomes referenced once */
static int32_t alloc_block(kvo_pool *p) {
    int32_t b = p->ring[p->head % (uint64_t)p->NB];
    p->head += 1;
    p->refcount[b] = 1;
    note_live(p);
    return b;
}
/* drop one reference; a block nobody references returns to the ring's tail */
static void release_block(kvo_pool *p, int32_t b) {
    p->refcount[b] -= 1;
    if (p->refcount[b] == 0) {
        p->ring[p->tail % (uint64_t)p->NB] = b;
        p->tail += 1;
    }
}
/* copy one token (all layers, K and V) between two pool slots */
static void copy_token(kvo_pool *p, int32_t db, int ds, int32_t sb, int ss) {
    for (int l = 0; l < p->L; ++l)
        for (int kv = 0; kv < 2; ++kv) {
            memcpy(pool_row(p, l, db, kv, ds), pool_row(p, l, sb, kv, ss), (size_t)p->row);
            p->rows_copied += 1;
        }
}
/* store token t of an n-token buffer at position pos of a block table */
static void store_token(kvo_pool *p, const int32_t *table, int64_t pos, const void *buf, int64_t n, int64_t t) {
    for (int l = 0; l < p->L; ++l)
        for (int kv = 0; kv < 2; ++kv) {
            memcpy(pool_row(p, l, table[pos / p->BS], kv, (int)(pos % p->BS)), buf_row(buf, n, p, l, kv, t),
                   (size_t)p->row);
            p->rows_copied += 1;
        }
}
static int32_t smallest_free_ctx(const kvo_pool *p) {
    for (int32_t c = 0; c < p->max_ctx; ++c)
        if (p->len[c] < 0) return c;
    return -1;
}
static int has_duplicates(const int32_t *v, int32_t n) {
    for (int32_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < i; ++j)
            if (v[i] == v[j]) return 1;
    return 0;
}

/* Catalog bookkeeping (metadata catalog of App. A.2: "last_access: timestamp or logical clock for
 * eviction"; the reuse term of the eviction score).  The logical clock counts successful
 * state-touching operators; an operator stamps every state it reads, writes or creates. */
static void born(kvo_pool *p, int32_t c, int32_t origin, int32_t parent) {
    p->reuse[c] = 0;
    p->last_access[c] = p->clock;
    p->born[c] = p->clock;
    p->origin[c] = origin;
    p->parent[c] = parent;
    p->parent_born[c] = parent >= 0 ? p->born[parent] : -1;
}
static void read_by_other(kvo_pool *p, int32_t c) { p->reuse[c] += 1; p->last_access[c] = p->clock; }

/* ---------------------------------------------------------------- create / destroy */

/* Pool creation: no block referenced, free ring = free_order (a permutation of
 * [0,NB)) or the identity, no live context.  The pool bytes start at zero; the
 * caller may overwrite them through kvo_pool_bytes() before the first operator. */
kvo_pool *kvo_create(int32_t L, int32_t H, int32_t D, int32_t BS, int32_t E, int32_t NB, int32_t max_ctx,
                     int32_t max_blk, const int32_t *free_order) {
    if (L < 1 || H < 1 || D < 1 || BS < 1 || E < 1 || NB < 1 || max_ctx < 1 || max_blk < 1) return NULL;
    kvo_pool *p = (kvo_pool *)calloc(1, sizeof(kvo_pool));
    if (!p) return NULL;
    p->L = L; p->H = H; p->D = D; p->BS = BS; p->E = E; p->NB = NB;
    p->max_ctx = max_ctx; p->max_blk = max_blk;
    p->row = (int64_t)H * D * E;
    p->pool = (uint8_t *)calloc((size_t)L * NB * 2 * BS, (size_t)p->row);
    p->refcount = (int32_t *)calloc((size_t)NB, sizeof(int32_t));
    p->ring = (int32_t *)malloc((size_t)NB * sizeof(int32_t));
    p->table = (int32_t *)calloc((size_t)max_ctx * max_blk, sizeof(int32_t));
    p->len = (int64_t *)malloc((size_t)max_ctx * sizeof(int64_t));
    p->reuse = (int64_t *)calloc((size_t)max_ctx, sizeof(int64_t));
    p->last_access = (int64_t *)calloc((size_t)max_ctx, sizeof(int64_t));
    p->origin = (int32_t *)calloc((size_t)max_ctx, sizeof(int32_t));
    p->parent = (int32_t *)calloc((size_t)max_ctx, sizeof(int32_t));
    p->born = (int64_t *)calloc((size_t)max_ctx, sizeof(int64_t));
    p->parent_born = (int64_t *)calloc((size_t)max_ctx, sizeof(int64_t));
    if (!p->pool || !p->refcount || !p->ring || !p->table || !p->len || !p->reuse || !p->last_access || !p->origin ||
        !p->parent || !p->born || !p->parent_born)
        return NULL;
    for (int32_t i = 0; i < NB; ++i) p->ring[i] = free_order ? free_order[i] : i;
    for (int32_t c = 0; c < max_ctx; ++c) p->len[c] = -1;
    p->head = 0;
    p->tail = (uint64_t)NB;
    return p;
}

void kvo_destroy(kvo_pool *p) {
    if (!p) return;
    free(p->pool); free(p->refcount); free(p->ring); free(p->table); free(p->len);
    free(p->reuse); free(p->last_access); free(p->origin); free(p->parent); free(p->born); free(p->parent_born);
    free(p);
}

/* deep copy (used by the exhaustive search over operator sequences) */
kvo_pool *kvo_clone(const kvo_pool *s) {
    kvo_pool *p = kvo_create(s->L, s->H, s->D, s->BS, s->E, s->NB, s->max_ctx, s->max_blk, NULL);
    if (!p) return NULL;
    memcpy(p->pool, s->pool, (size_t)s->L * s->NB * 2 * s->BS * (size_t)s->row);
    memcpy(p->refcount, s->refcount, (size_t)s->NB * sizeof(int32_t));
    memcpy(p->ring, s->ring, (size_t)s->NB * sizeof(int32_t));
    memcpy(p->table, s->table, (size_t)s->max_ctx * s->max_blk * sizeof(int32_t));
    memcpy(p->len, s->len, (size_t)s->max_ctx * sizeof(int64_t));
    memcpy(p->reuse, s->reuse, (size_t)s->max_ctx * sizeof(int64_t));
    memcpy(p->last_access, s->last_access, (size_t)s->max_ctx * sizeof(int64_t));
    memcpy(p->origin, s->origin, (size_t)s->max_ctx * sizeof(int32_t));
    memcpy(p->parent, s->parent, (size_t)s->max_ctx * sizeof(int32_t));
    memcpy(p->born, s->born, (size_t)s->max_ctx * sizeof(int64_t));
    memcpy(p->parent_born, s->parent_born, (size_t)s->max_ctx * sizeof(int64_t));
    p->clock = s->clock;
    p->head = s->head; p->tail = s->tail;
    p->peak_live = s->peak_live; p->cow_count = s->cow_count; p->rows_copied = s->rows_copied;
    return p;
}

uint8_t *kvo_pool_bytes(kvo_pool *p) { return p->pool; }
int64_t kvo_pool_nbytes(const kvo_pool *p) { return (int64_t)p->L * p->NB * 2 * p->BS * p->row; }

/* ---------------------------------------------------------------- import */

/* Registration of received / freshly produced KV (Alg. "KV-Materialize" steps 4-6:
 * partition the layer-wise tensors into blocks and register them; Alg.
 * "KV-Transfer": register received blocks at the destination).  The n tokens of
 * buf ([L][2][n][row]) become a new context whose blocks are taken from the ring
 * in order; each new block is referenced once. */
int kvo_import(kvo_pool *p, const void *buf, int64_t n, int32_t *out_ctx) {
    if (!buf || !out_ctx || n < 1) return KVO_INVALID_ARG;
    if (nblk(p, n) > p->max_blk) return KVO_TOO_LONG;
    int32_t c = smallest_free_ctx(p);
    if (c < 0) return KVO_OOM_CTX;
    if (free_blocks(p) < nblk(p, n)) return KVO_OOM_BLOCKS;
    int32_t *t = tbl(p, c);
    for (int64_t j = 0; j < nblk(p, n); ++j) t[j] = alloc_block(p);
    for (int64_t tok = 0; tok < n; ++tok) store_token(p, t, tok, buf, n, tok);
    p->len[c] = n;
    p->clock += 1;
    born(p, c, 1, -1);
    *out_ctx = c;
    return KVO_OK;
}

/* ---------------------------------------------------------------- materialize */

/* Packing of a context's token range [t0,t1) into a contiguous transfer buffer
 * (Alg. "KV-Transfer": select the required blocks by position range, then hand
 * raw buffers to the transport; Sec. 5.4: block granularity, prefix subsets).
 * A pure read of the pool: dst[l][kv][t-t0] = pool[l][table[t/BS]][kv][t mod BS].
 * Transfer changes placement, never logical content (Sec. 3.3). */
int kvo_materialize(kvo_pool *p, int32_t c, int64_t t0, int64_t t1, void *dst, int64_t dst_bytes) {
    if (!dst) return KVO_INVALID_ARG;
    if (!live(p, c)) return KVO_BAD_CTX;
    if (t0 < 0 || t0 >= t1 || t1 > p->len[c]) return KVO_INVALID_ARG;
    int64_t n = t1 - t0;
    if (dst_bytes < n * 2 * p->L * p->row) return KVO_DST_TOO_SMALL;
    const int32_t *t = tbl(p, c);
    for (int64_t tok = t0; tok < t1; ++tok)
        for (int l = 0; l < p->L; ++l)
            for (int kv = 0; kv < 2; ++kv) {
                memcpy(buf_row(dst, n, p, l, kv, tok - t0), pool_row(p, l, t[tok / p->BS], kv, (int)(tok % p->BS)),
                       (size_t)p->row);
                p->rows_copied += 1;
            }
    p->clock += 1;
    read_by_other(p, c);
    return KVO_OK;
}

/* ---------------------------------------------------------------- fork */

/* Alg. "KV-Fork": k logical children alias the parent's blocks by raising the
 * block reference counts; nothing is copied and no block is allocated.  Children
 * share physical blocks until they diverge (Sec. 3.3). */
int kvo_fork(kvo_pool *p, int32_t parent, int32_t k, int32_t *out_children) {
    if (!out_children || k < 1) return KVO_INVALID_ARG;
    if (!live(p, parent)) return KVO_BAD_CTX;
    int32_t free_slots = 0;
    for (int32_t c = 0; c < p->max_ctx; ++c) free_slots += p->len[c] < 0;
    if (free_slots < k) return KVO_OOM_CTX;
    int64_t nb = nblk(p, p->len[parent]);
    p->clock += 1;
    read_by_other(p, parent);
    for (int32_t j = 0; j < k; ++j) {
        int32_t c = smallest_free_ctx(p);
        for (int64_t q = 0; q < nb; ++q) {
            tbl(p, c)[q] = tbl(p, parent)[q];
            p->refcount[tbl(p, parent)[q]] += 1;
        }
        p->len[c] = p->len[parent];
        born(p, c, 2, parent);
        out_children[j] = c;
    }
    return KVO_OK;
}

/* ---------------------------------------------------------------- append (+ copy-on-write) */

/* One context grows by n tokens (Alg. "KV-Resume": register newly generated
 * continuation blocks).  Copy-on-write on divergence (Sec. 3.3; App. A.2: shared
 * prefix blocks stay aliased, continuation blocks are allocated separately): only
 * the partial tail block can be written by an append, so only it is ever copied,
 * and only its valid rows. */
static void append_one(kvo_pool *p, int32_t c, const void *src, int64_t n) {
    int64_t T = p->len[c];
    int64_t r = T % p->BS;
    int32_t *t = tbl(p, c);
    if (r > 0 && p->refcount[t[nblk(p, T) - 1]] > 1) {
        int32_t old = t[nblk(p, T) - 1];
        int32_t nb = alloc_block(p);
        for (int64_t s = 0; s < r; ++s) copy_token(p, nb, (int)s, old, (int)s);
        release_block(p, old);
        t[nblk(p, T) - 1] = nb;
        p->cow_count += 1;
    }
    for (int64_t j = nblk(p, T); j < nblk(p, T + n); ++j) t[j] = alloc_block(p);
    for (int64_t q = 0; q < n; ++q) store_token(p, t, T + q, src, n, q);
    p->len[c] = T + n;
}

/* A batch is the for-loop over its entries in array order; it is all-or-nothing:
 * the block need of the whole loop is found first on a scratch copy of the
 * reference counts. */
int kvo_append(kvo_pool *p, int32_t n, const int32_t *ctxs, const int32_t *n_new, const void *const *src) {
    if (n < 1 || !ctxs || !n_new || !src) return KVO_INVALID_ARG;
    for (int32_t i = 0; i < n; ++i) {
        if (!live(p, ctxs[i])) return KVO_BAD_CTX;
        if (n_new[i] < 1 || !src[i]) return KVO_INVALID_ARG;
    }
    if (has_duplicates(ctxs, n)) return KVO_INVALID_ARG;
    for (int32_t i = 0; i < n; ++i)
        if (nblk(p, p->len[ctxs[i]] + n_new[i]) > p->max_blk) return KVO_TOO_LONG;
    int32_t *rc = (int32_t *)malloc((size_t)p->NB * sizeof(int32_t));
    memcpy(rc, p->refcount, (size_t)p->NB * sizeof(int32_t));
    int64_t need = 0;
    for (int32_t i = 0; i < n; ++i) {
        int64_t T = p->len[ctxs[i]];
        if (T % p->BS > 0) {
            int32_t b = tbl(p, ctxs[i])[nblk(p, T) - 1];
            if (rc[b] > 1) { rc[b] -= 1; need += 1; }
        }
        need += nblk(p, T + n_new[i]) - nblk(p, T);
    }
    free(rc);
    if (free_blocks(p) < need) return KVO_OOM_BLOCKS;
    p->clock += 1;
    for (int32_t i = 0; i < n; ++i) {
        append_one(p, ctxs[i], src[i], n_new[i]);
        p->last_access[ctxs[i]] = p->clock;
    }
    return KVO_OK;
}

/* ---------------------------------------------------------------- compose */

/* Alg. "Restricted-KV-Merge", concatenation branch: the result is the strictly
 * sequential, non-overlapping concatenation of the segments (Sec. 4.5), bytes
 * moved verbatim.  A segment that starts on a block boundary shares its full
 * blocks by reference; everything behind the first partial tail is re-packed
 * into fresh blocks so that the result is an ordinary dense block table.  With
 * KVO_COMPOSE_COPY_ALL (merge policy mu that forbids aliasing) nothing is shared.
 * Sources stay live and unchanged; the same context may appear more than once. */
int kvo_compose(kvo_pool *p, int32_t m, const int32_t *segs, uint32_t flags, int32_t *out_ctx) {
    if (m < 1 || !segs || !out_ctx || (flags & ~KVO_COMPOSE_COPY_ALL)) return KVO_INVALID_ARG;
    for (int32_t i = 0; i < m; ++i)
        if (!live(p, segs[i])) return KVO_BAD_CTX;
    int copy_all = (flags & KVO_COMPOSE_COPY_ALL) != 0;
    /* block need is a function of the lengths alone */
    int64_t off = 0, need = 0;
    for (int32_t i = 0; i < m; ++i) {
        int64_t T = p->len[segs[i]];
        if (copy_all || off % p->BS != 0) need += nblk(p, off + T) - nblk(p, off);
        else if (T % p->BS > 0 && i != m - 1) need += 1;
        off += T;
    }
    if (nblk(p, off) > p->max_blk) return KVO_TOO_LONG;
    int32_t c = smallest_free_ctx(p);
    if (c < 0) return KVO_OOM_CTX;
    if (free_blocks(p) < need) return KVO_OOM_BLOCKS;

    p->clock += 1;
    for (int32_t i = 0; i < m; ++i) read_by_other(p, segs[i]);
    int32_t *nt = tbl(p, c);
    int64_t cnt = 0; /* entries of the new table so far */
    off = 0;
    for (int32_t i = 0; i < m; ++i) {
        const int32_t *st = tbl(p, segs[i]);
        int64_t T = p->len[segs[i]];
        if (!copy_all && off % p->BS == 0) {
            int64_t full = T / p->BS, rem = T % p->BS;
            for (int64_t j = 0; j < full; ++j) {
                nt[cnt++] = st[j];
                p->refcount[st[j]] += 1;
            }
            if (rem > 0) {
                if (i == m - 1) {
                    nt[cnt++] = st[full];
                    p->refcount[st[full]] += 1;
                } else {
                    int32_t nb = alloc_block(p);
                    for (int64_t s = 0; s < rem; ++s) copy_token(p, nb, (int)s, st[full], (int)s);
                    nt[cnt++] = nb;
                }
            }
        } else {
            while (cnt < nblk(p, off + T)) nt[cnt++] = alloc_block(p);
            for (int64_t t = 0; t < T; ++t)
                copy_token(p, nt[(off + t) / p->BS], (int)((off + t) % p->BS), st[t / p->BS], (int)(t % p->BS));
        }
        off += T;
    }
    p->len[c] = off;
    born(p, c, 3, segs[0]);
    *out_ctx = c;
    return KVO_OK;
}

/* ---------------------------------------------------------------- evict */

/* Alg. "KV-Evict", release step: evicting a logical state drops one reference per
 * block-table entry; a block still referenced by another state survives, a block
 * nobody references returns to the free ring (shared prefix blocks are retained
 * while any branch references them).  Victim selection (the score) is the
 * caller's policy and is not part of this function. */
int kvo_evict(kvo_pool *p, int32_t n, const int32_t *ctxs) {
    if (n < 1 || !ctxs) return KVO_INVALID_ARG;
    for (int32_t i = 0; i < n; ++i)
        if (!live(p, ctxs[i])) return KVO_BAD_CTX;
    if (has_duplicates(ctxs, n)) return KVO_INVALID_ARG;
    p->clock += 1;
    for (int32_t i = 0; i < n; ++i) {
        int32_t c = ctxs[i];
        for (int64_t j = 0; j < nblk(p, p->len[c]); ++j) release_block(p, tbl(p, c)[j]);
        p->len[c] = -1;
    }
    return KVO_OK;
}

/* Alg. "KV-Evict", the whole loop: score(S) = alpha * reuse(S) - beta * size(S) - gamma * age(S) for
 * every live state, size in blocks, age = clock - last_access with the clock of this call; while the
 * allocated blocks exceed the budget, the state with the lowest score (ties: smallest handle) is
 * evicted by the release rule above.  Scores are computed once, before the loop, in double
 * precision with one rounding per operation, (alpha*reuse - beta*size) - gamma*age.
 * out_victims (cap >= number of live states) receives the evicted handles in eviction order. */
int kvo_evict_to_budget(kvo_pool *p, double alpha, double beta, double gamma, int64_t budget_blocks,
                        int32_t *out_victims, int32_t cap, int32_t *n_victims) {
    if (!out_victims || !n_victims || budget_blocks < 0) return KVO_INVALID_ARG;
    int32_t live_ctx = 0;
    for (int32_t c = 0; c < p->max_ctx; ++c) live_ctx += p->len[c] >= 0;
    if (cap < live_ctx) return KVO_INVALID_ARG;
    p->clock += 1;
    double *score = (double *)malloc((size_t)p->max_ctx * sizeof(double));
    for (int32_t c = 0; c < p->max_ctx; ++c) {
        if (p->len[c] < 0) continue;
        double t1 = alpha * (double)p->reuse[c];
        double t2 = beta * (double)nblk(p, p->len[c]);
        double t3 = gamma * (double)(p->clock - p->last_access[c]);
        score[c] = (t1 - t2) - t3;
    }
    int32_t nv = 0;
    while (p->NB - free_blocks(p) > budget_blocks) {
        int32_t best = -1;
        for (int32_t c = 0; c < p->max_ctx; ++c)
            if (p->len[c] >= 0 && (best < 0 || score[c] < score[best])) best = c;
        if (best < 0) break;
        for (int64_t j = 0; j < nblk(p, p->len[best]); ++j) release_block(p, tbl(p, best)[j]);
        p->len[best] = -1;
        out_victims[nv++] = best;
    }
    free(score);
    *n_victims = nv;
    return KVO_OK;
}

/* Columnar export of the metadata catalog (App. A.2, table of catalog fields; Sec. 5.3: metadata in a
 * columnar, zero-copy encoding).  State rows: one per live state in ascending handle order
 * (state_id, n_tokens, reuse, last_access, lineage: origin, parent, born, parent_born) plus list offsets into the block rows (offsets[i] =
 * number of block rows of the states before i, offsets[n_states] = total); block rows: one per
 * block-table entry (block_id, position range [pos_begin, pos_end) within the state, refcount of the
 * block, byte address of the block's layer-0 K run relative to the pool base).  Returns the counts. */
int kvo_export_catalog(const kvo_pool *p, int32_t *state_id, int64_t *n_tokens, int64_t *reuse,
                       int64_t *last_access, int32_t *origin, int32_t *parent, int64_t *born_at,
                       int64_t *parent_born, int32_t *block_offsets, int32_t *block_id, int64_t *pos_begin,
                       int64_t *pos_end, int32_t *refcount, int64_t *address, int32_t *n_states,
                       int32_t *n_block_rows) {
    int32_t ns = 0, nr = 0;
    for (int32_t c = 0; c < p->max_ctx; ++c) {
        if (p->len[c] < 0) continue;
        state_id[ns] = c;
        n_tokens[ns] = p->len[c];
        reuse[ns] = p->reuse[c];
        last_access[ns] = p->last_access[c];
        origin[ns] = p->origin[c];
        parent[ns] = p->parent[c];
        born_at[ns] = p->born[c];
        parent_born[ns] = p->parent_born[c];
        block_offsets[ns] = nr;
        for (int64_t j = 0; j < nblk(p, p->len[c]); ++j) {
            int32_t b = tbl(p, c)[j];
            block_id[nr] = b;
            pos_begin[nr] = j * p->BS;
            pos_end[nr] = (j + 1) * p->BS < p->len[c] ? (j + 1) * p->BS : p->len[c];
            refcount[nr] = p->refcount[b];
            address[nr] = (int64_t)b * 2 * p->BS * p->row;
            nr += 1;
        }
        ns += 1;
    }
    block_offsets[ns] = nr;
    *n_states = ns;
    *n_block_rows = nr;
    return KVO_OK;
}

/* catalog read-out: out[0] = clock; per handle reuse and last_access (-1 for a free handle) */
int kvo_get_catalog(const kvo_pool *p, int64_t *clock, int64_t *reuse, int64_t *last_access) {
    *clock = p->clock;
    for (int32_t c = 0; c < p->max_ctx; ++c) {
        reuse[c] = p->len[c] >= 0 ? p->reuse[c] : -1;
        last_access[c] = p->len[c] >= 0 ? p->last_access[c] : -1;
    }
    return KVO_OK;
}

/* ---------------------------------------------------------------- introspection */

int kvo_ctx_len(const kvo_pool *p, int32_t c, int64_t *n_tokens) {
    if (!live(p, c)) return KVO_BAD_CTX;
    *n_tokens = p->len[c];
    return KVO_OK;
}
int kvo_get_table(const kvo_pool *p, int32_t c, int32_t *out, int32_t cap, int32_t *n_blocks) {
    if (!live(p, c)) return KVO_BAD_CTX;
    int64_t nb = nblk(p, p->len[c]);
    if (cap < nb) return KVO_DST_TOO_SMALL;
    for (int64_t j = 0; j < nb; ++j) out[j] = tbl(p, c)[j];
    *n_blocks = (int32_t)nb;
    return KVO_OK;
}
int kvo_get_refcounts(const kvo_pool *p, int32_t *out) {
    for (int32_t b = 0; b < p->NB; ++b) out[b] = p->refcount[b];
    return KVO_OK;
}
/* free block ids in ring order starting at head */
int kvo_get_free_list(const kvo_pool *p, int32_t *out, int32_t *n_free) {
    int64_t f = free_blocks(p);
    for (int64_t i = 0; i < f; ++i) out[i] = p->ring[(p->head + (uint64_t)i) % (uint64_t)p->NB];
    *n_free = (int32_t)f;
    return KVO_OK;
}
/* out[0..5] = free blocks, live blocks, peak live blocks, live contexts, COW count, rows copied */
int kvo_stats(const kvo_pool *p, int64_t *out) {
    int64_t live_ctx = 0;
    for (int32_t c = 0; c < p->max_ctx; ++c) live_ctx += p->len[c] >= 0;
    out[0] = free_blocks(p);
    out[1] = p->NB - free_blocks(p);
    out[2] = p->peak_live;
    out[3] = live_ctx;
    out[4] = p->cow_count;
    out[5] = p->rows_copied;
    return KVO_OK;
}
