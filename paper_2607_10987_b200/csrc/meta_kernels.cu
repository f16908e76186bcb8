// Metadata kernels of libaafkv.so: the device-resident block allocator (FIFO free ring),
// the reference-count table and the block tables, plus the planners that turn an operator
// into a piece list for the copy engines.
//
// Determinism: which block a table entry gets, and where a freed block lands on the ring, must
// be a function of the call sequence alone.  So a batch makes ONE reservation on the ring
// (head advances once, by the batch's total need) and every entry finds its blocks at a
// prefix-sum offset from the old head; reference counts are updated with atomics whose order
// cannot change the result; frees are compacted in flattened (context, table position) order
// by a block-wide prefix scan.
#include <cuda_runtime.h>
#include <stdint.h>

#include "aafkv_internal.h"

namespace aafkv {

constexpr int PLAN_THREADS = 1024;

__device__ __forceinline__ void set_status(DevCtl *ctl, int code, int detail) {
    if (atomicCAS(&ctl->status, 0, code) == 0) ctl->status_detail = detail;
}
__device__ __forceinline__ void note_alloc(DevCtl *ctl, const Geom &g, unsigned long long new_head,
                                           unsigned long long tail) {
    const long long live = (long long)g.NB - (long long)(tail - new_head);
    if (live > ctl->peak_live) ctl->peak_live = live;
}
__device__ __forceinline__ int ring_at(const int *ring, unsigned long long pos, int NB) {
    return ring[pos % (unsigned long long)NB];
}
__device__ __forceinline__ Piece make_piece(const char *src, long long ssl, long long sskv, char *dst, long long dsl,
                                            long long dskv, unsigned nbytes) {
    Piece p;
    p.src = src; p.dst = dst;
    p.src_sl = ssl; p.src_skv = sskv;
    p.dst_sl = dsl; p.dst_skv = dskv;
    p.nbytes = nbytes;
    p.nbytes2 = 0;
    p.src2_off = 0;
    return p;
}
// marks a piece slot unused (both parts: a slot may still hold an earlier operator's two-part piece)
__device__ __forceinline__ void clear_piece(Piece &p) {
    p.nbytes = 0;
    p.nbytes2 = 0;
}
__device__ __forceinline__ char *pool_slot(const Geom &g, int b, long long slot) {
    return g.pool + (long long)b * 2 * g.run + slot * g.row;
}
// takes a fresh block for exclusive use; a block on the ring must be unreferenced
__device__ __forceinline__ void claim_block(const DevState &s, int b, int NB) {
    if (b < 0 || b >= NB) {
        set_status(s.ctl, AAF_ERR_CORRUPT, 1);
        return;
    }
    if (s.refcount[b] != 0) set_status(s.ctl, AAF_ERR_CORRUPT, 2);
    s.refcount[b] = 1;
}

// Adds a thread's byte count to the pool's payload counter: one atomic per warp instead of one per piece.
// Must be called by all threads of the CTA (converged).
__device__ __forceinline__ void add_payload(DevCtl *ctl, unsigned long long bytes) {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) bytes += __shfl_down_sync(0xffffffffu, bytes, d);
    if ((threadIdx.x & 31) == 0 && bytes) atomicAdd(&ctl->payload_bytes, bytes);
}

// Catalog entry of a state that has just been created (lineage: origin 1 = registered from a buffer,
// 2 = fork, 3 = merge; parent = handle it descends from or -1).
__device__ __forceinline__ void catalog_born(const DevState &s, int c, long long len, long long clock, int origin,
                                             int parent) {
    s.cat_len[c] = len;
    s.cat_reuse[c] = 0;
    s.cat_last[c] = clock;
    s.cat_origin[c] = origin;
    s.cat_parent[c] = parent;
    s.cat_born[c] = clock;
    s.cat_parent_born[c] = parent >= 0 ? s.cat_born[parent] : -1;
}

// Argument records arrive in pinned host memory that the kernel reads over PCIe; every such read costs
// a bus round trip and is not cached, so a kernel that searches its records stages them first: one
// coalesced pass into shared memory (when they fit), then all further reads are on-chip.
template <typename T>
__device__ __forceinline__ const T *stage_args(const T *src, int count, T *smem_buf, int cap) {
    static_assert(sizeof(T) % 4 == 0, "records are copied as 32-bit words");
    if (count > cap) return src;
    const int words = count * (int)(sizeof(T) / 4);
    const int *s32 = reinterpret_cast<const int *>(src);
    int *d32 = reinterpret_cast<int *>(smem_buf);
    for (int i = threadIdx.x; i < words; i += blockDim.x) d32[i] = s32[i];
    __syncthreads();
    return smem_buf;
}

// CTA-wide exclusive prefix sum of one int per thread (warp shuffles + one shared array).
// Returns the exclusive prefix of `v`; *total receives the CTA's sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int *total) {
    __shared__ int warp_sums[32];
    __shared__ int block_total;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += t;
    }
    __syncthreads();  // protects warp_sums / block_total of a previous call
    if (lane == 31) warp_sums[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        int w = lane < nw ? warp_sums[lane] : 0;
        int wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wi, d);
            if (lane >= d) wi += t;
        }
        warp_sums[lane] = wi - w;  // exclusive prefix of the warp sums
        if (lane == 31) block_total = wi;
    }
    __syncthreads();
    *total = block_total;
    return warp_sums[wid] + incl - v;
}

// ------------------------------------------------------------------------------------------
// last record whose first slot is <= sl (records sorted by their first slot)
template <typename T, typename F>
__device__ __forceinline__ int find_record(const T *rec, int n, int sl, F first_slot) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (first_slot(rec[mid]) <= sl) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ------------------------------------------------------------------------------------------
// materialize: one piece per block of every token range of the batch.  A pure read of the pool, so a batch is
// the loop over its entries in any order; the catalog is stamped as the loop would stamp it.
constexpr int MAT_STAGE = 512;
__global__ void __launch_bounds__(256) plan_materialize_kernel(Geom g, DevState s,
                                                               const MatEntry *__restrict__ ents_host, SmallMat small,
                                                               int n, int total_pieces, long long clock) {
    __shared__ MatEntry sh_ent[MAT_STAGE];
    const MatEntry *ent;
    if (ents_host) {
        ent = stage_args(ents_host, n, sh_ent, MAT_STAGE);
    } else {  // a small batch arrives as kernel parameters
        if (threadIdx.x < n) sh_ent[threadIdx.x] = small.e[threadIdx.x];
        __syncthreads();
        ent = sh_ent;
    }
    for (int sl = blockIdx.x * blockDim.x + threadIdx.x; sl < total_pieces; sl += gridDim.x * blockDim.x) {
        const MatEntry e = ent[find_record(ent, n, sl, [](const MatEntry &r) { return r.piece_off; })];
        const long long cnt = e.t1 - e.t0;
        const long long j = e.t0 / g.BS + (sl - e.piece_off);  // table position of the block
        const long long lo = max(e.t0, j * g.BS), hi = min(e.t1, (j + 1) * g.BS);
        const int b = s.tables[(long long)e.ctx * g.max_blk + (j - e.table_j0)];
        if (b < 0 || b >= g.NB) {  // never gather through an entry that does not name a pool block
            clear_piece(s.pieces[sl]);
            set_status(s.ctl, AAF_ERR_CORRUPT, 10);
            continue;
        }
        s.pieces[sl] = make_piece(pool_slot(g, b, lo - j * g.BS), g.layer_stride, g.run, e.dst + (lo - e.t0) * g.row,
                                  2 * cnt * g.row, cnt * g.row, (unsigned)((hi - lo) * g.row));
    }
    if (blockIdx.x == 0)
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            atomicAdd(&s.ctl->payload_bytes, (unsigned long long)((ent[i].t1 - ent[i].t0) * 2 * g.L * g.row));
            if (s.cat_len) {  // the state was read by a transfer
                atomicAdd(&s.cat_reuse[ent[i].ctx], 1ull);
                atomicMax(&s.cat_last[ent[i].ctx], clock + ent[i].out_index);
            }
        }
}

// ------------------------------------------------------------------------------------------
// import: one ring reservation for the whole batch; entry i takes ceil(n_i / BS) entries behind those of the
// entries before it (what the loop over the batch would take), writes its table, one piece per block
constexpr int IMP_STAGE = 512;
__global__ void __launch_bounds__(PLAN_THREADS) plan_import_kernel(Geom g, DevState s,
                                                                   const ImpEntry *__restrict__ ents_host,
                                                                   SmallImp small, int n, int total_blocks,
                                                                   long long clock) {
    __shared__ ImpEntry sh_ent[IMP_STAGE];
    const ImpEntry *ent;
    if (ents_host) {
        ent = stage_args(ents_host, n, sh_ent, IMP_STAGE);
    } else {  // a small batch arrives as kernel parameters
        if (threadIdx.x < n) sh_ent[threadIdx.x] = small.e[threadIdx.x];
        __syncthreads();
        ent = sh_ent;
    }
    const unsigned long long head0 = s.ctl->head, tail = s.ctl->tail;
    const bool ok = (tail - head0) >= (unsigned long long)total_blocks;
    for (int sl = threadIdx.x; sl < total_blocks; sl += blockDim.x) {
        if (!ok) {
            clear_piece(s.pieces[sl]);
            continue;
        }
        const ImpEntry e = ent[find_record(ent, n, sl, [](const ImpEntry &r) { return r.block_off; })];
        const int j = sl - e.block_off;
        const int b = ring_at(s.ring, head0 + (unsigned long long)sl, g.NB);
        claim_block(s, b, g.NB);
        s.tables[(long long)e.ctx * g.max_blk + j] = b;
        const long long lo = (long long)j * g.BS, hi = min(e.n, lo + g.BS);
        s.pieces[sl] = make_piece(e.src + lo * g.row, 2 * e.n * g.row, e.n * g.row, pool_slot(g, b, 0), g.layer_stride,
                                  g.run, (unsigned)((hi - lo) * g.row));
    }
    if (ok)
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            atomicAdd(&s.ctl->payload_bytes, (unsigned long long)(ent[i].n * 2 * g.L * g.row));
            if (s.cat_len) catalog_born(s, ent[i].ctx, ent[i].n, clock + ent[i].out_index, 1, -1);
        }
    __syncthreads();  // every thread has read head0 before it moves
    if (threadIdx.x == 0) {
        if (!ok) {
            set_status(s.ctl, AAF_ERR_CORRUPT, 3);
        } else {
            s.ctl->head = head0 + total_blocks;
            note_alloc(s.ctl, g, head0 + total_blocks, tail);
        }
    }
}

// ------------------------------------------------------------------------------------------
// fork: k table copies, refcount += k per parent entry
__global__ void __launch_bounds__(256) fork_kernel(Geom g, DevState s, int parent, long long T, int k,
                                                   const int *__restrict__ children_host, SmallInts small,
                                                   long long clock) {
    const int nblk = (int)((T + g.BS - 1) / g.BS);
    __shared__ int sh_children[1024];
    const int *children;
    if (children_host) {
        children = stage_args(children_host, k, sh_children, 1024);
    } else {  // a small fan-out arrives as kernel parameters
        if (threadIdx.x < k) sh_children[threadIdx.x] = small.v[threadIdx.x];
        __syncthreads();
        children = sh_children;
    }
    const int *pt = s.tables + (long long)parent * g.max_blk;
    const long long total = (long long)nblk * k;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int q = (int)(e / nblk), j = (int)(e % nblk);
        const int b = pt[j];
        s.tables[(long long)children[q] * g.max_blk + j] = b;
        if (q == 0) atomicAdd(&s.refcount[b], k);
        if (j == 0 && s.cat_len) {  // catalog: the child is born, the parent was read
            catalog_born(s, children[q], T, clock, 2, parent);
            if (q == 0) {
                s.cat_reuse[parent] += 1;
                s.cat_last[parent] = clock;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// append (+ copy-on-write)
//
// Sequential meaning of a batch: entry i copies its partial tail block iff the block is still
// shared when the loop reaches i.  Among the batch entries whose partial tail is the same block b,
// the one with rank q (q-th in array order) therefore copies iff q < refcount_before[b] - 1; the
// entry that finds the count at 1 appends in place.  It writes only slots >= r while the copiers
// read slots < r, so the batch's copies have no ordering hazard.
//
// scratch layout (ints): tailb[n] | need[n] | alloc_off[n]
__global__ void __launch_bounds__(PLAN_THREADS) plan_append_kernel(Geom g, DevState s,
                                                                   const AppendEntry *__restrict__ ent_host,
                                                                   SmallAppend small, int n, int total_slots,
                                                                   int max_batch, int dry_run, long long clock) {
    __shared__ AppendEntry sh_ent[768];
    const AppendEntry *ent;
    if (ent_host) {
        ent = stage_args(ent_host, n, sh_ent, 768);
    } else {  // a small batch arrives as kernel parameters
        if (threadIdx.x < n) sh_ent[threadIdx.x] = small.e[threadIdx.x];
        __syncthreads();
        ent = sh_ent;
    }
    int *tailb = s.scratch;
    int *need = s.scratch + max_batch;
    int *alloc_off = s.scratch + 2 * max_batch;
    __shared__ int sh_total_need;
    const unsigned long long head0 = s.ctl->head, tail = s.ctl->tail;

    // phase 1: the partial tail block of every entry (-1 if the context ends on a block boundary)
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const long long T = ent[i].T;
        const int r = (int)(T % g.BS);
        tailb[i] = r > 0 ? s.tables[(long long)ent[i].ctx * g.max_blk + (T - 1) / g.BS] : -1;
    }
    __syncthreads();
    // phase 2: copy-on-write decision and block need of every entry.  The rank of an entry among the earlier
    // entries with the same tail block is a scan of tailb[0 .. i): from shared memory when the batch fits.
    __shared__ int sh_tailb[1024];
    const int *tb = tailb;
    if (n <= 1024) {
        for (int i = threadIdx.x; i < n; i += blockDim.x) sh_tailb[i] = tailb[i];
        __syncthreads();
        tb = sh_tailb;
    }
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const long long T = ent[i].T;
        const int b = tb[i];
        int cow = 0;
        if (b >= 0) {
            int rank = 0;
            for (int i2 = 0; i2 < i; ++i2) rank += (tb[i2] == b);
            cow = rank < s.refcount[b] - 1;
        }
        const int fresh = (int)((T + ent[i].n_new + g.BS - 1) / g.BS - (T + g.BS - 1) / g.BS);
        need[i] = (cow << 30) | (cow + fresh);  // bit 30 remembers the decision
    }
    __syncthreads();
    // phase 3: exclusive scan of the needs -> offset of each entry's blocks from the old ring head
    int carry = 0;
    for (int base = 0; base < n; base += blockDim.x) {
        const int i = base + threadIdx.x;
        const int v = i < n ? (need[i] & 0x3fffffff) : 0;
        int tot;
        const int ex = block_exclusive_scan(v, &tot);
        if (i < n) alloc_off[i] = carry + ex;
        carry += tot;
    }
    if (threadIdx.x == 0) sh_total_need = carry;
    __syncthreads();
    const int total_need = sh_total_need;
    if (dry_run) {
        if (threadIdx.x == 0) s.ctl->probe_need = (unsigned long long)total_need;
        return;
    }
    const bool ok = (tail - head0) >= (unsigned long long)total_need;

    // phase 4: one thread per piece slot.  Slot piece_off[i] is entry i's copy-on-write piece, the
    // slots behind it are the blocks its new tokens touch, in table order.
    unsigned long long my_bytes = 0;
    for (int sl = threadIdx.x; sl < total_slots; sl += blockDim.x) {
        if (!ok) {
            clear_piece(s.pieces[sl]);
            continue;
        }
        int lo = 0, hi = n - 1;  // last entry whose piece_off <= sl
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (ent[mid].piece_off <= sl) lo = mid; else hi = mid - 1;
        }
        const int i = lo;
        const AppendEntry e = ent[i];
        const long long T = e.T;
        const int r = (int)(T % g.BS);
        const int cow = (need[i] >> 30) & 1;
        const unsigned long long first = head0 + (unsigned long long)alloc_off[i];
        int *table = s.tables + (long long)e.ctx * g.max_blk;
        const long long nblk_T = (T + g.BS - 1) / g.BS;
        const int w = sl - e.piece_off;
        if (w == 0) {
            if (cow) {
                const int old = tailb[i];
                const int nb = ring_at(s.ring, first, g.NB);
                claim_block(s, nb, g.NB);
                if (atomicSub(&s.refcount[old], 1) <= 1) set_status(s.ctl, AAF_ERR_CORRUPT, 4);
                table[nblk_T - 1] = nb;
                s.pieces[sl] = make_piece(pool_slot(g, old, 0), g.layer_stride, g.run, pool_slot(g, nb, 0),
                                          g.layer_stride, g.run, (unsigned)(r * g.row));
                atomicAdd(&s.ctl->cow_count, 1ull);
                my_bytes += (unsigned long long)(r * g.row * 2 * g.L);
            } else {
                clear_piece(s.pieces[sl]);
            }
            continue;
        }
        const long long jpos = T / g.BS + (w - 1);  // table position of the touched block
        int b;
        if (jpos >= nblk_T) {  // a fresh continuation block
            b = ring_at(s.ring, first + cow + (unsigned long long)(jpos - nblk_T), g.NB);
            claim_block(s, b, g.NB);
            table[jpos] = b;
        } else {  // the partial tail: the copy if there is one, else written in place
            b = cow ? ring_at(s.ring, first, g.NB) : tailb[i];
        }
        const long long tlo = max(T, jpos * g.BS), thi = min(T + e.n_new, (jpos + 1) * g.BS);
        s.pieces[sl] = make_piece(e.src + (tlo - T) * g.row, 2ll * e.n_new * g.row, (long long)e.n_new * g.row,
                                  pool_slot(g, b, tlo - jpos * g.BS), g.layer_stride, g.run,
                                  (unsigned)((thi - tlo) * g.row));
        my_bytes += (unsigned long long)((thi - tlo) * g.row * 2 * g.L);
    }
    add_payload(s.ctl, my_bytes);
    if (ok && s.cat_len)
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            s.cat_len[ent[i].ctx] = ent[i].T + ent[i].n_new;
            s.cat_last[ent[i].ctx] = clock;
        }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!ok) {
            set_status(s.ctl, AAF_ERR_CORRUPT, 5);
        } else {
            s.ctl->head = head0 + total_need;
            note_alloc(s.ctl, g, head0 + total_need, tail);
        }
    }
}

// ------------------------------------------------------------------------------------------
// compose: flattened over the work items of all segments of all merges of the batch (host supplies the prefix
// sums of the lengths, which it knows; block ids come from the ring at rank offsets from the old head).
//   share segment : item w < full -> share entry w; item w == full -> the partial tail (shared by
//                   reference if it ends the result, else re-packed into a fresh block through the
//                   segment's single piece slot)
//   copy segment  : item w -> destination block nblk(off)-(off%BS>0) + w, which receives tokens
//                   from at most two source blocks (one two-part piece per item)
// A batch of merges is the for-loop over its merges: every merge reads only contexts that were live before the
// call, writes only its own fresh blocks and its own table, and takes its fresh blocks behind those of the merges
// before it; reference counts add up in any order; the catalog is stamped as the loop would stamp it (merge i at
// clock + i, a source's last access = the latest merge that read it).
__global__ void __launch_bounds__(PLAN_THREADS) plan_compose_kernel(Geom g, DevState s,
                                                                    const ComposeSeg *__restrict__ segs_host,
                                                                    SmallCompose small, int m, int total_work,
                                                                    int total_fresh, int total_slots, long long clock) {
    __shared__ ComposeSeg sh_segs[512];
    const ComposeSeg *segs;
    if (segs_host) {
        segs = stage_args(segs_host, m, sh_segs, 512);
    } else {  // a few segments arrive as kernel parameters
        if (threadIdx.x < m) sh_segs[threadIdx.x] = small.s[threadIdx.x];
        __syncthreads();
        segs = sh_segs;
    }
    const unsigned long long head0 = s.ctl->head, tail = s.ctl->tail;
    const bool ok = (tail - head0) >= (unsigned long long)total_fresh;
    if (!ok) {
        for (int sl = threadIdx.x; sl < total_slots; sl += blockDim.x) clear_piece(s.pieces[sl]);
    }
    unsigned long long my_bytes = 0;
    for (int it = threadIdx.x; ok && it < total_work; it += blockDim.x) {
        int lo = 0, hi = m - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (segs[mid].work_off <= it) lo = mid; else hi = mid - 1;
        }
        const ComposeSeg sg = segs[lo];
        const int w = it - sg.work_off;
        const int *st = s.tables + (long long)sg.ctx * g.max_blk;
        int *out = s.tables + (long long)sg.out_ctx * g.max_blk;
        if (sg.mode == 0) {
            const long long full = sg.T / g.BS;
            const int rem = (int)(sg.T % g.BS);
            if (w < full || sg.share_tail) {
                const int b = st[w];
                out[sg.dst_tbl_start + w] = b;
                atomicAdd(&s.refcount[b], 1);
            } else {  // w == full, rem > 0, not the last segment: re-pack the tail (the segment's one piece slot)
                const int nb = ring_at(s.ring, head0 + (unsigned long long)sg.fresh_start, g.NB);
                claim_block(s, nb, g.NB);
                out[sg.dst_tbl_start + w] = nb;
                s.pieces[sg.piece_off] = make_piece(pool_slot(g, st[full], 0), g.layer_stride, g.run,
                                                    pool_slot(g, nb, 0), g.layer_stride, g.run,
                                                    (unsigned)(rem * g.row));
                my_bytes += (unsigned long long)(rem * g.row * 2 * g.L);
            }
        } else {
            const long long nblk_off = (sg.off + g.BS - 1) / g.BS;
            const long long d = sg.off / g.BS + w;  // destination table position
            const int db = ring_at(s.ring, head0 + (unsigned long long)(sg.fresh_start + (d - nblk_off)), g.NB);
            if (d >= nblk_off) {  // allocated by this segment
                claim_block(s, db, g.NB);
                out[d] = db;
            }
            const long long lo_t = max(sg.off, d * g.BS), hi_t = min(sg.off + sg.T, (d + 1) * g.BS);
            const long long s_lo = lo_t - sg.off, s_hi = hi_t - sg.off;  // source token range
            const long long sb0 = s_lo / g.BS;
            const long long a_hi = min(s_hi, (sb0 + 1) * g.BS);
            // one two-part piece per destination block: the rows from source block sb0, then (if the range
            // crosses into it) the rows from the start of source block sb0 + 1, stored as one contiguous run
            Piece pc = make_piece(pool_slot(g, st[sb0], s_lo - sb0 * g.BS), g.layer_stride, g.run,
                                  pool_slot(g, db, lo_t - d * g.BS), g.layer_stride, g.run,
                                  (unsigned)((a_hi - s_lo) * g.row));
            if (a_hi < s_hi) {
                pc.nbytes2 = (unsigned)((s_hi - a_hi) * g.row);
                pc.src2_off = pool_slot(g, st[sb0 + 1], 0) - pc.src;
            }
            s.pieces[sg.piece_off + w] = pc;
            my_bytes += (unsigned long long)((s_hi - s_lo) * g.row * 2 * g.L);
        }
    }
    add_payload(s.ctl, my_bytes);
    if (ok && s.cat_len)
        for (int i = threadIdx.x; i < m; i += blockDim.x) {  // every occurrence of a segment is one read
            atomicAdd(&s.cat_reuse[segs[i].ctx], 1ull);
            atomicMax(&s.cat_last[segs[i].ctx], clock + segs[i].out_index);
        }
    __syncthreads();
    if (ok && s.cat_len)
        for (int i = threadIdx.x; i < m; i += blockDim.x)  // the last segment of a result registers the result
            if (segs[i].first_ctx >= 0)
                catalog_born(s, segs[i].out_ctx, segs[i].off + segs[i].T, clock + segs[i].out_index, 3,
                             segs[i].first_ctx);
    if (threadIdx.x == 0) {
        if (!ok) {
            set_status(s.ctl, AAF_ERR_CORRUPT, 6);
        } else {
            s.ctl->head = head0 + total_fresh;
            note_alloc(s.ctl, g, head0 + total_fresh, tail);
        }
    }
}

// ------------------------------------------------------------------------------------------
// evict
//   release : every flattened entry drops one reference and marks its block with
//             stamp | position, keeping the largest (atomicMax): the block's LAST occurrence in the batch.
//   push    : a block is freed by the entry at its last occurrence iff its count is now 0 (that is
//             where the sequential loop would have freed it); freed ids are compacted in flattened
//             order by a prefix scan and pushed at the ring's tail.
//   The mark's high 32 bits are the call's logical clock, so marks of earlier calls are always
//   smaller and the mark array never needs clearing.
//   Small batches (<= EVICT_FUSED_MAX entries) run both phases in one CTA; larger ones run the release
//   over a grid and the compaction as count / scan / scatter over tiles.
constexpr int EVICT_STAGE = 2064;        // ints staged in shared memory: ctx[n] followed by ent_off[n + 1] (n <= 1031)
constexpr int EVICT_ITEMS = 8;           // consecutive flattened entries per thread and pass
constexpr int EVICT_FUSED_MAX = 32768;
constexpr int EVICT_TILE = 1024 * EVICT_ITEMS;  // entries per CTA and pass (PLAN_THREADS threads)

__device__ __forceinline__ int find_ctx_index(const int *ent_off, int n, int e) {
    int lo = 0, hi = n - 1;  // last context whose first entry is <= e
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (ent_off[mid] <= e) lo = mid; else hi = mid - 1;
    }
    return lo;
}

__device__ __forceinline__ void evict_release_entry(const Geom &g, const DevState &s, const int *ctx,
                                                    const int *ent_off, int n, int e, unsigned long long stamp) {
    const int ci = find_ctx_index(ent_off, n, e);
    const int b = s.tables[(long long)ctx[ci] * g.max_blk + (e - ent_off[ci])];
    if (atomicSub(&s.refcount[b], 1) <= 0) set_status(s.ctl, AAF_ERR_CORRUPT, 7);
    atomicMax(&s.last_pos[b], stamp | (unsigned long long)(unsigned)e);
}

// One thread's share of a tile: its EVICT_ITEMS consecutive entries starting at e0.  Fills blk[] and
// returns the bit mask of the entries that free their block (count reached 0 and this entry is the
// block's last occurrence in the batch).  Reads only; the same call gives the same answer in every
// kernel that runs after the release phase.
__device__ __forceinline__ unsigned evict_thread_flags(const Geom &g, const DevState &s, const int *ctx,
                                                       const int *ent_off, int n, int total, int e0,
                                                       unsigned long long stamp, int (&blk)[EVICT_ITEMS]) {
    // locate the first entry once, then walk (context, position) forward: all table reads are independent
    int ci = e0 < total ? find_ctx_index(ent_off, n, e0) : 0;
#pragma unroll
    for (int k = 0; k < EVICT_ITEMS; ++k) {
        const int e = e0 + k;
        blk[k] = -1;
        if (e < total) {
            while (e >= ent_off[ci + 1]) ++ci;
            blk[k] = s.tables[(long long)ctx[ci] * g.max_blk + (e - ent_off[ci])];
        }
    }
    int rc[EVICT_ITEMS];
    unsigned long long lp[EVICT_ITEMS];
#pragma unroll
    for (int k = 0; k < EVICT_ITEMS; ++k) {
        rc[k] = blk[k] >= 0 ? s.refcount[blk[k]] : 1;
        lp[k] = blk[k] >= 0 ? s.last_pos[blk[k]] : 0ull;
    }
    unsigned flags = 0;
#pragma unroll
    for (int k = 0; k < EVICT_ITEMS; ++k) {
        const bool f = blk[k] >= 0 && rc[k] == 0 && lp[k] == (stamp | (unsigned long long)(unsigned)(e0 + k));
        flags |= (f ? 1u : 0u) << k;
    }
    return flags;
}

__device__ __forceinline__ void evict_write_ring(const Geom &g, const DevState &s, unsigned long long tail0, int pos,
                                                 unsigned flags, const int (&blk)[EVICT_ITEMS]) {
#pragma unroll
    for (int k = 0; k < EVICT_ITEMS; ++k)
        if (flags & (1u << k)) {
            s.ring[(tail0 + (unsigned long long)pos) % (unsigned long long)g.NB] = blk[k];
            ++pos;
        }
}

__device__ __forceinline__ void evict_finish(const Geom &g, const DevState &s, const int *ctx, int n,
                                             unsigned long long tail0, int freed) {
    if (s.cat_len)
        for (int i = threadIdx.x; i < n; i += blockDim.x) s.cat_len[ctx[i]] = -1;
    if (threadIdx.x == 0) {
        if (tail0 + freed - s.ctl->head > (unsigned long long)g.NB) set_status(s.ctl, AAF_ERR_CORRUPT, 8);
        s.ctl->tail = tail0 + freed;
    }
}

// compaction of the freed blocks by one CTA (all threads of the CTA must call it)
__device__ __forceinline__ void evict_push_phase(const Geom &g, const DevState &s, const int *ctx, const int *ent_off,
                                                 int n, int total, unsigned long long stamp) {
    const unsigned long long tail0 = s.ctl->tail;
    int carry = 0;
    for (int base = 0; base < total; base += EVICT_TILE) {
        int blk[EVICT_ITEMS];
        const unsigned flags =
            evict_thread_flags(g, s, ctx, ent_off, n, total, base + threadIdx.x * EVICT_ITEMS, stamp, blk);
        int tot;
        const int pos = carry + block_exclusive_scan(__popc(flags), &tot);
        evict_write_ring(g, s, tail0, pos, flags, blk);
        carry += tot;
    }
    evict_finish(g, s, ctx, n, tail0, carry);
}

// Large batches: the same compaction over a grid, one tile of EVICT_TILE entries per CTA.
//   count   : freed blocks per tile
//   scan    : exclusive prefix sum of the tile counts (one CTA), ring tail and catalog update
//   scatter : every tile recomputes its flags and writes its ids at tail0 + tile offset + local rank
__global__ void __launch_bounds__(PLAN_THREADS) evict_count_kernel(Geom g, DevState s,
                                                                   const EvictArgs *__restrict__ a, int n, int total,
                                                                   unsigned long long stamp, int *tile_count) {
    __shared__ int sh_args[EVICT_STAGE];
    const int *ctx = stage_args(reinterpret_cast<const int *>(a + 1), 2 * n + 1, sh_args, EVICT_STAGE);
    int blk[EVICT_ITEMS];
    const unsigned flags = evict_thread_flags(g, s, ctx, ctx + n, n, total,
                                              blockIdx.x * EVICT_TILE + threadIdx.x * EVICT_ITEMS, stamp, blk);
    int tot;
    block_exclusive_scan(__popc(flags), &tot);
    if (threadIdx.x == 0) tile_count[blockIdx.x] = tot;
}

__global__ void __launch_bounds__(PLAN_THREADS) evict_scan_kernel(Geom g, DevState s,
                                                                  const EvictArgs *__restrict__ a, int n, int n_tiles,
                                                                  int *tile_count) {
    const int *ctx = reinterpret_cast<const int *>(a + 1);
    const unsigned long long tail0 = s.ctl->tail;
    int carry = 0;
    for (int base = 0; base < n_tiles; base += blockDim.x) {
        const int t = base + threadIdx.x;
        const int v = t < n_tiles ? tile_count[t] : 0;
        int tot;
        const int ex = block_exclusive_scan(v, &tot);
        if (t < n_tiles) tile_count[t] = carry + ex;  // in place: count -> offset
        carry += tot;
    }
    if (threadIdx.x == 0) s.ctl->evict_tail0 = tail0;  // the scatter kernel needs the tail before this call
    evict_finish(g, s, ctx, n, tail0, carry);
}

__global__ void __launch_bounds__(PLAN_THREADS) evict_scatter_kernel(Geom g, DevState s,
                                                                     const EvictArgs *__restrict__ a, int n,
                                                                     int total, unsigned long long stamp,
                                                                     const int *tile_off) {
    __shared__ int sh_args[EVICT_STAGE];
    const int *ctx = stage_args(reinterpret_cast<const int *>(a + 1), 2 * n + 1, sh_args, EVICT_STAGE);
    int blk[EVICT_ITEMS];
    const unsigned flags = evict_thread_flags(g, s, ctx, ctx + n, n, total,
                                              blockIdx.x * EVICT_TILE + threadIdx.x * EVICT_ITEMS, stamp, blk);
    int tot;
    const int pos = tile_off[blockIdx.x] + block_exclusive_scan(__popc(flags), &tot);
    evict_write_ring(g, s, s.ctl->evict_tail0, pos, flags, blk);
}

__global__ void __launch_bounds__(256) evict_release_kernel(Geom g, DevState s, const EvictArgs *__restrict__ a,
                                                            int n, int total, unsigned long long stamp) {
    __shared__ int sh_args[EVICT_STAGE];
    const int *ctx = stage_args(reinterpret_cast<const int *>(a + 1), 2 * n + 1, sh_args, EVICT_STAGE);
    const int *ent_off = ctx + n;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x)
        evict_release_entry(g, s, ctx, ent_off, n, e, stamp);
}

__global__ void __launch_bounds__(PLAN_THREADS) evict_fused_kernel(Geom g, DevState s,
                                                                   const EvictArgs *__restrict__ a, SmallInts small,
                                                                   int n, int total, unsigned long long stamp) {
    __shared__ int sh_args[EVICT_STAGE];
    const int *ctx;
    if (a) {
        ctx = stage_args(reinterpret_cast<const int *>(a + 1), 2 * n + 1, sh_args, EVICT_STAGE);
    } else {  // a small batch arrives as kernel parameters
        if (threadIdx.x < 2 * n + 1) sh_args[threadIdx.x] = small.v[threadIdx.x];
        __syncthreads();
        ctx = sh_args;
    }
    const int *ent_off = ctx + n;
    for (int e = threadIdx.x; e < total; e += blockDim.x) evict_release_entry(g, s, ctx, ent_off, n, e, stamp);
    __syncthreads();  // one CTA: every reference has been dropped and every mark set
    evict_push_phase(g, s, ctx, ent_off, n, total, stamp);
}

// ------------------------------------------------------------------------------------------
// scored eviction (Alg. KV-Evict, the whole loop) in one CTA
//   score(S) = alpha * reuse(S) - beta * size(S) - gamma * age(S), size in blocks, age = clock - last access,
//   computed once in double precision with one rounding per operation (no fused multiply-add), so that
//   the victim order is the same on any IEEE machine.  While the live blocks exceed the budget the
//   state with the lowest score (ties: smallest handle) is released entry by entry with the same
//   rules as evict: a block is freed at its last occurrence in the victim's table, in table order.
__global__ void __launch_bounds__(PLAN_THREADS) evict_to_budget_kernel(Geom g, DevState s, double alpha, double beta,
                                                                       double gamma, long long budget,
                                                                       long long clock, int *result) {
    const unsigned long long stamp = (unsigned long long)clock << 32;
    __shared__ double sh_score[32];
    __shared__ int sh_id[32];
    __shared__ int sh_victim;
    __shared__ long long sh_live;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int c = threadIdx.x; c < g.max_ctx; c += blockDim.x) {
        const long long len = s.cat_len[c];
        if (len < 0) continue;
        const double t1 = __dmul_rn(alpha, (double)s.cat_reuse[c]);
        const double t2 = __dmul_rn(beta, (double)((len + g.BS - 1) / g.BS));
        const double t3 = __dmul_rn(gamma, (double)(clock - s.cat_last[c]));
        s.cat_score[c] = __dsub_rn(__dsub_rn(t1, t2), t3);
    }
    if (threadIdx.x == 0) sh_live = (long long)g.NB - (long long)(s.ctl->tail - s.ctl->head);
    __syncthreads();
    int nv = 0;
    while (true) {
        if (sh_live <= budget) break;  // uniform: read after a barrier
        // lowest (score, handle) among the live states
        double best = 0.0;
        int best_id = -1;
        for (int c = threadIdx.x; c < g.max_ctx; c += blockDim.x) {
            if (s.cat_len[c] < 0) continue;
            const double sc = s.cat_score[c];
            if (best_id < 0 || sc < best) { best = sc; best_id = c; }  // ascending c: ties keep the smaller handle
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            const double os = __shfl_down_sync(0xffffffffu, best, d);
            const int oi = __shfl_down_sync(0xffffffffu, best_id, d);
            if (oi >= 0 && (best_id < 0 || os < best || (os == best && oi < best_id))) { best = os; best_id = oi; }
        }
        if (lane == 0) { sh_score[wid] = best; sh_id[wid] = best_id; }
        __syncthreads();
        if (wid == 0) {
            best = sh_score[lane];
            best_id = sh_id[lane];
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) {
                const double os = __shfl_down_sync(0xffffffffu, best, d);
                const int oi = __shfl_down_sync(0xffffffffu, best_id, d);
                if (oi >= 0 && (best_id < 0 || os < best || (os == best && oi < best_id))) { best = os; best_id = oi; }
            }
            if (lane == 0) sh_victim = best_id;
        }
        __syncthreads();
        const int v = sh_victim;
        if (v < 0) break;
        // release the victim's entries
        const int nb = (int)((s.cat_len[v] + g.BS - 1) / g.BS);
        const int *table = s.tables + (long long)v * g.max_blk;
        // marks grow from victim to victim (max_ctx * max_blk < 2^31), so none has to be cleared
        const unsigned long long vstamp = stamp + (unsigned long long)nv * (unsigned long long)g.max_blk;
        for (int e = threadIdx.x; e < nb; e += blockDim.x) {
            const int b = table[e];
            if (atomicSub(&s.refcount[b], 1) <= 0) set_status(s.ctl, AAF_ERR_CORRUPT, 9);
            atomicMax(&s.last_pos[b], vstamp + (unsigned long long)(unsigned)e);
        }
        __syncthreads();
        const unsigned long long tail0 = s.ctl->tail;
        int carry = 0;
        for (int base = 0; base < nb; base += blockDim.x) {
            const int e = base + threadIdx.x;
            int b = -1, flag = 0;
            if (e < nb) {
                b = table[e];
                flag = (s.refcount[b] == 0 && s.last_pos[b] == (vstamp + (unsigned long long)(unsigned)e));
            }
            int tot;
            const int ex = block_exclusive_scan(flag, &tot);
            if (flag) s.ring[(tail0 + (unsigned long long)(carry + ex)) % (unsigned long long)g.NB] = b;
            carry += tot;
        }
        if (threadIdx.x == 0) {
            s.ctl->tail = tail0 + carry;
            sh_live -= carry;
            s.cat_len[v] = -1;
            result[2 + nv] = v;
        }
        ++nv;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        result[0] = nv;
        result[1] = (int)(s.ctl->tail - s.ctl->head);
    }
}

// ------------------------------------------------------------------------------------------
// columnar catalog export
//   kernel 1 (one CTA): two exclusive prefix scans over the handles -- live flags give each state its
//   row, block-table lengths give the list offsets -- and the state columns.
//   kernel 2 (grid): one thread per block row; the row's state is found by binary search in the
//   offsets, then the row is filled from the table and the reference counts (coalesced writes).
__global__ void __launch_bounds__(PLAN_THREADS) export_states_kernel(Geom g, DevState s, aaf_kv_catalog_cols cols) {
    int row_carry = 0, blk_carry = 0;
    for (int base = 0; base < g.max_ctx; base += blockDim.x) {
        const int c = base + threadIdx.x;
        const long long len = c < g.max_ctx ? s.cat_len[c] : -1;
        const int live = len >= 0;
        const int nb = live ? (int)((len + g.BS - 1) / g.BS) : 0;
        int live_tot, blk_tot;
        const int row = row_carry + block_exclusive_scan(live, &live_tot);
        const int off = blk_carry + block_exclusive_scan(nb, &blk_tot);
        if (live) {
            cols.state_id[row] = c;
            cols.n_tokens[row] = len;
            cols.reuse[row] = (long long)s.cat_reuse[c];
            cols.last_access[row] = s.cat_last[c];
            cols.origin[row] = s.cat_origin[c];
            cols.parent[row] = s.cat_parent[c];
            cols.born[row] = s.cat_born[c];
            cols.parent_born[row] = s.cat_parent_born[c];
            cols.block_offsets[row] = off;
        }
        row_carry += live_tot;
        blk_carry += blk_tot;
    }
    if (threadIdx.x == 0) cols.block_offsets[row_carry] = blk_carry;
}

__global__ void __launch_bounds__(256) export_blocks_kernel(Geom g, DevState s, aaf_kv_catalog_cols cols,
                                                            int n_states, long long n_rows) {
    for (long long r = blockIdx.x * (long long)blockDim.x + threadIdx.x; r < n_rows;
         r += (long long)gridDim.x * blockDim.x) {
        int lo = 0, hi = n_states - 1;  // last state whose offset <= r
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (cols.block_offsets[mid] <= r) lo = mid; else hi = mid - 1;
        }
        const int c = cols.state_id[lo];
        const long long j = r - cols.block_offsets[lo];
        const long long len = cols.n_tokens[lo];
        const int b = s.tables[(long long)c * g.max_blk + j];
        cols.block_id[r] = b;
        cols.pos_begin[r] = j * g.BS;
        cols.pos_end[r] = min((j + 1) * g.BS, len);
        cols.refcount[r] = s.refcount[b];
        cols.address[r] = (long long)b * 2 * g.run;
    }
}

// ------------------------------------------------------------------------------------------
// launchers

static int grid_for(long long items, int threads, int cap) {
    long long gsz = (items + threads - 1) / threads;
    if (gsz < 1) gsz = 1;
    if (gsz > cap) gsz = cap;
    return (int)gsz;
}

cudaError_t launch_plan_materialize_batch(const Geom &g, const DevState &s, const MatEntry *ents_dev,
                                          const SmallMat &small, int n, int total_pieces, long long clock,
                                          cudaStream_t st) {
    plan_materialize_kernel<<<grid_for(total_pieces, 256, 64), 256, 0, st>>>(g, s, ents_dev, small, n, total_pieces,
                                                                              clock);
    return cudaGetLastError();
}
cudaError_t launch_plan_materialize(const Geom &g, const DevState &s, int ctx, long long t0, long long t1, char *dst,
                                    long long clock, cudaStream_t st, int table_j0) {
    SmallMat one{};
    one.e[0].dst = dst; one.e[0].t0 = t0; one.e[0].t1 = t1; one.e[0].ctx = ctx; one.e[0].table_j0 = table_j0;
    return launch_plan_materialize_batch(g, s, nullptr, one, 1, (int)((t1 - 1) / g.BS - t0 / g.BS + 1), clock, st);
}
cudaError_t launch_plan_import_batch(const Geom &g, const DevState &s, const ImpEntry *ents_dev, const SmallImp &small,
                                     int n, int total_blocks, long long clock, cudaStream_t st) {
    plan_import_kernel<<<1, PLAN_THREADS, 0, st>>>(g, s, ents_dev, small, n, total_blocks, clock);
    return cudaGetLastError();
}
cudaError_t launch_plan_import(const Geom &g, const DevState &s, int ctx, long long n, const char *src,
                               long long clock, cudaStream_t st) {
    SmallImp one{};
    one.e[0].src = src; one.e[0].n = n; one.e[0].ctx = ctx;
    return launch_plan_import_batch(g, s, nullptr, one, 1, (int)((n + g.BS - 1) / g.BS), clock, st);
}
cudaError_t launch_fork(const Geom &g, const DevState &s, int parent, long long T, int k, const int *children_dev,
                        const SmallInts &small, long long clock, cudaStream_t st) {
    const long long nblk = (T + g.BS - 1) / g.BS;
    fork_kernel<<<grid_for(nblk * k, 256, 148), 256, 0, st>>>(g, s, parent, T, k, children_dev, small, clock);
    return cudaGetLastError();
}
cudaError_t launch_plan_append(const Geom &g, const DevState &s, const AppendEntry *entries_dev,
                               const SmallAppend &small, int n, int total_slots, int max_batch, int dry_run,
                               long long clock, cudaStream_t st) {
    plan_append_kernel<<<1, PLAN_THREADS, 0, st>>>(g, s, entries_dev, small, n, total_slots, max_batch, dry_run,
                                                   clock);
    return cudaGetLastError();
}
cudaError_t launch_plan_compose(const Geom &g, const DevState &s, const ComposeSeg *segs_dev, const SmallCompose &small,
                                int m, int total_work, int total_fresh, int total_slots, long long clock,
                                cudaStream_t st) {
    plan_compose_kernel<<<1, PLAN_THREADS, 0, st>>>(g, s, segs_dev, small, m, total_work, total_fresh, total_slots,
                                                    clock);
    return cudaGetLastError();
}
cudaError_t launch_evict(const Geom &g, const DevState &s, const EvictArgs *args_dev, const SmallInts &small, int n,
                         int total, long long clock, int *n_launches, cudaStream_t st) {
    const unsigned long long stamp = (unsigned long long)clock << 32;
    if (total <= EVICT_FUSED_MAX) {
        *n_launches = 1;
        evict_fused_kernel<<<1, PLAN_THREADS, 0, st>>>(g, s, args_dev, small, n, total, stamp);
        return cudaGetLastError();
    }
    if (!args_dev) return cudaErrorInvalidValue;  // the grid path reads its records from memory
    *n_launches = 4;
    const int n_tiles = (total + EVICT_TILE - 1) / EVICT_TILE;
    evict_release_kernel<<<grid_for(total, 256, 148), 256, 0, st>>>(g, s, args_dev, n, total, stamp);
    evict_count_kernel<<<n_tiles, PLAN_THREADS, 0, st>>>(g, s, args_dev, n, total, stamp, s.tile_count);
    evict_scan_kernel<<<1, PLAN_THREADS, 0, st>>>(g, s, args_dev, n, n_tiles, s.tile_count);
    evict_scatter_kernel<<<n_tiles, PLAN_THREADS, 0, st>>>(g, s, args_dev, n, total, stamp, s.tile_count);
    return cudaGetLastError();
}

cudaError_t launch_export_catalog(const Geom &g, const DevState &s, const aaf_kv_catalog_cols &cols, int n_states,
                                  long long n_block_rows, cudaStream_t st) {
    export_states_kernel<<<1, PLAN_THREADS, 0, st>>>(g, s, cols);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || n_block_rows == 0) return e;
    export_blocks_kernel<<<grid_for(n_block_rows, 256, 1184), 256, 0, st>>>(g, s, cols, n_states, n_block_rows);
    return cudaGetLastError();
}

cudaError_t launch_evict_to_budget(const Geom &g, const DevState &s, double alpha, double beta, double gamma,
                                   long long budget_blocks, long long clock, int *result, cudaStream_t st) {
    evict_to_budget_kernel<<<1, PLAN_THREADS, 0, st>>>(g, s, alpha, beta, gamma, budget_blocks, clock, result);
    return cudaGetLastError();
}

}  // namespace aafkv
