// Internal declarations shared by the translation units of libaafkv.so.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "aaf_kv.h"

namespace aafkv {

// One copy, described once for all (layer, K/V) planes:
//   plane (l, kv):  src + l * src_sl + kv * src_skv  ->  dst + l * dst_sl + kv * dst_skv,  nbytes bytes,
// optionally followed by a second part from the same operand: nbytes2 bytes from src + src2_off (same
// plane strides) that land directly behind the first part, at dst + nbytes.  The second part lets a
// destination block that is filled from two source blocks (the shifted copy of a compose) be one unit of
// work with one contiguous store.  For a pool operand the strides are (layer_stride, run); for an
// n-token transfer buffer they are (2 * n * row, n * row).  nbytes and nbytes2 are multiples of row
// (hence of 16) and nbytes + nbytes2 <= run; nbytes == 0 marks an unused slot.
struct __align__(16) Piece {
    const char *src;
    char *dst;
    long long src_sl, src_skv;
    long long dst_sl, dst_skv;
    unsigned int nbytes;
    unsigned int nbytes2;
    long long src2_off;
};
static_assert(sizeof(Piece) == 64, "Piece must be 64 bytes");

// Device-resident control block at the start of the workspace.
struct DevCtl {
    unsigned long long head;   // ring counters: free = tail - head
    unsigned long long tail;
    int status;                // sticky: first AAF_ERR_CORRUPT / AAF_ERR_TIMEOUT seen by a kernel
    int status_detail;
    unsigned long long payload_bytes;  // bytes moved by copy kernels (one direction)
    unsigned long long cow_count;
    long long peak_live;
    unsigned long long probe_need;     // dry-run result of the append planner
    unsigned int one;                  // constant 1: source of the host-visible chunk completion flags
    unsigned int pad32;
    unsigned long long evict_tail0;    // ring tail before the current large evict (read by its scatter kernel)
    // work distribution of the copy engines: CTAs draw unit tickets from copy_ticket; the last CTA to leave
    // (counted in copy_done) sets both back to 0, so every launch starts from 0 without a host-side reset
    unsigned long long copy_ticket;
    unsigned int copy_done;
    unsigned int pad32b;
    unsigned long long pad[5];
};
static_assert(sizeof(DevCtl) == 128, "DevCtl layout");

struct Geom {
    int L, H, D, BS, E, NB, max_ctx, max_blk;
    long long row, run, layer_stride;
    char *pool;
};

// Device views of the workspace.
struct DevState {
    DevCtl *ctl;
    int *refcount;   // [NB]
    int *ring;       // [NB]
    unsigned long long *last_pos;  // [NB] evict marks: (clock << 32) | last flattened position of the block
    int *tables;     // [max_ctx][max_blk]
    Piece *pieces;   // [max_pieces]
    int *scratch;    // [3 * max_batch] per-batch scratch of the append planner
    int *tile_count; // [max_ctx * max_blk / 8192 + 2] per-tile counts / offsets of a large evict
    // metadata catalog per handle (App. A.2): tokens (-1 = free handle), reads by other states, last access
    long long *cat_len;
    unsigned long long *cat_reuse;
    long long *cat_last;
    double *cat_score;  // scratch of the scored eviction
    // lineage per handle: how the state was produced (1 buffer, 2 fork, 3 merge), from which handle, when
    int *cat_origin;
    int *cat_parent;
    long long *cat_born;
    long long *cat_parent_born;
};

// ---- per-call argument records (written by the host into pinned memory, read by planners)
struct AppendEntry {      // 32 bytes
    const char *src;      // device payload [L][2][n_new][row]
    long long T;          // tokens before the append
    int ctx;
    int n_new;
    int piece_off;        // first piece slot of this entry (slot 0 = COW piece)
    int pad;
};
struct ComposeSeg {       // 56 bytes; one per segment of every merge of a batch
    long long T;          // tokens of the segment
    long long off;        // token offset of the segment in its result
    int ctx;
    int mode;             // 0 = share (aligned), 1 = copy
    int share_tail;       // share mode: 1 = partial tail shared by reference (last segment of its result)
    int work_off;         // first flattened work item of the segment (over the whole batch)
    int fresh_start;      // rank (from ring head, over the whole batch) of the first fresh block the segment allocates
    int piece_off;        // first piece slot of the segment (over the whole batch)
    int dst_tbl_start;    // share mode: first result-table index written
    int out_ctx;          // handle of the result this segment belongs to
    int out_index;        // which result of the batch (its logical clock is the call's clock + out_index)
    int first_ctx;        // last segment of a result only: handle of the result's first segment, else -1
};
static_assert(sizeof(ComposeSeg) == 56, "ComposeSeg layout");
struct MatEntry {         // 40 bytes; one token range of one context gathered into one transfer buffer
    char *dst;            // device transfer buffer of t1 - t0 tokens
    long long t0, t1;     // token range
    int ctx;
    int piece_off;        // first piece slot of the entry: one piece per block of the range
    int out_index;        // position in the batch (its logical clock is the call's clock + out_index)
    int table_j0;         // table position held by the first entry of the context's table row (0 for a pool)
};
struct ImpEntry {         // 32 bytes; one transfer buffer registered as one new context
    const char *src;      // device transfer buffer of n tokens
    long long n;
    int ctx;              // handle of the new context
    int block_off;        // rank (from the ring head, over the batch) of its first block = its first piece slot
    int out_index;
    int pad;
};
struct EvictArgs {        // followed by int ctx[n], int ent_off[n + 1]
    int n;
    int total;
};
// Small batches travel as kernel parameters instead of through the pinned argument ring: the kernel then starts
// without a read across PCIe and the host records no event for the ring slot.
constexpr int SMALL_ARGS = 16;
struct SmallInts {        // fork: children[k]; evict: ctx[n] followed by ent_off[n + 1]
    int v[2 * SMALL_ARGS + 1];
};
constexpr int SMALL_RECORDS = 8;   // append entries / compose segments that travel as kernel parameters
struct SmallAppend {
    AppendEntry e[SMALL_RECORDS];
};
struct SmallCompose {
    ComposeSeg s[SMALL_RECORDS];
};
struct SmallMat {
    MatEntry e[SMALL_RECORDS];
};
struct SmallImp {
    ImpEntry e[SMALL_RECORDS];
};

// ---- launchers (each returns cudaGetLastError() of its launches)
// `clock` is the logical clock of the call (count of successful state-touching calls); planners stamp
// it into the catalog.  A DevState without catalog arrays (cat_len == nullptr) skips the stamping.
cudaError_t launch_plan_materialize(const Geom &g, const DevState &s, int ctx, long long t0, long long t1, char *dst,
                                    long long clock, cudaStream_t st, int table_j0 = 0);
// batched forms: ents_dev == nullptr means the n <= SMALL_RECORDS records are in `small`; entry i is stamped clock + i
cudaError_t launch_plan_materialize_batch(const Geom &g, const DevState &s, const MatEntry *ents_dev,
                                          const SmallMat &small, int n, int total_pieces, long long clock,
                                          cudaStream_t st);
cudaError_t launch_plan_import_batch(const Geom &g, const DevState &s, const ImpEntry *ents_dev, const SmallImp &small,
                                     int n, int total_blocks, long long clock, cudaStream_t st);
cudaError_t launch_plan_import(const Geom &g, const DevState &s, int ctx, long long n, const char *src,
                               long long clock, cudaStream_t st);
// children_dev == nullptr: the k <= SMALL_ARGS children are in `small`
cudaError_t launch_fork(const Geom &g, const DevState &s, int parent, long long T, int k, const int *children_dev,
                        const SmallInts &small, long long clock, cudaStream_t st);
// entries_dev / segs_dev == nullptr: the n (m) <= SMALL_RECORDS records are in `small`
cudaError_t launch_plan_append(const Geom &g, const DevState &s, const AppendEntry *entries_dev,
                               const SmallAppend &small, int n, int total_slots, int max_batch, int dry_run,
                               long long clock, cudaStream_t st);
// `clock` is the logical clock of the batch's first merge; merge i of the batch is stamped clock + i
cudaError_t launch_plan_compose(const Geom &g, const DevState &s, const ComposeSeg *segs_dev, const SmallCompose &small,
                                int m, int total_work, int total_fresh, int total_slots, long long clock,
                                cudaStream_t st);
// args_dev == nullptr: the n <= SMALL_ARGS contexts and their entry offsets are in `small` (total <= 32768)
cudaError_t launch_evict(const Geom &g, const DevState &s, const EvictArgs *args_dev, const SmallInts &small, int n,
                         int total, long long clock, int *n_launches, cudaStream_t st);
// Scored eviction (Alg. KV-Evict): result[0] = number of victims, result[1] = free blocks afterwards,
// result[2..] = victims in eviction order; `result` is host memory the device can write.
cudaError_t launch_evict_to_budget(const Geom &g, const DevState &s, double alpha, double beta, double gamma,
                                   long long budget_blocks, long long clock, int *result, cudaStream_t st);
// launch shapes of the copy engines for one pool geometry (see copy_tuning_init)
struct CopyTuning {
    int bulk_chunk, bulk_stages, bulk_ctas, bulk_l2;
    int vec_unroll, vec_ctas;
    int warp_unroll, warp_ctas;
    int auto_engine;               // 0 = choose per launch, else forced engine
    long long auto_bulk_min_piece; // AUTO: mean piece size from which the bulk engine is used
};
cudaError_t copy_tuning_init(long long run, CopyTuning *t);
cudaError_t launch_expire_wait(const DevState &s, long long limit_cycles, cudaStream_t st);
cudaError_t launch_copy(int engine, const CopyTuning &t, const Geom &g, const DevState &s, int n_slots, int plane0,
                        int n_planes, long long avg_piece_bytes, int sm_count, cudaStream_t st);

// columnar catalog export: state rows + offsets by a prefix scan (one CTA), block rows by a grid
cudaError_t launch_export_catalog(const Geom &g, const DevState &s, const aaf_kv_catalog_cols &cols, int n_states,
                                  long long n_block_rows, cudaStream_t st);

}  // namespace aafkv
