// Host side of libaafkv.so: the C ABI declared in include/aaf_kv.h.
//
// The host object mirrors only what it can know without asking the device: which handles are
// live and how many tokens each holds (every length is a function of the call sequence), plus a
// guaranteed lower bound of the free-block count.  Block ids, reference counts and the ring live
// on the device.  A call validates everything against the mirror, writes its argument records
// into a pinned ring the planners read directly, and launches: planner kernel(s) then the copy
// engine.  Planners run on a library-owned metadata stream and copies on the caller's stream, joined
// by events and two alternating piece buffers, so the planner of the next operator runs while the
// copy of the current one is still streaming.  The device's free count is read back (one synchronising 16-byte copy) only when the
// lower bound cannot prove that a call fits, so out-of-blocks is reported exactly and
// synchronously without a sync on the common path.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include "aafkv_internal.h"

// Profiler ranges: built with -DAAFKV_NVTX every C-ABI operator call is an NVTX range named after the entry
// point (header-only NVTX 3, no extra library); without the switch the macro is empty.
#ifdef AAFKV_NVTX
#include <nvtx3/nvToolsExt.h>
namespace {
struct ScopedRange {
    explicit ScopedRange(const char *name) { nvtxRangePushA(name); }
    ~ScopedRange() { nvtxRangePop(); }
};
}  // namespace
#define AAF_RANGE(name) ScopedRange aaf_range_(name)
#else
#define AAF_RANGE(name) do { } while (0)
#endif

using namespace aafkv;

namespace {

constexpr int ARG_SLOTS = 16;
constexpr size_t ARG_RECORD_BYTES = 64;  // per-record room in a slot of the pinned argument ring
static_assert(sizeof(ComposeSeg) <= ARG_RECORD_BYTES && sizeof(AppendEntry) <= ARG_RECORD_BYTES &&
                  sizeof(MatEntry) <= ARG_RECORD_BYTES && sizeof(ImpEntry) <= ARG_RECORD_BYTES,
              "argument records must fit their room in the pinned ring");

struct Layout {
    size_t ctl, refcount, ring, last_pos, tables, pieces, scratch, cat_len, cat_reuse, cat_last, cat_score, cat_origin, cat_parent, cat_born, cat_parent_born, tile_count, total;
    int max_pieces, max_batch;
};

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool geometry_ok(const aaf_kv_pool_desc *d) {
    if (!d || d->struct_size != sizeof(aaf_kv_pool_desc) || d->abi_version != AAF_KV_ABI_VERSION) return false;
    if (d->n_layers < 1 || d->n_kv_heads < 1 || d->head_dim < 1 || d->block_size < 1 || d->elt_bytes < 1) return false;
    if (d->n_blocks < 1 || d->max_ctx < 1 || d->max_blocks_per_ctx < 1 || d->max_batch < 0) return false;
    const long long row = (long long)d->n_kv_heads * d->head_dim * d->elt_bytes;
    if (row % 16 != 0) return false;
    if (row * d->block_size > (1ll << 30)) return false;  // a run must fit the 32-bit piece size
    if ((long long)d->max_ctx * d->max_blocks_per_ctx >= (1ll << 31)) return false;  // flattened entry indices are ints
    return true;
}

Layout make_layout(const aaf_kv_pool_desc *d) {
    Layout L{};
    L.max_batch = d->max_batch > 0 ? d->max_batch : 1024;
    L.max_pieces = 2 * d->max_blocks_per_ctx + 4 * L.max_batch + 64;
    size_t off = 0;
    L.ctl = off; off = align_up(off + sizeof(DevCtl), 256);
    L.refcount = off; off = align_up(off + sizeof(int) * (size_t)d->n_blocks, 256);
    L.ring = off; off = align_up(off + sizeof(int) * (size_t)d->n_blocks, 256);
    L.last_pos = off; off = align_up(off + sizeof(unsigned long long) * (size_t)d->n_blocks, 256);
    L.tables = off; off = align_up(off + sizeof(int) * (size_t)d->max_ctx * d->max_blocks_per_ctx, 256);
    L.pieces = off; off = align_up(off + 2 * sizeof(Piece) * (size_t)L.max_pieces, 256);  // two alternating buffers
    L.scratch = off; off = align_up(off + sizeof(int) * 3 * (size_t)L.max_batch, 256);
    L.cat_len = off; off = align_up(off + sizeof(long long) * (size_t)d->max_ctx, 256);
    L.cat_reuse = off; off = align_up(off + sizeof(long long) * (size_t)d->max_ctx, 256);
    L.cat_last = off; off = align_up(off + sizeof(long long) * (size_t)d->max_ctx, 256);
    L.cat_score = off; off = align_up(off + sizeof(double) * (size_t)d->max_ctx, 256);
    L.cat_origin = off; off = align_up(off + sizeof(int) * (size_t)d->max_ctx, 256);
    L.cat_parent = off; off = align_up(off + sizeof(int) * (size_t)d->max_ctx, 256);
    L.cat_born = off; off = align_up(off + sizeof(long long) * (size_t)d->max_ctx, 256);
    L.cat_parent_born = off; off = align_up(off + sizeof(long long) * (size_t)d->max_ctx, 256);
    L.tile_count = off;
    off = align_up(off + sizeof(int) * ((size_t)d->max_ctx * d->max_blocks_per_ctx / 8192 + 2), 256);
    L.total = off;
    return L;
}

struct TimedLaunch {
    cudaEvent_t start, stop;
    int cls;
};

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

}  // namespace

struct aaf_kv_pool {
    aaf_kv_pool_desc desc;
    Geom g;
    DevState s;
    Layout lay;
    int device = 0, sm_count = 148;
    bool broken = false;  // a CUDA call failed after device state had changed: every later call returns AAF_ERR_CUDA
    CopyTuning tuning{};
    std::vector<long long> len;  // tokens per handle, -1 = free
    int live_ctx = 0;
    long long free_lb = 0;       // guaranteed lower bound of the device's free-block count
    long long clock = 0;         // logical clock: successful state-touching calls so far
    int *result = nullptr;       // pinned, device-writable: result of the scored eviction (max_ctx + 2 ints)
    cudaStream_t last_stream = nullptr;  // the caller's stream of the most recent call (copies run there)
    // Metadata kernels run on their own stream: they touch tables, reference counts, the ring and the piece
    // buffers only, never payload, so the planner of operator i+1 can run while the copy of operator i is
    // still streaming.  Two piece buffers alternate; events order planner -> copy and copy -> buffer reuse.
    cudaStream_t meta_stream = nullptr;
    cudaEvent_t plan_done[2] = {}, copy_done[2] = {};
    int next_buf = 0;
    // Copy launches of a pool share the ticket counter of its control block, so they must never overlap on the
    // device.  Calls on one stream are ordered anyway; when a call arrives on ANOTHER stream than the previous
    // copy launch, that stream is made to wait for the previous operator's last copy launch first.
    cudaStream_t last_copy_stream = nullptr;
    cudaEvent_t last_copy_event = nullptr;
    // pinned argument ring
    char *args = nullptr;
    size_t slot_bytes = 0;
    int next_slot = 0;
    cudaEvent_t slot_ev[ARG_SLOTS] = {};
    bool slot_busy[ARG_SLOTS] = {};
    int cur_slot = -1;
    // knobs and counters
    int engine = AAF_ENGINE_AUTO;
    bool timing = false;
    long long copy_launches[AAF_OP_CLASSES] = {};
    long long meta_launches = 0;
    double copy_ms[AAF_OP_CLASSES] = {};
    long long timed_launches[AAF_OP_CLASSES] = {};
    std::vector<TimedLaunch> pending;
    std::vector<cudaEvent_t> spare_events;
    // chunked host transfers: a second stream for the PCIe copies and ordering events
    // chunked / host-buffer transfers: one library-owned stream per PCIe direction, so that uploads queue behind
    // each other in call order (the first one needed arrives first) while a download runs beside them
    cudaStream_t xfer_stream = nullptr;     // device -> host (aaf_kv_materialize_host_chunked)
    cudaStream_t upload_stream = nullptr;   // host -> device (aaf_kv_import_host_chunked, aaf_kv_append_host)
    // the scatter launches of the last upload call per staging role have read their staging buffer
    cudaEvent_t upload_reader_done = nullptr, import_reader_done = nullptr;
    bool upload_reader_pending = false, import_reader_pending = false;
    std::vector<cudaEvent_t> order_events;  // created on demand, reused round-robin
    size_t next_order_event = 0;
};

namespace {

long long nblk_of(const aaf_kv_pool *p, long long tokens) { return (tokens + p->g.BS - 1) / p->g.BS; }
bool is_live(const aaf_kv_pool *p, int c) { return c >= 0 && c < p->g.max_ctx && p->len[c] >= 0; }
// A CUDA runtime call failed after a planner may already have changed the device's metadata: the host mirror
// can no longer be trusted, so the pool refuses all further work.
int broke(aaf_kv_pool *p) {
    p->broken = true;
    return AAF_ERR_CUDA;
}
bool aligned16(const void *q) { return q && (reinterpret_cast<uintptr_t>(q) & 15u) == 0; }
long long bpt_of(const aaf_kv_pool *p) { return 2ll * p->g.L * p->g.row; }

// next pinned argument slot; waits (host side) until the device has finished reading its last use
char *acquire_args(aaf_kv_pool *p) {
    const int sl = p->next_slot;
    p->next_slot = (sl + 1) % ARG_SLOTS;
    if (p->slot_busy[sl]) {
        cudaEventSynchronize(p->slot_ev[sl]);
        p->slot_busy[sl] = false;
    }
    p->cur_slot = sl;
    return p->args + (size_t)sl * p->slot_bytes;
}
void release_args(aaf_kv_pool *p, cudaStream_t st) {
    if (p->cur_slot < 0) return;
    cudaEventRecord(p->slot_ev[p->cur_slot], st);
    p->slot_busy[p->cur_slot] = true;
    p->cur_slot = -1;
}

// exact free-block count: synchronises the stream and reads the ring counters
int refresh_free(aaf_kv_pool *p, cudaStream_t st) {
    (void)st;
    unsigned long long ht[2];
    if (cudaStreamSynchronize(p->meta_stream) != cudaSuccess) return AAF_ERR_CUDA;  // the counters are metadata
    if (cudaMemcpy(ht, p->s.ctl, sizeof(ht), cudaMemcpyDeviceToHost) != cudaSuccess) return AAF_ERR_CUDA;
    p->free_lb = (long long)(ht[1] - ht[0]);
    return AAF_OK;
}
int ensure_free(aaf_kv_pool *p, long long need, cudaStream_t st) {
    if (p->free_lb >= need) return AAF_OK;
    const int rc = refresh_free(p, st);
    if (rc != AAF_OK) return rc;
    return p->free_lb >= need ? AAF_OK : AAF_ERR_OOM_BLOCKS;
}

int smallest_free_ctx(const aaf_kv_pool *p, int start = 0) {
    for (int c = start; c < p->g.max_ctx; ++c)
        if (p->len[c] < 0) return c;
    return -1;
}

cudaEvent_t get_event(aaf_kv_pool *p) {
    if (!p->spare_events.empty()) {
        cudaEvent_t e = p->spare_events.back();
        p->spare_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

void drain_timing(aaf_kv_pool *p) {
    for (auto &t : p->pending) {
        float ms = 0.f;
        if (cudaEventSynchronize(t.stop) == cudaSuccess && cudaEventElapsedTime(&ms, t.start, t.stop) == cudaSuccess) {
            p->copy_ms[t.cls] += ms;
            p->timed_launches[t.cls] += 1;
        }
        p->spare_events.push_back(t.start);
        p->spare_events.push_back(t.stop);
    }
    p->pending.clear();
}

// copy-engine launch for one operator class over planes [plane0, plane0 + n_planes)
struct PlanSlot {
    DevState view;  // device state whose `pieces` is the buffer this operator plans into
    int buf;
};

// Before a planner: pick the next piece buffer and make the metadata stream wait until the copy launch
// that last read that buffer has finished.
PlanSlot begin_plan(aaf_kv_pool *p) {
    PlanSlot ps;
    ps.buf = p->next_buf;
    ps.view = p->s;
    ps.view.pieces = p->s.pieces + (size_t)ps.buf * (size_t)p->lay.max_pieces;
    cudaStreamWaitEvent(p->meta_stream, p->copy_done[ps.buf], 0);
    return ps;
}
// After the planner: the caller's stream (where the copy runs) waits for it.
bool end_plan(aaf_kv_pool *p, const PlanSlot &ps, cudaStream_t st) {
    return cudaEventRecord(p->plan_done[ps.buf], p->meta_stream) == cudaSuccess &&
           cudaStreamWaitEvent(st, p->plan_done[ps.buf], 0) == cudaSuccess;
}
// After the operator's last copy launch: mark the buffer's readers done and switch buffers.
void end_copy(aaf_kv_pool *p, const PlanSlot &ps, cudaStream_t st) {
    cudaEventRecord(p->copy_done[ps.buf], st);
    p->last_copy_stream = st;
    p->last_copy_event = p->copy_done[ps.buf];
    p->next_buf ^= 1;
}

int run_copy(aaf_kv_pool *p, const PlanSlot &ps, int cls, int n_slots, long long payload_tokens, cudaStream_t st,
             int piece0 = 0) {
    const int plane0 = 0, n_planes = 2 * p->g.L;
    DevState view = ps.view;
    view.pieces += piece0;  // a launch may cover a sub-range of the planned pieces (chunked transfers)
    const long long avg_piece = n_slots > 0 ? payload_tokens * p->g.row / n_slots : 0;
    if (n_slots <= 0) return AAF_OK;
    if (p->last_copy_event && st != p->last_copy_stream) {  // a different stream: serialise behind the last copy launch
        if (cudaStreamWaitEvent(st, p->last_copy_event, 0) != cudaSuccess) return broke(p);
        p->last_copy_stream = st;  // the wait is queued; later launches of this operator need not repeat it
    }
    TimedLaunch t{};
    if (p->timing) {
        t.start = get_event(p);
        t.stop = get_event(p);
        t.cls = cls;
        cudaEventRecord(t.start, st);
    }
    const cudaError_t e = launch_copy(p->engine, p->tuning, p->g, view, n_slots, plane0, n_planes, avg_piece, p->sm_count, st);
    if (p->timing) {
        cudaEventRecord(t.stop, st);
        p->pending.push_back(t);
        if (p->pending.size() > 4096) drain_timing(p);
    }
    p->copy_launches[cls] += 1;
    return e == cudaSuccess ? AAF_OK : broke(p);
}

void fill_desc(const aaf_kv_pool *p, aaf_kv_xfer_desc *d, long long pos_start, long long n) {
    d->model_id = p->desc.model_id;
    d->config_hash = p->desc.config_hash;
    d->n_layers = p->g.L; d->n_kv_heads = p->g.H; d->head_dim = p->g.D; d->elt_bytes = p->g.E;
    d->pos_start = pos_start;
    d->n_tokens = n;
}

// Compat(S_a, S_b) = 1[M_a = M_b] * 1[Theta_a = Theta_b] (Sec. 3.2); positions are carried, not enforced
bool compatible(const aaf_kv_pool *p, const aaf_kv_xfer_desc *d) {
    return d->model_id == p->desc.model_id && d->config_hash == p->desc.config_hash && d->n_layers == p->g.L &&
           d->n_kv_heads == p->g.H && d->head_dim == p->g.D && d->elt_bytes == p->g.E;
}

int materialize_impl(aaf_kv_pool *p, aaf_ctx_t ctx, int64_t t0, int64_t t1, void *dst_dev, size_t dst_bytes,
                     aaf_kv_xfer_desc *out_desc, cudaStream_t st) {
    if (!is_live(p, ctx)) return AAF_ERR_BAD_CTX;
    if (!aligned16(dst_dev) || t0 < 0 || t0 >= t1 || t1 > p->len[ctx]) return AAF_ERR_INVALID_ARG;
    const long long n = t1 - t0;
    if ((unsigned long long)dst_bytes < (unsigned long long)(n * bpt_of(p))) return AAF_ERR_DST_TOO_SMALL;
    p->last_stream = st;
    const PlanSlot ps = begin_plan(p);
    if (launch_plan_materialize(p->g, ps.view, ctx, t0, t1, static_cast<char *>(dst_dev), p->clock + 1,
                                p->meta_stream) != cudaSuccess ||
        !end_plan(p, ps, st))
        return broke(p);
    p->clock += 1;
    p->meta_launches += 1;
    const int n_slots = (int)((t1 - 1) / p->g.BS - t0 / p->g.BS + 1);
    const int rc = run_copy(p, ps, AAF_OP_MATERIALIZE, n_slots, n, st);
    end_copy(p, ps, st);
    if (rc == AAF_OK && out_desc) fill_desc(p, out_desc, t0, n);
    return rc;
}

int import_impl(aaf_kv_pool *p, const void *src_dev, const aaf_kv_xfer_desc *desc, aaf_ctx_t *out_ctx,
                cudaStream_t st, const void *src_host) {
    if (!desc || !out_ctx || !aligned16(src_dev)) return AAF_ERR_INVALID_ARG;
    if (!compatible(p, desc)) return AAF_ERR_INCOMPAT;
    const long long n = desc->n_tokens;
    if (n < 1) return AAF_ERR_INVALID_ARG;
    const long long nb = nblk_of(p, n);
    if (nb > p->g.max_blk) return AAF_ERR_TOO_LONG;
    const int c = smallest_free_ctx(p);
    if (c < 0) return AAF_ERR_OOM_CTX;
    const int rc0 = ensure_free(p, nb, st);
    if (rc0 != AAF_OK) return rc0;
    p->last_stream = st;
    if (src_host) {
        if (cudaMemcpyAsync(const_cast<void *>(src_dev), src_host, (size_t)(n * bpt_of(p)), cudaMemcpyHostToDevice,
                            st) != cudaSuccess)
            return broke(p);
    }
    const PlanSlot ps = begin_plan(p);
    if (launch_plan_import(p->g, ps.view, c, n, static_cast<const char *>(src_dev), p->clock + 1, p->meta_stream) !=
            cudaSuccess ||
        !end_plan(p, ps, st))
        return broke(p);
    p->clock += 1;
    p->meta_launches += 1;
    p->free_lb -= nb;
    p->len[c] = n;
    p->live_ctx += 1;
    *out_ctx = c;
    const int rc = run_copy(p, ps, AAF_OP_IMPORT, (int)nb, n, st);
    end_copy(p, ps, st);
    return rc;
}

cudaEvent_t order_event(aaf_kv_pool *p) {
    if (p->order_events.size() < 64) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        p->order_events.push_back(e);
        return e;
    }
    cudaEvent_t e = p->order_events[p->next_order_event];
    p->next_order_event = (p->next_order_event + 1) % p->order_events.size();
    return e;
}

bool ensure_xfer_stream(aaf_kv_pool *p) {
    if (p->xfer_stream) return true;
    return cudaStreamCreateWithFlags(&p->xfer_stream, cudaStreamNonBlocking) == cudaSuccess;
}
bool ensure_upload_stream(aaf_kv_pool *p) {
    if (!p->upload_stream && cudaStreamCreateWithFlags(&p->upload_stream, cudaStreamNonBlocking) != cudaSuccess)
        return false;
    if (!p->upload_reader_done &&
        cudaEventCreateWithFlags(&p->upload_reader_done, cudaEventDisableTiming) != cudaSuccess)
        return false;
    if (!p->import_reader_done &&
        cudaEventCreateWithFlags(&p->import_reader_done, cudaEventDisableTiming) != cudaSuccess)
        return false;
    return true;
}

// column slab [col0, col0 + cnt) tokens of an n-token transfer buffer: 2L rows of cnt*row bytes, pitch n*row
cudaError_t copy_slab(aaf_kv_pool *p, char *dst, const char *src, long long n, long long col0, long long cnt,
                      cudaMemcpyKind kind, cudaStream_t st) {
    const size_t pitch = (size_t)(n * p->g.row);
    return cudaMemcpy2DAsync(dst + col0 * p->g.row, pitch, src + col0 * p->g.row, pitch, (size_t)(cnt * p->g.row),
                             (size_t)(2 * p->g.L), kind, st);
}

}  // namespace

// =============================================================================================
extern "C" {

size_t aaf_kv_pool_workspace_bytes(const aaf_kv_pool_desc *desc) {
    if (!geometry_ok(desc)) return 0;
    return make_layout(desc).total;
}

int aaf_kv_pool_create(const aaf_kv_pool_desc *desc, aaf_kv_pool **out) {
    AAF_RANGE("aaf_kv_pool_create");
    if (!out) return AAF_ERR_INVALID_ARG;
    *out = nullptr;
    if (!geometry_ok(desc)) return AAF_ERR_INVALID_ARG;
    const Layout lay = make_layout(desc);
    const long long row = (long long)desc->n_kv_heads * desc->head_dim * desc->elt_bytes;
    const long long run = row * desc->block_size;
    if (!aligned16(desc->pool_base) || !desc->workspace || (reinterpret_cast<uintptr_t>(desc->workspace) & 255u))
        return AAF_ERR_INVALID_ARG;
    if (desc->layer_stride_bytes % 16 != 0 || desc->layer_stride_bytes < (size_t)(2 * run * desc->n_blocks))
        return AAF_ERR_INVALID_ARG;
    if (desc->workspace_bytes < lay.total) return AAF_ERR_INVALID_ARG;
    std::vector<int> ring((size_t)desc->n_blocks);
    if (desc->free_order) {
        std::vector<char> seen((size_t)desc->n_blocks, 0);
        for (int i = 0; i < desc->n_blocks; ++i) {
            const int b = desc->free_order[i];
            if (b < 0 || b >= desc->n_blocks || seen[(size_t)b]) return AAF_ERR_INVALID_ARG;
            seen[(size_t)b] = 1;
            ring[(size_t)i] = b;
        }
    } else {
        for (int i = 0; i < desc->n_blocks; ++i) ring[(size_t)i] = i;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || desc->device < 0 || desc->device >= ndev) return AAF_ERR_CUDA;

    aaf_kv_pool *p = new (std::nothrow) aaf_kv_pool();
    if (!p) return AAF_ERR_INVALID_ARG;
    p->desc = *desc;
    p->desc.free_order = nullptr;
    p->lay = lay;
    p->device = desc->device;
    DeviceGuard guard(p->device);
    p->g.L = desc->n_layers; p->g.H = desc->n_kv_heads; p->g.D = desc->head_dim; p->g.BS = desc->block_size;
    p->g.E = desc->elt_bytes; p->g.NB = desc->n_blocks; p->g.max_ctx = desc->max_ctx;
    p->g.max_blk = desc->max_blocks_per_ctx;
    p->g.row = row; p->g.run = run; p->g.layer_stride = (long long)desc->layer_stride_bytes;
    p->g.pool = static_cast<char *>(desc->pool_base);
    char *ws = static_cast<char *>(desc->workspace);
    p->s.ctl = reinterpret_cast<DevCtl *>(ws + lay.ctl);
    p->s.refcount = reinterpret_cast<int *>(ws + lay.refcount);
    p->s.ring = reinterpret_cast<int *>(ws + lay.ring);
    p->s.last_pos = reinterpret_cast<unsigned long long *>(ws + lay.last_pos);
    p->s.tables = reinterpret_cast<int *>(ws + lay.tables);
    p->s.pieces = reinterpret_cast<Piece *>(ws + lay.pieces);
    p->s.scratch = reinterpret_cast<int *>(ws + lay.scratch);
    p->s.cat_len = reinterpret_cast<long long *>(ws + lay.cat_len);
    p->s.cat_reuse = reinterpret_cast<unsigned long long *>(ws + lay.cat_reuse);
    p->s.cat_last = reinterpret_cast<long long *>(ws + lay.cat_last);
    p->s.cat_score = reinterpret_cast<double *>(ws + lay.cat_score);
    p->s.cat_origin = reinterpret_cast<int *>(ws + lay.cat_origin);
    p->s.cat_parent = reinterpret_cast<int *>(ws + lay.cat_parent);
    p->s.cat_born = reinterpret_cast<long long *>(ws + lay.cat_born);
    p->s.cat_parent_born = reinterpret_cast<long long *>(ws + lay.cat_parent_born);
    p->s.tile_count = reinterpret_cast<int *>(ws + lay.tile_count);
    p->len.assign((size_t)desc->max_ctx, -1);
    p->free_lb = desc->n_blocks;

    bool ok = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device) == cudaSuccess;
    ok = ok && copy_tuning_init(p->g.run, &p->tuning) == cudaSuccess;
    p->slot_bytes = align_up(ARG_RECORD_BYTES * (size_t)lay.max_batch + 256, 256);
    ok = ok && cudaHostAlloc(reinterpret_cast<void **>(&p->args), p->slot_bytes * ARG_SLOTS, cudaHostAllocMapped) ==
                   cudaSuccess;
    for (int i = 0; ok && i < ARG_SLOTS; ++i)
        ok = cudaEventCreateWithFlags(&p->slot_ev[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&p->meta_stream, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < 2; ++i)
        ok = cudaEventCreateWithFlags(&p->plan_done[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&p->copy_done[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaHostAlloc(reinterpret_cast<void **>(&p->result), sizeof(int) * ((size_t)desc->max_ctx + 2),
                             cudaHostAllocMapped) == cudaSuccess;
    // device state: counters, reference counts 0, ring, evict scratch -1
    DevCtl ctl;
    memset(&ctl, 0, sizeof(ctl));
    ctl.tail = (unsigned long long)desc->n_blocks;
    ctl.one = 1u;
    ok = ok && cudaMemset(ws, 0, lay.tables) == cudaSuccess;
    ok = ok && cudaMemcpy(p->s.ctl, &ctl, sizeof(ctl), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(p->s.ring, ring.data(), sizeof(int) * ring.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemset(p->s.cat_len, 0xff, sizeof(long long) * (size_t)desc->max_ctx) == cudaSuccess;  // -1: free
    ok = ok && cudaMemset(p->s.cat_reuse, 0, lay.total - lay.cat_reuse) == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        aaf_kv_pool_destroy(p);
        return AAF_ERR_CUDA;
    }
    *out = p;
    return AAF_OK;
}

int aaf_kv_pool_destroy(aaf_kv_pool *p) {
    if (!p) return AAF_ERR_INVALID_ARG;
    DeviceGuard guard(p->device);
    if (p->meta_stream) cudaStreamSynchronize(p->meta_stream);
    if (p->last_stream || !p->pending.empty()) cudaStreamSynchronize(p->last_stream);
    for (auto &t : p->pending) {
        cudaEventDestroy(t.start);
        cudaEventDestroy(t.stop);
    }
    for (auto e : p->spare_events) cudaEventDestroy(e);
    if (p->xfer_stream) {
        cudaStreamSynchronize(p->xfer_stream);
        cudaStreamDestroy(p->xfer_stream);
    }
    if (p->upload_stream) {
        cudaStreamSynchronize(p->upload_stream);
        cudaStreamDestroy(p->upload_stream);
    }
    if (p->upload_reader_done) cudaEventDestroy(p->upload_reader_done);
    if (p->import_reader_done) cudaEventDestroy(p->import_reader_done);
    for (auto e : p->order_events) cudaEventDestroy(e);
    for (int i = 0; i < 2; ++i) {
        if (p->plan_done[i]) cudaEventDestroy(p->plan_done[i]);
        if (p->copy_done[i]) cudaEventDestroy(p->copy_done[i]);
    }
    if (p->meta_stream) cudaStreamDestroy(p->meta_stream);
    for (int i = 0; i < ARG_SLOTS; ++i)
        if (p->slot_ev[i]) cudaEventDestroy(p->slot_ev[i]);
    if (p->args) cudaFreeHost(p->args);
    if (p->result) cudaFreeHost(p->result);
    delete p;
    return AAF_OK;
}

int aaf_kv_materialize(aaf_kv_pool *p, aaf_ctx_t ctx, int64_t tok_begin, int64_t tok_end, void *dst_dev,
                       size_t dst_bytes, aaf_kv_xfer_desc *out_desc, void *stream) {
    AAF_RANGE("aaf_kv_materialize");
    if (!p) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    DeviceGuard guard(p->device);
    return materialize_impl(p, ctx, tok_begin, tok_end, dst_dev, dst_bytes, out_desc,
                            static_cast<cudaStream_t>(stream));
}

int aaf_kv_materialize_host(aaf_kv_pool *p, aaf_ctx_t ctx, int64_t tok_begin, int64_t tok_end, void *dst_host,
                            size_t dst_bytes, void *staging_dev, size_t staging_bytes, aaf_kv_xfer_desc *out_desc,
                            void *stream) {
    AAF_RANGE("aaf_kv_materialize_host");
    if (!p || !dst_host) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (is_live(p, ctx) && tok_begin >= 0 && tok_begin < tok_end &&
        (unsigned long long)dst_bytes < (unsigned long long)((tok_end - tok_begin) * bpt_of(p)))
        return AAF_ERR_DST_TOO_SMALL;
    const int rc = materialize_impl(p, ctx, tok_begin, tok_end, staging_dev, staging_bytes, out_desc, st);
    if (rc != AAF_OK) return rc;
    const size_t bytes = (size_t)((tok_end - tok_begin) * bpt_of(p));
    return cudaMemcpyAsync(dst_host, staging_dev, bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess ? AAF_OK
                                                                                                   : broke(p);
}

int aaf_kv_import(aaf_kv_pool *p, const void *src_dev, const aaf_kv_xfer_desc *desc, aaf_ctx_t *out_ctx,
                  void *stream) {
    AAF_RANGE("aaf_kv_import");
    if (!p) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    DeviceGuard guard(p->device);
    return import_impl(p, src_dev, desc, out_ctx, static_cast<cudaStream_t>(stream), nullptr);
}

int aaf_kv_materialize_batch(aaf_kv_pool *p, int32_t n, const aaf_ctx_t *ctxs, const int64_t *tok_begin,
                             const int64_t *tok_end, void *const *dst_dev, const size_t *dst_bytes,
                             aaf_kv_xfer_desc *out_descs, void *stream) {
    AAF_RANGE("aaf_kv_materialize_batch");
    if (!p || n < 1 || !ctxs || !tok_begin || !tok_end || !dst_dev || !dst_bytes) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    if (n > p->lay.max_batch) return AAF_ERR_TOO_MANY;
    long long slots = 0, tokens = 0;
    for (int i = 0; i < n; ++i) {
        if (!is_live(p, ctxs[i])) return AAF_ERR_BAD_CTX;
        const long long t0 = tok_begin[i], t1 = tok_end[i];
        if (!aligned16(dst_dev[i]) || t0 < 0 || t0 >= t1 || t1 > p->len[ctxs[i]]) return AAF_ERR_INVALID_ARG;
        if ((unsigned long long)dst_bytes[i] < (unsigned long long)((t1 - t0) * bpt_of(p))) return AAF_ERR_DST_TOO_SMALL;
        slots += (t1 - 1) / p->g.BS - t0 / p->g.BS + 1;
        tokens += t1 - t0;
    }
    if (slots > p->lay.max_pieces) return AAF_ERR_TOO_MANY;
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    // a small batch travels as kernel parameters, a large one through the pinned argument ring
    SmallMat small{};
    const bool by_value = n <= SMALL_RECORDS;
    MatEntry *ent = by_value ? small.e : reinterpret_cast<MatEntry *>(acquire_args(p));
    int off = 0;
    for (int i = 0; i < n; ++i) {
        MatEntry &e = ent[i];
        e.dst = static_cast<char *>(dst_dev[i]);
        e.t0 = tok_begin[i]; e.t1 = tok_end[i];
        e.ctx = ctxs[i]; e.piece_off = off; e.out_index = i; e.table_j0 = 0;
        off += (int)((e.t1 - 1) / p->g.BS - e.t0 / p->g.BS + 1);
    }
    const PlanSlot ps = begin_plan(p);
    const cudaError_t e = launch_plan_materialize_batch(p->g, ps.view, by_value ? nullptr : ent, small, n, (int)slots,
                                                        p->clock + 1, p->meta_stream);
    if (!by_value) release_args(p, p->meta_stream);
    if (e != cudaSuccess || !end_plan(p, ps, st)) return broke(p);
    p->clock += n;  // entry i of the batch is the call with clock + 1 + i
    p->meta_launches += 1;
    const int rc = run_copy(p, ps, AAF_OP_MATERIALIZE, (int)slots, tokens, st);
    end_copy(p, ps, st);
    if (rc == AAF_OK && out_descs)
        for (int i = 0; i < n; ++i) fill_desc(p, &out_descs[i], tok_begin[i], tok_end[i] - tok_begin[i]);
    return rc;
}

int aaf_kv_import_batch(aaf_kv_pool *p, int32_t n, const void *const *src_dev, const aaf_kv_xfer_desc *descs,
                        aaf_ctx_t *out_ctxs, void *stream) {
    AAF_RANGE("aaf_kv_import_batch");
    if (!p || n < 1 || !src_dev || !descs || !out_ctxs) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    if (n > p->lay.max_batch) return AAF_ERR_TOO_MANY;
    long long blocks = 0, tokens = 0;
    for (int i = 0; i < n; ++i) {
        if (!aligned16(src_dev[i])) return AAF_ERR_INVALID_ARG;
        if (!compatible(p, &descs[i])) return AAF_ERR_INCOMPAT;
        if (descs[i].n_tokens < 1) return AAF_ERR_INVALID_ARG;
        if (nblk_of(p, descs[i].n_tokens) > p->g.max_blk) return AAF_ERR_TOO_LONG;
        blocks += nblk_of(p, descs[i].n_tokens);
        tokens += descs[i].n_tokens;
    }
    if (blocks > p->lay.max_pieces) return AAF_ERR_TOO_MANY;
    if (p->g.max_ctx - p->live_ctx < n) return AAF_ERR_OOM_CTX;
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int rc0 = ensure_free(p, blocks, st);
    if (rc0 != AAF_OK) return rc0;
    p->last_stream = st;
    SmallImp small{};
    const bool by_value = n <= SMALL_RECORDS;
    ImpEntry *ent = by_value ? small.e : reinterpret_cast<ImpEntry *>(acquire_args(p));
    int c = -1, off = 0;
    for (int i = 0; i < n; ++i) {  // the n smallest free handles, in order: what the loop of imports would take
        c = smallest_free_ctx(p, c + 1);
        ImpEntry &e = ent[i];
        e.src = static_cast<const char *>(src_dev[i]);
        e.n = descs[i].n_tokens;
        e.ctx = c; e.block_off = off; e.out_index = i; e.pad = 0;
        off += (int)nblk_of(p, e.n);
    }
    const PlanSlot ps = begin_plan(p);
    const cudaError_t e = launch_plan_import_batch(p->g, ps.view, by_value ? nullptr : ent, small, n, (int)blocks,
                                                   p->clock + 1, p->meta_stream);
    // the handles are read back from the records before the ring slot is released
    for (int i = 0; i < n; ++i) out_ctxs[i] = ent[i].ctx;
    if (!by_value) release_args(p, p->meta_stream);
    if (e != cudaSuccess || !end_plan(p, ps, st)) return broke(p);
    p->clock += n;
    p->meta_launches += 1;
    p->free_lb -= blocks;
    for (int i = 0; i < n; ++i) p->len[out_ctxs[i]] = descs[i].n_tokens;
    p->live_ctx += n;
    const int rc = run_copy(p, ps, AAF_OP_IMPORT, (int)blocks, tokens, st);
    end_copy(p, ps, st);
    return rc;
}

int aaf_kv_import_host(aaf_kv_pool *p, const void *src_host, const aaf_kv_xfer_desc *desc, void *staging_dev,
                       size_t staging_bytes, aaf_ctx_t *out_ctx, void *stream) {
    AAF_RANGE("aaf_kv_import_host");
    if (!p || !src_host || !desc) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    DeviceGuard guard(p->device);
    if (desc->n_tokens >= 1 && (unsigned long long)staging_bytes < (unsigned long long)(desc->n_tokens * bpt_of(p)))
        return AAF_ERR_DST_TOO_SMALL;
    return import_impl(p, staging_dev, desc, out_ctx, static_cast<cudaStream_t>(stream), src_host);
}

int aaf_kv_materialize_host_chunked(aaf_kv_pool *p, aaf_ctx_t ctx, int64_t t0, int64_t t1, void *dst_host,
                                    size_t dst_bytes, void *staging_dev, size_t staging_bytes, int32_t chunk_tokens,
                                    uint32_t *done_flags_host, int32_t flags_cap, int32_t *n_chunks_out,
                                    aaf_kv_xfer_desc *out_desc, void *stream) {
    AAF_RANGE("aaf_kv_materialize_host_chunked");
    if (!p || !dst_host || chunk_tokens < 1 || chunk_tokens % p->g.BS != 0) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    if (!is_live(p, ctx)) return AAF_ERR_BAD_CTX;
    if (!aligned16(staging_dev) || t0 < 0 || t0 >= t1 || t1 > p->len[ctx]) return AAF_ERR_INVALID_ARG;
    const long long n = t1 - t0;
    if ((unsigned long long)dst_bytes < (unsigned long long)(n * bpt_of(p)) ||
        (unsigned long long)staging_bytes < (unsigned long long)(n * bpt_of(p)))
        return AAF_ERR_DST_TOO_SMALL;
    const int BS = p->g.BS;
    const long long j0 = t0 / BS, j1 = (t1 - 1) / BS;
    const int n_slots = (int)(j1 - j0 + 1), per_chunk = chunk_tokens / BS;
    const int n_chunks = (n_slots + per_chunk - 1) / per_chunk;
    if (done_flags_host && flags_cap < n_chunks) return AAF_ERR_DST_TOO_SMALL;
    DeviceGuard guard(p->device);
    if (!ensure_xfer_stream(p)) return broke(p);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    if (done_flags_host)
        for (int c = 0; c < n_chunks; ++c) done_flags_host[c] = 0;
    const PlanSlot ps = begin_plan(p);
    if (launch_plan_materialize(p->g, ps.view, ctx, t0, t1, static_cast<char *>(staging_dev), p->clock + 1,
                                p->meta_stream) != cudaSuccess ||
        !end_plan(p, ps, st))
        return broke(p);
    p->clock += 1;
    p->meta_launches += 1;
    bool ok = true;
    for (int c = 0; c < n_chunks && ok; ++c) {
        const int s0 = c * per_chunk, s1 = std::min(n_slots, s0 + per_chunk);
        const long long lo = std::max<long long>(t0, (j0 + s0) * BS), hi = std::min<long long>(t1, (j0 + s1) * BS);
        ok = run_copy(p, ps, AAF_OP_MATERIALIZE, s1 - s0, hi - lo, st, s0) == AAF_OK;  // gather of this chunk's blocks
        cudaEvent_t ev = order_event(p);
        ok = ok && ev && cudaEventRecord(ev, st) == cudaSuccess &&
             cudaStreamWaitEvent(p->xfer_stream, ev, 0) == cudaSuccess;
        // while the next chunk is gathered, this one crosses PCIe
        ok = ok && copy_slab(p, static_cast<char *>(dst_host), static_cast<const char *>(staging_dev), n, lo - t0,
                             hi - lo, cudaMemcpyDeviceToHost, p->xfer_stream) == cudaSuccess;
        if (ok && done_flags_host)  // completion flag of the chunk, written in stream order after its bytes
            ok = cudaMemcpyAsync(&done_flags_host[c], &p->s.ctl->one, sizeof(uint32_t), cudaMemcpyDeviceToHost,
                                 p->xfer_stream) == cudaSuccess;
    }
    end_copy(p, ps, st);
    // the caller's stream is complete only when the last chunk has landed
    cudaEvent_t fin = order_event(p);
    ok = ok && fin && cudaEventRecord(fin, p->xfer_stream) == cudaSuccess && cudaStreamWaitEvent(st, fin, 0) == cudaSuccess;
    if (!ok) return broke(p);
    if (n_chunks_out) *n_chunks_out = n_chunks;
    if (out_desc) fill_desc(p, out_desc, t0, n);
    return AAF_OK;
}

int aaf_kv_import_host_chunked(aaf_kv_pool *p, const void *src_host, const aaf_kv_xfer_desc *desc, void *staging_dev,
                               size_t staging_bytes, int32_t chunk_tokens, aaf_ctx_t *out_ctx, void *stream) {
    AAF_RANGE("aaf_kv_import_host_chunked");
    if (!p || !src_host || !desc || !out_ctx || chunk_tokens < 1 || chunk_tokens % p->g.BS != 0 ||
        !aligned16(staging_dev))
        return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    if (!compatible(p, desc)) return AAF_ERR_INCOMPAT;
    const long long n = desc->n_tokens;
    if (n < 1) return AAF_ERR_INVALID_ARG;
    if ((unsigned long long)staging_bytes < (unsigned long long)(n * bpt_of(p))) return AAF_ERR_DST_TOO_SMALL;
    const long long nb = nblk_of(p, n);
    if (nb > p->g.max_blk) return AAF_ERR_TOO_LONG;
    const int c = smallest_free_ctx(p);
    if (c < 0) return AAF_ERR_OOM_CTX;
    DeviceGuard guard(p->device);
    if (!ensure_upload_stream(p)) return broke(p);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int rc0 = ensure_free(p, nb, st);
    if (rc0 != AAF_OK) return rc0;
    p->last_stream = st;
    // staging_dev is this call's scratch: the only earlier reader the library knows of is the scatter of the
    // previous aaf_kv_import_host_chunked, so the upload waits for that and for nothing else on `stream`
    bool ok = !p->import_reader_pending ||
              cudaStreamWaitEvent(p->upload_stream, p->import_reader_done, 0) == cudaSuccess;
    const PlanSlot ps = begin_plan(p);
    ok = ok && launch_plan_import(p->g, ps.view, c, n, static_cast<const char *>(staging_dev), p->clock + 1,
                                  p->meta_stream) == cudaSuccess &&
         end_plan(p, ps, st);
    if (!ok) return broke(p);
    p->clock += 1;
    p->meta_launches += 1;
    p->free_lb -= nb;
    p->len[c] = n;
    p->live_ctx += 1;
    *out_ctx = c;
    const int BS = p->g.BS, per_chunk = chunk_tokens / BS;
    for (long long s0 = 0; s0 < nb && ok; s0 += per_chunk) {
        const long long s1 = std::min<long long>(nb, s0 + per_chunk);
        const long long lo = s0 * BS, hi = std::min<long long>(n, s1 * BS);
        ok = copy_slab(p, static_cast<char *>(staging_dev), static_cast<const char *>(src_host), n, lo, hi - lo,
                       cudaMemcpyHostToDevice, p->upload_stream) == cudaSuccess;
        cudaEvent_t ev = order_event(p);
        ok = ok && ev && cudaEventRecord(ev, p->upload_stream) == cudaSuccess &&
             cudaStreamWaitEvent(st, ev, 0) == cudaSuccess;
        // scatter of the chunk that has arrived, while the next one crosses PCIe
        ok = ok && run_copy(p, ps, AAF_OP_IMPORT, (int)(s1 - s0), hi - lo, st, (int)s0) == AAF_OK;
    }
    end_copy(p, ps, st);
    ok = ok && cudaEventRecord(p->import_reader_done, st) == cudaSuccess;
    if (!ok) return broke(p);
    p->import_reader_pending = true;
    return AAF_OK;
}

int aaf_kv_fork(aaf_kv_pool *p, aaf_ctx_t parent, int32_t k, aaf_ctx_t *out_children, void *stream) {
    AAF_RANGE("aaf_kv_fork");
    if (!p || !out_children || k < 1) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    if (!is_live(p, parent)) return AAF_ERR_BAD_CTX;
    if (k > p->lay.max_batch) return AAF_ERR_TOO_MANY;
    if (p->g.max_ctx - p->live_ctx < k) return AAF_ERR_OOM_CTX;
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    // a small fan-out travels as kernel parameters, a large one through the pinned argument ring
    SmallInts small{};
    const bool by_value = k <= SMALL_ARGS;
    int *children = by_value ? small.v : reinterpret_cast<int *>(acquire_args(p));
    int c = -1;
    for (int j = 0; j < k; ++j) {
        c = smallest_free_ctx(p, c + 1);
        children[j] = c;
    }
    const long long T = p->len[parent];
    const cudaError_t e = launch_fork(p->g, p->s, parent, T, k, by_value ? nullptr : children, small, p->clock + 1,
                                      p->meta_stream);
    if (!by_value) release_args(p, p->meta_stream);
    if (e != cudaSuccess) return broke(p);
    p->clock += 1;
    p->meta_launches += 1;
    for (int j = 0; j < k; ++j) {
        p->len[children[j]] = T;
        out_children[j] = children[j];
    }
    p->live_ctx += k;
    return AAF_OK;
}

// everything about an append batch that the host can check without the device
static int append_check(const aaf_kv_pool *p, int32_t n, const aaf_ctx_t *ctxs, const int32_t *n_new) {
    if (n > p->lay.max_batch) return AAF_ERR_TOO_MANY;
    for (int i = 0; i < n; ++i) {
        if (!is_live(p, ctxs[i])) return AAF_ERR_BAD_CTX;
        if (n_new[i] < 1) return AAF_ERR_INVALID_ARG;
    }
    std::vector<int> sorted(ctxs, ctxs + n);
    std::sort(sorted.begin(), sorted.end());
    if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return AAF_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i)
        if (nblk_of(p, p->len[ctxs[i]] + n_new[i]) > p->g.max_blk) return AAF_ERR_TOO_LONG;
    return AAF_OK;
}

int aaf_kv_append(aaf_kv_pool *p, int32_t n, const aaf_ctx_t *ctxs, const int32_t *n_new,
                  const void *const *src_dev, void *stream) {
    AAF_RANGE("aaf_kv_append");
    if (!p || n < 1 || !ctxs || !n_new || !src_dev) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    {
        const int rc = append_check(p, n, ctxs, n_new);
        if (rc != AAF_OK) return rc;
    }
    for (int i = 0; i < n; ++i)
        if (!aligned16(src_dev[i])) return AAF_ERR_INVALID_ARG;
    const int BS = p->g.BS;
    long long worst = 0, slots = 0, append_tokens = 0;  // append_tokens: new tokens plus the copy-on-write worst case
    for (int i = 0; i < n; ++i) {
        const long long T = p->len[ctxs[i]];
        append_tokens += n_new[i] + T % BS;
        worst += (T % BS ? 1 : 0) + nblk_of(p, T + n_new[i]) - nblk_of(p, T);
        slots += 1 + nblk_of(p, T + n_new[i]) - T / BS;
    }
    if (slots > p->lay.max_pieces) return AAF_ERR_TOO_MANY;
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;

    // a small batch travels as kernel parameters, a large one through the pinned argument ring
    SmallAppend small{};
    const bool by_value = n <= SMALL_RECORDS;
    AppendEntry *ent = by_value ? small.e : reinterpret_cast<AppendEntry *>(acquire_args(p));
    const AppendEntry *ent_dev = by_value ? nullptr : ent;
    int off = 0;
    for (int i = 0; i < n; ++i) {
        const long long T = p->len[ctxs[i]];
        ent[i].src = static_cast<const char *>(src_dev[i]);
        ent[i].T = T;
        ent[i].ctx = ctxs[i];
        ent[i].n_new = n_new[i];
        ent[i].piece_off = off;
        ent[i].pad = 0;
        off += (int)(1 + nblk_of(p, T + n_new[i]) - T / BS);
    }
    long long charge = worst;  // what the lower bound is reduced by
    if (p->free_lb < worst) {
        int rc = refresh_free(p, st);
        if (rc == AAF_OK && p->free_lb < worst) {
            // the worst case does not fit: ask the planner (dry run) how many blocks the batch really
            // needs; only tail blocks that are still shared are copied
            unsigned long long need = 0;
            if (launch_plan_append(p->g, p->s, ent_dev, small, n, (int)slots, p->lay.max_batch, 1, p->clock,
                                   p->meta_stream) != cudaSuccess ||
                cudaStreamSynchronize(p->meta_stream) != cudaSuccess ||
                cudaMemcpy(&need, &p->s.ctl->probe_need, sizeof(need), cudaMemcpyDeviceToHost) != cudaSuccess)
                rc = AAF_ERR_CUDA;
            else if ((long long)need > p->free_lb)
                rc = AAF_ERR_OOM_BLOCKS;
            p->meta_launches += 1;
            charge = (long long)need;
        }
        if (rc != AAF_OK) {
            if (!by_value) release_args(p, p->meta_stream);
            return rc;
        }
    }
    const PlanSlot ps = begin_plan(p);
    const cudaError_t e = launch_plan_append(p->g, ps.view, ent_dev, small, n, (int)slots, p->lay.max_batch, 0,
                                             p->clock + 1, p->meta_stream);
    if (!by_value) release_args(p, p->meta_stream);
    if (e != cudaSuccess || !end_plan(p, ps, st)) return broke(p);
    p->clock += 1;
    p->meta_launches += 1;
    p->free_lb -= charge;
    for (int i = 0; i < n; ++i) p->len[ctxs[i]] += n_new[i];
    const int rc_copy = run_copy(p, ps, AAF_OP_APPEND, (int)slots, append_tokens, st);
    end_copy(p, ps, st);
    return rc_copy;
}

int aaf_kv_append_host(aaf_kv_pool *p, int32_t n, const aaf_ctx_t *ctxs, const int32_t *n_new,
                       const void *const *src_host, void *staging_dev, size_t staging_bytes, void *stream) {
    AAF_RANGE("aaf_kv_append_host");
    if (!p || n < 1 || !ctxs || !n_new || !src_host || !aligned16(staging_dev)) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    {
        const int rc = append_check(p, n, ctxs, n_new);
        if (rc != AAF_OK) return rc;
    }
    unsigned long long need_bytes = 0;
    for (int i = 0; i < n; ++i) {
        if (!src_host[i]) return AAF_ERR_INVALID_ARG;
        need_bytes += (unsigned long long)n_new[i] * (unsigned long long)bpt_of(p);
    }
    if ((unsigned long long)staging_bytes < need_bytes) return AAF_ERR_DST_TOO_SMALL;
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!ensure_upload_stream(p)) return AAF_ERR_CUDA;
    // the staging buffer is this call's scratch: the only earlier reader the library knows of is the copy launch
    // of the previous aaf_kv_append_host, so the upload waits for that one and for nothing else on `stream`
    bool ok = !p->upload_reader_pending || cudaStreamWaitEvent(p->upload_stream, p->upload_reader_done, 0) == cudaSuccess;
    std::vector<const void *> dev_ptrs((size_t)n);
    char *cursor = static_cast<char *>(staging_dev);
    for (int i = 0; i < n && ok; ++i) {  // one copy per entry, back to back on the upload stream
        const size_t bytes = (size_t)n_new[i] * (size_t)bpt_of(p);
        ok = cudaMemcpyAsync(cursor, src_host[i], bytes, cudaMemcpyHostToDevice, p->upload_stream) == cudaSuccess;
        dev_ptrs[(size_t)i] = cursor;
        cursor += bytes;
    }
    cudaEvent_t arrived = order_event(p);
    ok = ok && arrived && cudaEventRecord(arrived, p->upload_stream) == cudaSuccess &&
         cudaStreamWaitEvent(st, arrived, 0) == cudaSuccess;
    if (!ok) return broke(p);
    const int rc = aaf_kv_append(p, n, ctxs, n_new, dev_ptrs.data(), stream);
    if (rc == AAF_OK) {
        if (cudaEventRecord(p->upload_reader_done, st) != cudaSuccess) return broke(p);
        p->upload_reader_pending = true;
    }
    return rc;
}

// n_out merges in one planner launch and one copy launch: merge i concatenates segs[seg_off[i] .. seg_off[i + 1])
static int compose_impl(aaf_kv_pool *p, int32_t n_out, const int32_t *seg_off, const aaf_ctx_t *segs, uint32_t flags,
                        aaf_ctx_t *out_ctxs, cudaStream_t st) {
    const int m = seg_off[n_out];
    if (m > p->lay.max_batch || n_out > p->lay.max_batch) return AAF_ERR_TOO_MANY;
    for (int i = 0; i < m; ++i)
        if (!is_live(p, segs[i])) return AAF_ERR_BAD_CTX;
    const bool copy_all = (flags & AAF_COMPOSE_COPY_ALL) != 0;
    const int BS = p->g.BS;
    // everything but the block ids follows from the lengths
    std::vector<ComposeSeg> rec((size_t)m);
    std::vector<long long> out_len((size_t)n_out);
    long long fresh = 0, work = 0, slots = 0, copied_tokens = 0;
    for (int o = 0; o < n_out; ++o) {
        long long off = 0, tbl = 0;
        const int s0 = seg_off[o], s1 = seg_off[o + 1];
        for (int i = s0; i < s1; ++i) {
            const long long T = p->len[segs[i]];
            const bool last = i == s1 - 1;
            ComposeSeg &r = rec[(size_t)i];
            memset(&r, 0, sizeof(r));
            r.T = T; r.off = off; r.ctx = segs[i];
            r.work_off = (int)work; r.fresh_start = (int)fresh; r.piece_off = (int)slots;
            r.out_index = o;
            r.first_ctx = last ? segs[s0] : -1;
            if (!copy_all && off % BS == 0) {
                r.mode = 0;
                r.share_tail = last;
                r.dst_tbl_start = (int)tbl;
                work += nblk_of(p, T);
                if (T % BS && !last) { fresh += 1; slots += 1; copied_tokens += T % BS; }
            } else {
                r.mode = 1;
                const long long items = (off + T - 1) / BS - off / BS + 1;
                work += items;
                slots += items;  // one two-part piece per destination block
                copied_tokens += T;
                fresh += nblk_of(p, off + T) - nblk_of(p, off);
            }
            off += T;
            tbl = nblk_of(p, off);
        }
        if (nblk_of(p, off) > p->g.max_blk) return AAF_ERR_TOO_LONG;
        out_len[(size_t)o] = off;
    }
    if (slots > p->lay.max_pieces || work >= (1ll << 31)) return AAF_ERR_TOO_MANY;
    if (p->g.max_ctx - p->live_ctx < n_out) return AAF_ERR_OOM_CTX;
    const int rc0 = ensure_free(p, fresh, st);
    if (rc0 != AAF_OK) return rc0;
    p->last_stream = st;
    std::vector<int> handles((size_t)n_out);
    int c = -1;
    for (int o = 0; o < n_out; ++o) {  // the n_out smallest free handles, in order: what the loop of merges would take
        c = smallest_free_ctx(p, c + 1);
        handles[(size_t)o] = c;
    }
    for (int i = 0; i < m; ++i) rec[(size_t)i].out_ctx = handles[(size_t)rec[(size_t)i].out_index];
    // a few segments travel as kernel parameters, more through the pinned argument ring
    SmallCompose small{};
    const bool by_value = m <= SMALL_RECORDS;
    ComposeSeg *dev_rec = by_value ? nullptr : reinterpret_cast<ComposeSeg *>(acquire_args(p));
    memcpy(by_value ? small.s : dev_rec, rec.data(), sizeof(ComposeSeg) * (size_t)m);
    const PlanSlot ps = begin_plan(p);
    const cudaError_t e = launch_plan_compose(p->g, ps.view, dev_rec, small, m, (int)work, (int)fresh, (int)slots,
                                              p->clock + 1, p->meta_stream);
    if (!by_value) release_args(p, p->meta_stream);
    if (e != cudaSuccess || !end_plan(p, ps, st)) return broke(p);
    p->clock += n_out;  // merge i of the batch is the call with clock + 1 + i
    p->meta_launches += 1;
    p->free_lb -= fresh;
    for (int o = 0; o < n_out; ++o) {
        p->len[handles[(size_t)o]] = out_len[(size_t)o];
        out_ctxs[o] = handles[(size_t)o];
    }
    p->live_ctx += n_out;
    const int rc_copy = run_copy(p, ps, AAF_OP_COMPOSE, (int)slots, copied_tokens, st);
    end_copy(p, ps, st);
    return rc_copy;
}

int aaf_kv_compose(aaf_kv_pool *p, int32_t m, const aaf_ctx_t *segs, uint32_t flags, aaf_ctx_t *out_ctx,
                   void *stream) {
    AAF_RANGE("aaf_kv_compose");
    if (!p || m < 1 || !segs || !out_ctx || (flags & ~AAF_COMPOSE_COPY_ALL)) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    DeviceGuard guard(p->device);
    const int32_t seg_off[2] = {0, m};
    return compose_impl(p, 1, seg_off, segs, flags, out_ctx, static_cast<cudaStream_t>(stream));
}

int aaf_kv_compose_batch(aaf_kv_pool *p, int32_t n_out, const int32_t *seg_off, const aaf_ctx_t *segs, uint32_t flags,
                         aaf_ctx_t *out_ctxs, void *stream) {
    AAF_RANGE("aaf_kv_compose_batch");
    if (!p || n_out < 1 || !seg_off || !segs || !out_ctxs || (flags & ~AAF_COMPOSE_COPY_ALL)) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    if (seg_off[0] != 0) return AAF_ERR_INVALID_ARG;
    for (int o = 0; o < n_out; ++o)
        if (seg_off[o + 1] <= seg_off[o]) return AAF_ERR_INVALID_ARG;  // every merge has at least one segment
    DeviceGuard guard(p->device);
    return compose_impl(p, n_out, seg_off, segs, flags, out_ctxs, static_cast<cudaStream_t>(stream));
}

int aaf_kv_evict(aaf_kv_pool *p, int32_t n, const aaf_ctx_t *ctxs, void *stream) {
    AAF_RANGE("aaf_kv_evict");
    if (!p || n < 1 || !ctxs) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    if (n > p->lay.max_batch) return AAF_ERR_TOO_MANY;
    for (int i = 0; i < n; ++i)
        if (!is_live(p, ctxs[i])) return AAF_ERR_BAD_CTX;
    {
        std::vector<int> sorted(ctxs, ctxs + n);
        std::sort(sorted.begin(), sorted.end());
        if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return AAF_ERR_INVALID_ARG;
    }
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    long long total = 0;
    for (int i = 0; i < n; ++i) total += nblk_of(p, p->len[ctxs[i]]);
    // a small batch travels as kernel parameters, a large one through the pinned argument ring
    SmallInts small{};
    const bool by_value = n <= SMALL_ARGS && total <= 32768;
    EvictArgs *a = by_value ? nullptr : reinterpret_cast<EvictArgs *>(acquire_args(p));
    int *ctx = by_value ? small.v : reinterpret_cast<int *>(a + 1);
    int *ent_off = ctx + n;
    total = 0;
    for (int i = 0; i < n; ++i) {
        ctx[i] = ctxs[i];
        ent_off[i] = (int)total;
        total += nblk_of(p, p->len[ctxs[i]]);
    }
    ent_off[n] = (int)total;
    if (a) {
        a->n = n;
        a->total = (int)total;
    }
    int n_launches = 0;
    const cudaError_t e = launch_evict(p->g, p->s, a, small, n, (int)total, p->clock + 1, &n_launches, p->meta_stream);
    if (a) release_args(p, p->meta_stream);
    if (e != cudaSuccess) return broke(p);
    p->clock += 1;
    p->meta_launches += n_launches;
    for (int i = 0; i < n; ++i) p->len[ctxs[i]] = -1;
    p->live_ctx -= n;
    // The lower bound of the free count stays valid (evict only adds free blocks), and the host can raise it without
    // asking the device: a live block is named by at least one table entry, so at most sum(table lengths) blocks
    // are live.  A caller that evicts what it created therefore never pays the synchronising refresh.
    long long entries = 0;
    for (int c = 0; c < p->g.max_ctx; ++c)
        if (p->len[c] >= 0) entries += nblk_of(p, p->len[c]);
    p->free_lb = std::max(p->free_lb, (long long)p->g.NB - entries);
    return AAF_OK;
}

int aaf_kv_evict_to_budget(aaf_kv_pool *p, double alpha, double beta, double gamma, int64_t budget_blocks,
                           aaf_ctx_t *out_victims, int32_t cap, int32_t *n_victims, void *stream) {
    AAF_RANGE("aaf_kv_evict_to_budget");
    if (!p || !out_victims || !n_victims || budget_blocks < 0) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    if (!(alpha == alpha && beta == beta && gamma == gamma) || alpha - alpha != 0.0 || beta - beta != 0.0 ||
        gamma - gamma != 0.0)
        return AAF_ERR_INVALID_ARG;  // NaN or infinite weights
    if (cap < p->live_ctx) return AAF_ERR_INVALID_ARG;
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    if (launch_evict_to_budget(p->g, p->s, alpha, beta, gamma, budget_blocks, p->clock + 1, p->result,
                               p->meta_stream) != cudaSuccess)
        return broke(p);
    p->meta_launches += 1;
    // the victims are chosen on the device; the host mirror needs them before the next call
    if (cudaStreamSynchronize(p->meta_stream) != cudaSuccess) return broke(p);
    p->clock += 1;
    const int nv = p->result[0];
    for (int i = 0; i < nv; ++i) {
        const int v = p->result[2 + i];
        out_victims[i] = v;
        p->len[v] = -1;
    }
    p->live_ctx -= nv;
    p->free_lb = p->result[1];  // exact
    *n_victims = nv;
    return AAF_OK;
}

int aaf_kv_catalog_rows(aaf_kv_pool *p, int32_t *n_states, int64_t *n_block_rows) {
    if (!p || !n_states || !n_block_rows) return AAF_ERR_INVALID_ARG;
    long long rows = 0;
    for (int c = 0; c < p->g.max_ctx; ++c)
        if (p->len[c] >= 0) rows += nblk_of(p, p->len[c]);
    *n_states = p->live_ctx;
    *n_block_rows = rows;
    return AAF_OK;
}

int aaf_kv_export_catalog(aaf_kv_pool *p, const aaf_kv_catalog_cols *cols, void *stream) {
    AAF_RANGE("aaf_kv_export_catalog");
    if (!p || !cols) return AAF_ERR_INVALID_ARG;
    if (p->broken) return AAF_ERR_CUDA;
    int32_t ns = 0;
    int64_t rows = 0;
    aaf_kv_catalog_rows(p, &ns, &rows);
    if (!cols->state_id || !cols->n_tokens || !cols->reuse || !cols->last_access || !cols->block_offsets ||
        !cols->origin || !cols->parent || !cols->born || !cols->parent_born)
        return AAF_ERR_INVALID_ARG;
    if (rows > 0 && (!cols->block_id || !cols->pos_begin || !cols->pos_end || !cols->refcount || !cols->address))
        return AAF_ERR_INVALID_ARG;
    if (rows > 0x7fffffffll) return AAF_ERR_TOO_LONG;  // Arrow int32 list offsets
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    // the columns are the caller's buffers: written on the metadata stream, then the caller's stream waits
    cudaEvent_t done = order_event(p);
    if (launch_export_catalog(p->g, p->s, *cols, ns, rows, p->meta_stream) != cudaSuccess || !done ||
        cudaEventRecord(done, p->meta_stream) != cudaSuccess || cudaStreamWaitEvent(st, done, 0) != cudaSuccess)
        return broke(p);
    p->meta_launches += rows > 0 ? 2 : 1;
    return AAF_OK;
}

int aaf_kv_get_catalog(aaf_kv_pool *p, int64_t *clock, int64_t *reuse_out, int64_t *last_access_out) {
    if (!p || !clock || !reuse_out || !last_access_out) return AAF_ERR_INVALID_ARG;
    DeviceGuard guard(p->device);
    if (cudaStreamSynchronize(p->meta_stream) != cudaSuccess || cudaStreamSynchronize(p->last_stream) != cudaSuccess)
        return AAF_ERR_CUDA;
    const size_t nbytes = sizeof(long long) * (size_t)p->g.max_ctx;
    if (cudaMemcpy(reuse_out, p->s.cat_reuse, nbytes, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(last_access_out, p->s.cat_last, nbytes, cudaMemcpyDeviceToHost) != cudaSuccess)
        return AAF_ERR_CUDA;
    for (int c = 0; c < p->g.max_ctx; ++c)
        if (p->len[c] < 0) reuse_out[c] = last_access_out[c] = -1;
    *clock = p->clock;
    return AAF_OK;
}

int aaf_kv_ctx_len(aaf_kv_pool *p, aaf_ctx_t ctx, int64_t *n_tokens) {
    if (!p || !n_tokens) return AAF_ERR_INVALID_ARG;
    if (!is_live(p, ctx)) return AAF_ERR_BAD_CTX;
    *n_tokens = p->len[ctx];
    return AAF_OK;
}

int aaf_kv_get_table(aaf_kv_pool *p, aaf_ctx_t ctx, int32_t *host_out, int32_t cap, int32_t *n_blocks) {
    if (!p || !host_out || !n_blocks) return AAF_ERR_INVALID_ARG;
    if (!is_live(p, ctx)) return AAF_ERR_BAD_CTX;
    const long long nb = nblk_of(p, p->len[ctx]);
    if (cap < nb) return AAF_ERR_DST_TOO_SMALL;
    DeviceGuard guard(p->device);
    if (cudaStreamSynchronize(p->meta_stream) != cudaSuccess || cudaStreamSynchronize(p->last_stream) != cudaSuccess)
        return AAF_ERR_CUDA;
    if (cudaMemcpy(host_out, p->s.tables + (long long)ctx * p->g.max_blk, sizeof(int) * (size_t)nb,
                   cudaMemcpyDeviceToHost) != cudaSuccess)
        return AAF_ERR_CUDA;
    *n_blocks = (int32_t)nb;
    return AAF_OK;
}

int aaf_kv_get_refcounts(aaf_kv_pool *p, int32_t *host_out) {
    if (!p || !host_out) return AAF_ERR_INVALID_ARG;
    DeviceGuard guard(p->device);
    if (cudaStreamSynchronize(p->meta_stream) != cudaSuccess || cudaStreamSynchronize(p->last_stream) != cudaSuccess)
        return AAF_ERR_CUDA;
    return cudaMemcpy(host_out, p->s.refcount, sizeof(int) * (size_t)p->g.NB, cudaMemcpyDeviceToHost) == cudaSuccess
               ? AAF_OK
               : AAF_ERR_CUDA;
}

int aaf_kv_get_free_list(aaf_kv_pool *p, int32_t *host_out, int32_t *n_free) {
    if (!p || !host_out || !n_free) return AAF_ERR_INVALID_ARG;
    DeviceGuard guard(p->device);
    if (cudaStreamSynchronize(p->meta_stream) != cudaSuccess || cudaStreamSynchronize(p->last_stream) != cudaSuccess)
        return AAF_ERR_CUDA;
    unsigned long long ht[2];
    std::vector<int> ring((size_t)p->g.NB);
    if (cudaMemcpy(ht, p->s.ctl, sizeof(ht), cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(ring.data(), p->s.ring, sizeof(int) * ring.size(), cudaMemcpyDeviceToHost) != cudaSuccess)
        return AAF_ERR_CUDA;
    const unsigned long long f = ht[1] - ht[0];
    if (f > (unsigned long long)p->g.NB) return AAF_ERR_CORRUPT;
    for (unsigned long long i = 0; i < f; ++i) host_out[i] = ring[(size_t)((ht[0] + i) % (unsigned long long)p->g.NB)];
    *n_free = (int32_t)f;
    p->free_lb = (long long)f;
    return AAF_OK;
}

int aaf_kv_pool_stats(aaf_kv_pool *p, aaf_kv_stats *out) {
    if (!p || !out) return AAF_ERR_INVALID_ARG;
    DeviceGuard guard(p->device);
    if (cudaStreamSynchronize(p->meta_stream) != cudaSuccess || cudaStreamSynchronize(p->last_stream) != cudaSuccess)
        return AAF_ERR_CUDA;
    drain_timing(p);
    DevCtl ctl;
    if (cudaMemcpy(&ctl, p->s.ctl, sizeof(ctl), cudaMemcpyDeviceToHost) != cudaSuccess) return AAF_ERR_CUDA;
    memset(out, 0, sizeof(*out));
    out->free_blocks = (int64_t)(ctl.tail - ctl.head);
    out->live_blocks = p->g.NB - out->free_blocks;
    out->peak_live_blocks = ctl.peak_live;
    out->live_ctx = p->live_ctx;
    out->cow_count = (int64_t)ctl.cow_count;
    out->payload_bytes = (int64_t)ctl.payload_bytes;
    out->meta_launches = p->meta_launches;
    for (int i = 0; i < AAF_OP_CLASSES; ++i) {
        out->copy_launches[i] = p->copy_launches[i];
        out->copy_ms[i] = p->copy_ms[i];
        out->timed_launches[i] = p->timed_launches[i];
    }
    p->free_lb = out->free_blocks;
    return AAF_OK;
}

int aaf_kv_sync_status(aaf_kv_pool *p) {
    if (!p) return AAF_ERR_INVALID_ARG;
    DeviceGuard guard(p->device);
    if (cudaStreamSynchronize(p->meta_stream) != cudaSuccess || cudaStreamSynchronize(p->last_stream) != cudaSuccess)
        return AAF_ERR_CUDA;
    int st[2] = {0, 0};
    if (cudaMemcpy(st, &p->s.ctl->status, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess) return AAF_ERR_CUDA;
    if (st[0] != 0) {
        const int zero[2] = {0, 0};
        cudaMemcpy(&p->s.ctl->status, zero, sizeof(zero), cudaMemcpyHostToDevice);
    }
    return st[0];
}

int aaf_kv_set_copy_engine(aaf_kv_pool *p, int engine) {
    if (!p || engine < AAF_ENGINE_AUTO || engine > AAF_ENGINE_WARP) return AAF_ERR_INVALID_ARG;
    p->engine = engine;
    return AAF_OK;
}

int aaf_kv_debug_expire_wait(aaf_kv_pool *p, uint64_t limit_cycles, void *stream) {
    if (!p || limit_cycles == 0 || limit_cycles > (1ull << 31)) return AAF_ERR_INVALID_ARG;
    DeviceGuard guard(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    p->meta_launches += 1;
    return launch_expire_wait(p->s, (long long)limit_cycles, p->meta_stream) == cudaSuccess ? AAF_OK : AAF_ERR_CUDA;
}

int aaf_kv_debug_mark_unusable(aaf_kv_pool *p) {
    if (!p) return AAF_ERR_INVALID_ARG;
    p->broken = true;
    return AAF_OK;
}

int aaf_kv_set_timing(aaf_kv_pool *p, int enable) {
    if (!p) return AAF_ERR_INVALID_ARG;
    p->timing = enable != 0;
    return AAF_OK;
}

const char *aaf_kv_strerror(int status) {
    switch (status) {
        case AAF_OK: return "ok";
        case AAF_ERR_INVALID_ARG: return "invalid argument";
        case AAF_ERR_BAD_CTX: return "not a live context";
        case AAF_ERR_OOM_BLOCKS: return "out of free blocks";
        case AAF_ERR_OOM_CTX: return "out of context handles";
        case AAF_ERR_TOO_LONG: return "context would exceed max_blocks_per_ctx";
        case AAF_ERR_INCOMPAT: return "descriptor incompatible with the pool";
        case AAF_ERR_DST_TOO_SMALL: return "destination too small";
        case AAF_ERR_CUDA: return "CUDA runtime error";
        case AAF_ERR_CORRUPT: return "device found pool metadata inconsistent";
        case AAF_ERR_TIMEOUT: return "bounded device wait expired";
        case AAF_ERR_TOO_MANY: return "batch exceeds max_batch or the piece capacity";
        case AAF_ERR_SCRATCH_LIMIT:
            return "request exceeds the built-in scratch of aaf_kv_materialize_noalloc (AAF_NOALLOC_MAX_BLOCKS blocks)";
        default: return "unknown status";
    }
}

}  // extern "C"
