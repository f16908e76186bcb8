// Copy engines of libaafkv.so: every byte a KV operator moves goes through one of the three
// kernels below.  All consume the same piece list (see Piece): a launch covers
// n_slots pieces x n_planes (layer, K/V) planes, split into chunks of at most `chunk` bytes.
//
// The path is pure streaming (each byte is read once and written once, nothing is reused), so
// the bound is HBM bandwidth: what matters is enough independent 16-byte accesses in flight per
// SM, fully coalesced, and a persistent grid of exactly one resident wave (a multiple of the SM count).
//
// Work distribution: the SMs of a B200 do not get equal shares of the memory bandwidth (measured: with
// equal static shares some CTAs were done after 70 % of the kernel's time and the slowest set the
// pace), so the BULK and WARP engines hand units out dynamically: a CTA (a warp) draws the next unit
// (group of 32 units) from a ticket counter in the pool's control block.  The last CTA to leave sets
// the counter back to 0.  Launches that share a control block must therefore not overlap on the GPU;
// the library issues all copy launches of a pool to the caller's stream, in order.
//
//   BULK : one elected thread per CTA drives a ring of shared-memory stages with
//          cp.async.bulk (global -> shared, completion on an mbarrier) and
//          cp.async.bulk (shared -> global, bulk async-group); no registers touch the data and the
//          SMs stay idle.  Every wait is bounded; on expiry the kernel records AAF_ERR_TIMEOUT and
//          leaves.  The default for pieces of about a run.
//   WARP : 16-byte streaming loads/stores scheduled per warp, 32 units decoded at once; the default
//          for small and ragged pieces.
//   VEC  : 256 threads per CTA, each thread keeps UNROLL 16-byte streaming loads in flight and
//          then stores them; one chunk per CTA iteration, equal static shares.  Kept as the plain baseline.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include "aafkv_internal.h"

namespace aafkv {

// ------------------------------------------------------------------------------------------
// unit decomposition shared by all engines: unit u -> (chunk c, piece p, plane q), plane-major
// so that neighbouring CTAs stream neighbouring addresses of the dense side.
struct Unit {
    const char *src;   // first part
    const char *src2;  // second part (lands at dst + nbytes)
    char *dst;
    unsigned nbytes;   // bytes of the first part in this chunk
    unsigned nbytes2;  // bytes of the second part in this chunk; nbytes + nbytes2 == 0: nothing to do
};

__device__ __forceinline__ Unit decode_unit(const Piece *__restrict__ pieces, long long u, int n_slots, int plane0,
                                            int cpp, unsigned chunk) {
    const int c = (int)(u % cpp);
    const long long t = u / cpp;
    const int p = (int)(t % n_slots);
    const int q = plane0 + (int)(t / n_slots);
    const uint4 *pw = reinterpret_cast<const uint4 *>(pieces + p);
    const uint4 w0 = __ldg(pw), w1 = __ldg(pw + 1), w2 = __ldg(pw + 2), w3 = __ldg(pw + 3);
    Piece pc;
    reinterpret_cast<uint4 *>(&pc)[0] = w0;
    reinterpret_cast<uint4 *>(&pc)[1] = w1;
    reinterpret_cast<uint4 *>(&pc)[2] = w2;
    reinterpret_cast<uint4 *>(&pc)[3] = w3;
    Unit r;
    const unsigned off = (unsigned)c * chunk;
    const unsigned tot = pc.nbytes ? pc.nbytes + pc.nbytes2 : 0u;  // nbytes == 0: unused slot, whatever else it holds
    if (off >= tot) {
        r.src = nullptr; r.src2 = nullptr; r.dst = nullptr; r.nbytes = 0; r.nbytes2 = 0;
        return r;
    }
    const long long l = q >> 1, kv = q & 1;
    const char *base = pc.src + l * pc.src_sl + kv * pc.src_skv;
    const unsigned len = min(chunk, tot - off);
    const unsigned na = off < pc.nbytes ? min(len, pc.nbytes - off) : 0u;  // share of the first part
    r.src = base + off;
    r.src2 = base + pc.src2_off + (off + na - pc.nbytes);
    r.dst = pc.dst + l * pc.dst_sl + kv * pc.dst_skv + off;
    r.nbytes = na;
    r.nbytes2 = len - na;
    return r;
}

// Ticket counter of the dynamic work distribution (see the header comment).  Every drawer (a CTA of the bulk
// engine, a warp of the warp engine) starts with the unit of its own index, so that the first loads of a launch do
// not wait for an atomic; tickets number the units behind those, hence `first` = number of drawers.
__device__ __forceinline__ long long take_ticket(DevCtl *ctl, long long first) {
    return first + (long long)atomicAdd(&ctl->copy_ticket, 1ull);
}
// Called once per CTA when it has drawn its last ticket: the last CTA of the grid re-arms the counters.
__device__ __forceinline__ void leave_copy(DevCtl *ctl) {
    __threadfence();
    if (atomicAdd(&ctl->copy_done, 1u) == gridDim.x - 1) {
        ctl->copy_ticket = 0;
        ctl->copy_done = 0;
        __threadfence();
    }
}

// 16-byte vector i of a unit: the first part's vectors, then the second part's
__device__ __forceinline__ const uint4 *unit_vec(const uint4 *s4, const uint4 *s4b, unsigned nvec_a, unsigned i) {
    return i < nvec_a ? s4 + i : s4b + (i - nvec_a);
}

// ------------------------------------------------------------------------------------------
// VEC engine
constexpr int VEC_THREADS = 256;

template <int UNROLL>
__global__ void __launch_bounds__(VEC_THREADS) copy_vec_kernel(const Piece *__restrict__ pieces, int n_slots,
                                                               int plane0, int n_planes, int cpp) {
    constexpr unsigned CHUNK = VEC_THREADS * UNROLL * 16;
    const long long total = (long long)n_slots * n_planes * cpp;
    for (long long u = blockIdx.x; u < total; u += gridDim.x) {
        const Unit un = decode_unit(pieces, u, n_slots, plane0, cpp, CHUNK);
        if (un.nbytes + un.nbytes2 == 0) continue;
        const uint4 *__restrict__ s4 = reinterpret_cast<const uint4 *>(un.src);
        const uint4 *__restrict__ s4b = reinterpret_cast<const uint4 *>(un.src2);
        uint4 *__restrict__ d4 = reinterpret_cast<uint4 *>(un.dst);
        const unsigned nvec_a = un.nbytes >> 4, nvec = (un.nbytes + un.nbytes2) >> 4;
        uint4 v[UNROLL];
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) {
            const unsigned i = threadIdx.x + k * VEC_THREADS;
            if (i < nvec) v[k] = __ldcs(unit_vec(s4, s4b, nvec_a, i));
        }
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) {
            const unsigned i = threadIdx.x + k * VEC_THREADS;
            if (i < nvec) __stcs(d4 + i, v[k]);
        }
    }
}

// ------------------------------------------------------------------------------------------
// WARP engine: the same 16-byte streaming copies, but the unit of work is a warp, not a CTA.  A warp
// takes 32 consecutive units, decodes all of them at once (one unit per lane, so the descriptor
// fetches overlap and empty units cost nothing further), then moves them one after the other with
// all 32 lanes.  Small and ragged pieces (copy-on-write tails, single-token appends, the two
// part-blocks of a shifted compose) no longer leave most of a CTA idle or serialise on descriptor
// latency; full runs are split into 32*U*16-byte chunks handled by neighbouring warps.
template <int UNROLL>
__global__ void __launch_bounds__(VEC_THREADS) copy_warp_kernel(const Piece *__restrict__ pieces, int n_slots,
                                                                int plane0, int n_planes, int cpp, DevCtl *ctl) {
    constexpr unsigned CHUNK = 32 * UNROLL * 16;
    constexpr unsigned FULL = 0xffffffffu;
    const long long total = (long long)n_slots * n_planes * cpp;
    const long long groups = (total + 31) / 32;  // a ticket is worth 32 consecutive units
    const int lane = threadIdx.x & 31;
    const long long n_warps = (long long)gridDim.x * (VEC_THREADS / 32);
    long long grp = (long long)blockIdx.x * (VEC_THREADS / 32) + (threadIdx.x >> 5);
    while (grp < groups) {
        long long grp_next = lane == 0 ? take_ticket(ctl, n_warps) : 0;  // drawn early: its latency hides behind the copies
        const long long base = grp * 32;
        Unit mine;
        mine.src = nullptr; mine.src2 = nullptr; mine.dst = nullptr; mine.nbytes = 0; mine.nbytes2 = 0;
        if (base + lane < total) mine = decode_unit(pieces, base + lane, n_slots, plane0, cpp, CHUNK);
        unsigned todo = __ballot_sync(FULL, mine.nbytes + mine.nbytes2 != 0);
        while (todo) {
            const int j = __ffs(todo) - 1;
            todo &= todo - 1;
            const uint4 *__restrict__ s4 = reinterpret_cast<const uint4 *>(
                __shfl_sync(FULL, reinterpret_cast<unsigned long long>(mine.src), j));
            const uint4 *__restrict__ s4b = reinterpret_cast<const uint4 *>(
                __shfl_sync(FULL, reinterpret_cast<unsigned long long>(mine.src2), j));
            uint4 *__restrict__ d4 =
                reinterpret_cast<uint4 *>(__shfl_sync(FULL, reinterpret_cast<unsigned long long>(mine.dst), j));
            const unsigned nvec_a = __shfl_sync(FULL, mine.nbytes, j) >> 4;
            const unsigned nvec = nvec_a + (__shfl_sync(FULL, mine.nbytes2, j) >> 4);
            uint4 v[UNROLL];
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) {
                const unsigned i = lane + k * 32;
                if (i < nvec) v[k] = __ldcs(unit_vec(s4, s4b, nvec_a, i));
            }
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) {
                const unsigned i = lane + k * 32;
                if (i < nvec) __stcs(d4 + i, v[k]);
            }
        }
        grp = __shfl_sync(FULL, grp_next, 0);
    }
    __syncthreads();  // every warp of the CTA has drawn its last ticket
    if (threadIdx.x == 0) leave_copy(ctl);
}

// ------------------------------------------------------------------------------------------
// BULK engine
constexpr int BULK_MAX_STAGES = 8;
constexpr long long BULK_WAIT_CYCLES = 1ll << 32;  // about two seconds of SM clock

__device__ __forceinline__ unsigned smem_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait: false if the phase did not complete within `limit` SM clock cycles
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity, long long limit = BULK_WAIT_CYCLES) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
    }
    return true;
}

// Test hook: exercises the give-up path of the bounded wait without any fault.  One thread waits, with a
// short limit, on an mbarrier that nothing ever arrives at; when the limit expires it records
// AAF_ERR_TIMEOUT in the status word and returns, exactly as the bulk engine would.
__global__ void expire_wait_kernel(DevCtl *ctl, long long limit_cycles) {
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x != 0) return;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait_bounded(smem_u32(&bar), 0, limit_cycles)) atomicCAS(&ctl->status, 0, (int)AAF_ERR_TIMEOUT);
}

cudaError_t launch_expire_wait(const DevState &s, long long limit_cycles, cudaStream_t st) {
    expire_wait_kernel<<<1, 32, 0, st>>>(s.ctl, limit_cycles);
    return cudaGetLastError();
}
// L2 policy for data that is touched once: mark the lines evict-first so that the stream does not push
// other tenants' data out of the 126 MB L2 (optional: see copy_tuning_init)
__device__ __forceinline__ unsigned long long l2_evict_first_policy() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_g2s(unsigned smem_dst, const void *gsrc, unsigned bytes, unsigned bar,
                                         unsigned long long pol, bool hint) {
    if (hint)
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::
                "r"(smem_dst), "l"(gsrc), "r"(bytes), "r"(bar), "l"(pol)
            : "memory");
    else
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         smem_dst),
                     "l"(gsrc), "r"(bytes), "r"(bar)
                     : "memory");
}
__device__ __forceinline__ void bulk_s2g(void *gdst, unsigned smem_src, unsigned bytes, unsigned long long pol,
                                         bool hint) {
    if (hint)
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(gdst),
                     "r"(smem_src), "r"(bytes), "l"(pol)
                     : "memory");
    else
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_src),
                     "r"(bytes)
                     : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__global__ void __launch_bounds__(32) copy_bulk_kernel(const Piece *__restrict__ pieces, int n_slots, int plane0,
                                                       int n_planes, int cpp, unsigned chunk, int stages,
                                                       int l2_hints, DevCtl *ctl) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[BULK_MAX_STAGES];
    __shared__ char *dstq[BULK_MAX_STAGES];   // destination and size of the unit held by each stage
    __shared__ unsigned nbq[BULK_MAX_STAGES];  // (indexed dynamically: shared memory, not a local frame)
    if (threadIdx.x != 0) return;

    const long long total = (long long)n_slots * n_planes * cpp;
    const unsigned smem0 = smem_u32(smem);
    const unsigned long long pol = l2_evict_first_policy();
    const bool hint_ld = (l2_hints & 1) != 0, hint_st = (l2_hints & 2) != 0;
    for (int s = 0; s < stages; ++s) mbar_init(smem_u32(&bars[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

    long long u_next = blockIdx.x;  // next unit to look at for loading
    int k_load = 0;                       // units whose load has been issued
    int k_store = 0;                      // units whose store has been issued
    bool timed_out = false;

    // finds the next non-empty unit and issues its load (two loads for a two-part unit) into stage
    // k_load % stages; the ticket after it is drawn at once, so that its latency hides behind the copies
    auto issue_load = [&]() -> bool {
        while (u_next < total) {
            const Unit un = decode_unit(pieces, u_next, n_slots, plane0, cpp, chunk);
            u_next = take_ticket(ctl, gridDim.x);
            const unsigned nb = un.nbytes + un.nbytes2;
            if (nb == 0) continue;
            const int s = k_load % stages;
            const unsigned bar = smem_u32(&bars[s]);
            const unsigned stage = smem0 + (unsigned)s * chunk;
            mbar_expect_tx(bar, nb);
            if (un.nbytes) bulk_g2s(stage, un.src, un.nbytes, bar, pol, hint_ld);
            if (un.nbytes2) bulk_g2s(stage + un.nbytes, un.src2, un.nbytes2, bar, pol, hint_ld);
            dstq[s] = un.dst;
            nbq[s] = nb;
            ++k_load;
            return true;
        }
        return false;
    };

    for (int i = 0; i < stages - 1; ++i)
        if (!issue_load()) break;

    while (k_store < k_load) {
        const int s = k_store % stages;
        if (!mbar_wait_bounded(smem_u32(&bars[s]), (unsigned)(k_store / stages) & 1u)) {
            timed_out = true;
            break;
        }
        bulk_s2g(dstq[s], smem0 + (unsigned)s * chunk, nbq[s], pol, hint_st);
        bulk_commit();
        ++k_store;
        // the stage of the store before this one is the next load target: wait until that store has
        // finished reading shared memory (the store just issued may stay pending)
        bulk_wait_read_1();
        issue_load();
    }
    if (timed_out) {
        atomicCAS(&ctl->status, 0, (int)AAF_ERR_TIMEOUT);
        // loads still in flight target this CTA's shared memory: give each one bounded wait before leaving
        for (int k = k_store + 1; k < k_load; ++k)
            mbar_wait_bounded(smem_u32(&bars[k % stages]), (unsigned)(k / stages) & 1u);
    }
    bulk_wait_all();
    leave_copy(ctl);
}

// ------------------------------------------------------------------------------------------
// host side

static int env_int(const char *name, int dflt, int lo, int hi) {
    const char *v = getenv(name);
    if (!v || !*v) return dflt;
    long x = strtol(v, nullptr, 10);
    if (x < lo || x > hi) return dflt;
    return (int)x;
}

// resident CTAs per SM of a kernel, capped by `limit`: the persistent grid must fit in ONE wave,
// otherwise the CTAs of the second wave start when the first ones are done and the tail doubles
template <typename K>
static int resident_ctas(K kernel, int threads, size_t dyn_smem, int limit) {
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, threads, dyn_smem) != cudaSuccess || occ < 1) {
        cudaGetLastError();
        occ = 1;
    }
    return occ < limit ? occ : limit;
}

// Picks the launch shapes for a pool geometry (run = bytes of one block, one layer, K or V).
// Defaults come from measurements on B200 with 2 KiB rows; every knob can be overridden through the
// environment for experiments (AAFKV_ENGINE, AAFKV_BULK_CHUNK / _STAGES / _CTAS / _L2, AAFKV_VEC_UNROLL /
// _CTAS, AAFKV_WARP_UNROLL).  Called with the pool's device current; allocates nothing.
cudaError_t copy_tuning_init(long long run, CopyTuning *t) {
    long long chunk = run < 32768 ? ((run + 15) / 16) * 16 : 32768;
    if (chunk < 1024) chunk = 1024;
    t->bulk_chunk = env_int("AAFKV_BULK_CHUNK", (int)chunk, 1024, 65536) & ~15;
    t->bulk_stages = env_int("AAFKV_BULK_STAGES", 3, 2, BULK_MAX_STAGES);
    while ((long long)t->bulk_chunk * t->bulk_stages > 220 * 1024) --t->bulk_stages;
    int ctas = (int)(196608 / ((long long)t->bulk_chunk * t->bulk_stages));  // fill about 192 KiB per SM
    if (ctas < 1) ctas = 1;
    if (ctas > 8) ctas = 8;
    t->bulk_ctas = env_int("AAFKV_BULK_CTAS", ctas, 1, 16);
    // L2 evict-first hints (bit 0 loads, bit 1 stores) keep the stream from displacing other tenants' lines but cost
    // about 1.5 % of the copy rate when the GPU runs nothing else: off unless asked for
    t->bulk_l2 = env_int("AAFKV_BULK_L2", 0, 0, 3);
    t->vec_unroll = env_int("AAFKV_VEC_UNROLL", 4, 1, 8);
    if (t->vec_unroll == 3 || (t->vec_unroll > 4 && t->vec_unroll < 8)) t->vec_unroll = 4;
    t->warp_unroll = env_int("AAFKV_WARP_UNROLL", 8, 4, 8) == 4 ? 4 : 8;
    t->auto_engine = env_int("AAFKV_ENGINE", 0, 0, 3);
    t->auto_bulk_min_piece = (long long)t->bulk_chunk * 7 / 16;  // 14 KiB with 32 KiB chunks
    const cudaError_t e = cudaFuncSetAttribute(copy_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               220 * 1024);
    if (e != cudaSuccess) return e;
    t->bulk_ctas = resident_ctas(copy_bulk_kernel, 32, (size_t)t->bulk_chunk * t->bulk_stages, t->bulk_ctas);
    const int vlim = env_int("AAFKV_VEC_CTAS", 8, 1, 8);
    switch (t->vec_unroll) {
        case 1: t->vec_ctas = resident_ctas(copy_vec_kernel<1>, VEC_THREADS, 0, vlim); break;
        case 2: t->vec_ctas = resident_ctas(copy_vec_kernel<2>, VEC_THREADS, 0, vlim); break;
        case 8: t->vec_ctas = resident_ctas(copy_vec_kernel<8>, VEC_THREADS, 0, vlim); break;
        default: t->vec_ctas = resident_ctas(copy_vec_kernel<4>, VEC_THREADS, 0, vlim); break;
    }
    t->warp_ctas = t->warp_unroll == 4 ? resident_ctas(copy_warp_kernel<4>, VEC_THREADS, 0, 8)
                                       : resident_ctas(copy_warp_kernel<8>, VEC_THREADS, 0, 8);
    return cudaSuccess;
}

template <int UNROLL>
static void launch_vec(const CopyTuning &t, const DevState &s, int n_slots, int plane0, int n_planes, long long run,
                       int sm_count, cudaStream_t st) {
    constexpr long long CHUNK = (long long)VEC_THREADS * UNROLL * 16;
    const int cpp = (int)((run + CHUNK - 1) / CHUNK);
    const long long total = (long long)n_slots * n_planes * cpp;
    const long long cap = (long long)sm_count * t.vec_ctas;
    const int grid = (int)(total < cap ? total : cap);
    copy_vec_kernel<UNROLL><<<grid, VEC_THREADS, 0, st>>>(s.pieces, n_slots, plane0, n_planes, cpp);
}

template <int UNROLL>
static void launch_warp(const CopyTuning &t, const DevState &s, int n_slots, int plane0, int n_planes, long long run,
                        int sm_count, cudaStream_t st) {
    constexpr long long CHUNK = 32ll * UNROLL * 16;
    const int cpp = (int)((run + CHUNK - 1) / CHUNK);
    const long long total = (long long)n_slots * n_planes * cpp;
    const long long need = (total + 255) / 256;  // CTAs needed if every warp takes one round of 32 units
    const long long cap = (long long)sm_count * t.warp_ctas;
    const int grid = (int)(need < cap ? (need < 1 ? 1 : need) : cap);
    copy_warp_kernel<UNROLL><<<grid, VEC_THREADS, 0, st>>>(s.pieces, n_slots, plane0, n_planes, cpp, s.ctl);
}

// AUTO: pieces of about a run or more -> the bulk engine (fastest, and it leaves the SMs idle);
// small or ragged pieces -> the warp engine (many independent small copies in flight).
cudaError_t launch_copy(int engine, const CopyTuning &t, const Geom &g, const DevState &s, int n_slots, int plane0,
                        int n_planes, long long avg_piece_bytes, int sm_count, cudaStream_t st) {
    if (n_slots <= 0 || n_planes <= 0) return cudaSuccess;
    if (engine == AAF_ENGINE_AUTO) engine = t.auto_engine;
    if (engine == AAF_ENGINE_AUTO)
        engine = avg_piece_bytes >= t.auto_bulk_min_piece ? AAF_ENGINE_BULK : AAF_ENGINE_WARP;
    if (engine == AAF_ENGINE_BULK) {
        const int cpp = (int)((g.run + t.bulk_chunk - 1) / t.bulk_chunk);
        const long long total = (long long)n_slots * n_planes * cpp;
        const long long cap = (long long)sm_count * t.bulk_ctas;
        const int grid = (int)(total < cap ? total : cap);
        copy_bulk_kernel<<<grid, 32, (size_t)t.bulk_chunk * t.bulk_stages, st>>>(
            s.pieces, n_slots, plane0, n_planes, cpp, (unsigned)t.bulk_chunk, t.bulk_stages, t.bulk_l2, s.ctl);
    } else if (engine == AAF_ENGINE_WARP) {
        if (t.warp_unroll == 4) launch_warp<4>(t, s, n_slots, plane0, n_planes, g.run, sm_count, st);
        else launch_warp<8>(t, s, n_slots, plane0, n_planes, g.run, sm_count, st);
    } else {
        switch (t.vec_unroll) {
            case 1: launch_vec<1>(t, s, n_slots, plane0, n_planes, g.run, sm_count, st); break;
            case 2: launch_vec<2>(t, s, n_slots, plane0, n_planes, g.run, sm_count, st); break;
            case 8: launch_vec<8>(t, s, n_slots, plane0, n_planes, g.run, sm_count, st); break;
            default: launch_vec<4>(t, s, n_slots, plane0, n_planes, g.run, sm_count, st); break;
        }
    }
    return cudaGetLastError();
}

}  // namespace aafkv
