// aaf_kv_materialize_noalloc: the gather of aaf_kv_materialize for callers that cannot allocate.
//
// Who cannot allocate: a caller that runs inside a serving process whose start-up handed all of
// the GPU's free memory to its own KV pool (cudaMalloc then fails or has to wait for somebody
// else's free), a caller on a latency-critical path that must not take cudaMalloc's device-wide
// synchronisation, and a caller that is simply not allowed to own device memory (a plug-in that is
// handed pointers).  The regular entry points need a workspace the caller allocates and a pool
// object whose creation allocates pinned host memory and events; this one needs neither.
//
// The scratch the gather needs (the block-table slice on the device and the piece list the copy
// engine consumes) lives in a file-scope __device__ array of fixed size, so the request is limited
// to AAF_NOALLOC_MAX_BLOCKS blocks.  Every GPU that loads the library carries that array
// (about 273 KB) until the process exits.
//
// In host code the array's NAME is only a host-side stand-in for the symbol, not a device address.
// The device address is looked up once per device with cudaGetSymbolAddress, with that device
// current, and that pointer is what the kernels get.
#include <cuda_runtime.h>
#include <stdint.h>

#include "aafkv_internal.h"

using namespace aafkv;

namespace {

struct NoAllocScratch {
    DevCtl ctl;                              // counters the planner updates; cleared by every call
    int table[AAF_NOALLOC_MAX_BLOCKS];       // slice of the caller's block table
    Piece pieces[AAF_NOALLOC_MAX_BLOCKS];    // one copy descriptor per block of the range
};

static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

constexpr int MAX_DEVICES = 64;
NoAllocScratch *g_scratch_ptr[MAX_DEVICES] = {};  // device address of the array, per device
int g_sm_count[MAX_DEVICES] = {};
CopyTuning g_tuning[MAX_DEVICES] = {};     // launch shapes of the copy engine, per device

// first call on a device: resolve the array's device address with that device current
int setup_device(int dev) {
    if (g_scratch_ptr[dev]) return AAF_OK;
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
        cudaGetLastError();
        return AAF_ERR_CUDA;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
        cudaGetLastError();
        return AAF_ERR_CUDA;
    }
    if (copy_tuning_init(32768, &g_tuning[dev]) != cudaSuccess) {  // occupancy queries only, no allocation
        cudaGetLastError();
        return AAF_ERR_CUDA;
    }
    g_sm_count[dev] = sms;
    g_scratch_ptr[dev] = static_cast<NoAllocScratch *>(ptr);
    return AAF_OK;
}

}  // namespace

extern "C" int aaf_kv_materialize_noalloc(const void *pool_base_dev, size_t layer_stride_bytes, int32_t n_layers,
                                          int32_t n_kv_heads, int32_t head_dim, int32_t block_size,
                                          int32_t elt_bytes, int32_t n_blocks, const int32_t *block_table_host,
                                          int32_t n_table_blocks, int64_t tok_begin, int64_t tok_end, void *dst_dev,
                                          size_t dst_bytes, void *stream) {
    if (!pool_base_dev || !block_table_host || !dst_dev) return AAF_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(pool_base_dev) & 15u) || (reinterpret_cast<uintptr_t>(dst_dev) & 15u))
        return AAF_ERR_INVALID_ARG;
    if (n_layers < 1 || n_kv_heads < 1 || head_dim < 1 || block_size < 1 || elt_bytes < 1 || n_blocks < 1 ||
        n_table_blocks < 1)
        return AAF_ERR_INVALID_ARG;
    // sizes are bounded before anything is multiplied: a row and a run fit 2^30 bytes, the layer count 2^16
    if (n_layers > 65536) return AAF_ERR_INVALID_ARG;
    long long row = 0, run = 0;
    if (__builtin_mul_overflow((long long)n_kv_heads, (long long)head_dim, &row) ||
        __builtin_mul_overflow(row, (long long)elt_bytes, &row) || row > (1ll << 30) ||
        __builtin_mul_overflow(row, (long long)block_size, &run) || run > (1ll << 30))
        return AAF_ERR_INVALID_ARG;
    if (row % 16 != 0) return AAF_ERR_INVALID_ARG;
    if (layer_stride_bytes % 16 != 0 || layer_stride_bytes < (size_t)(2 * run * n_blocks)) return AAF_ERR_INVALID_ARG;
    if (tok_begin < 0 || tok_begin >= tok_end || tok_end > (long long)n_table_blocks * block_size)
        return AAF_ERR_INVALID_ARG;
    const long long n = tok_end - tok_begin;
    const long long j0 = tok_begin / block_size, j1 = (tok_end - 1) / block_size;
    const long long nb = j1 - j0 + 1;
    if (nb > AAF_NOALLOC_MAX_BLOCKS) return AAF_ERR_SCRATCH_LIMIT;  // also bounds n: n <= 4096 * block_size
    // n <= 2^12 * block_size and block_size * row <= 2^30, so n * row <= 2^42; times 2 * n_layers <= 2^17: no overflow
    if ((unsigned long long)dst_bytes < (unsigned long long)(n * row) * 2ull * (unsigned long long)n_layers)
        return AAF_ERR_DST_TOO_SMALL;
    for (long long j = j0; j <= j1; ++j)
        if (block_table_host[j] < 0 || block_table_host[j] >= n_blocks) return AAF_ERR_INVALID_ARG;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return AAF_ERR_CUDA;
    // both buffers must be memory of the current device: the scratch and the launch shapes used below are
    // this device's (the query allocates nothing)
    for (const void *q : {pool_base_dev, static_cast<const void *>(dst_dev)}) {
        cudaPointerAttributes pa{};
        if (cudaPointerGetAttributes(&pa, q) != cudaSuccess) {
            cudaGetLastError();
            return AAF_ERR_INVALID_ARG;
        }
        if ((pa.type == cudaMemoryTypeDevice || pa.type == cudaMemoryTypeManaged) && pa.device != dev)
            return AAF_ERR_INVALID_ARG;
    }
    const int rc = setup_device(dev);
    if (rc != AAF_OK) return rc;
    NoAllocScratch *sc = g_scratch_ptr[dev];
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // the array keeps the previous call's contents: clear the counters, overwrite the table slice;
    // the planner rewrites every piece slot this call's copy launch reads
    if (cudaMemsetAsync(&sc->ctl, 0, sizeof(DevCtl), st) != cudaSuccess) return AAF_ERR_CUDA;
    if (cudaMemcpyAsync(sc->table, block_table_host + j0, sizeof(int) * (size_t)nb, cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
        return AAF_ERR_CUDA;

    Geom g{};
    g.L = n_layers; g.H = n_kv_heads; g.D = head_dim; g.BS = block_size; g.E = elt_bytes; g.NB = n_blocks;
    g.max_ctx = 1; g.max_blk = n_table_blocks;
    g.row = row; g.run = run; g.layer_stride = (long long)layer_stride_bytes;
    g.pool = static_cast<char *>(const_cast<void *>(pool_base_dev));
    DevState s{};
    s.ctl = &sc->ctl;
    s.tables = sc->table;  // holds entries j0 .. j1 of the caller's table: the planner subtracts j0
    s.pieces = sc->pieces;
    if (launch_plan_materialize(g, s, 0, tok_begin, tok_end, static_cast<char *>(dst_dev), 0, st, (int)j0) !=
        cudaSuccess)
        return AAF_ERR_CUDA;
    if (launch_copy(AAF_ENGINE_VEC, g_tuning[dev], g, s, (int)nb, 0, 2 * n_layers, run, g_sm_count[dev], st) !=
        cudaSuccess)
        return AAF_ERR_CUDA;
    return AAF_OK;
}
