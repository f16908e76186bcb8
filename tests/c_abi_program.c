/*
 * A plain C caller of libaafkv.so: no Python, no PyTorch.  It owns the device memory itself
 * (cudaMalloc), drives the operators through the C ABI of include/aaf_kv.h and checks the bytes
 * of a fork / append / compose round against expectations written out token by token.
 * Built and run by tests/test_c_abi_program.py on a machine with a GPU.
 */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "aaf_kv.h"

#define CHECK(x)                                                                   \
    do {                                                                           \
        int rc_ = (x);                                                             \
        if (rc_ != 0) {                                                            \
            fprintf(stderr, "%s:%d: %s -> %d (%s)\n", __FILE__, __LINE__, #x, rc_, \
                    aaf_kv_strerror(rc_));                                         \
            return 1;                                                              \
        }                                                                          \
    } while (0)

enum { L = 2, H = 2, D = 16, BS = 4, E = 2, NB = 32, ROW = H * D * E, BPT = 2 * L * ROW };

/* byte j of row (layer l, K/V kv) of the token with identity `tok` */
static unsigned char token_byte(int tok, int l, int kv, int j) { return (unsigned char)(tok * 37 + l * 11 + kv * 5 + j); }

/* transfer buffer [L][2][n][ROW] of the tokens ids[0..n) */
static void encode(unsigned char *buf, const int *ids, int n) {
    for (int l = 0; l < L; ++l)
        for (int kv = 0; kv < 2; ++kv)
            for (int t = 0; t < n; ++t)
                for (int j = 0; j < ROW; ++j) buf[(((size_t)l * 2 + kv) * n + t) * ROW + j] = token_byte(ids[t], l, kv, j);
}

int main(void) {
    aaf_kv_pool_desc d;
    memset(&d, 0, sizeof(d));
    d.struct_size = sizeof(d);
    d.abi_version = AAF_KV_ABI_VERSION;
    d.n_layers = L; d.n_kv_heads = H; d.head_dim = D; d.block_size = BS; d.elt_bytes = E;
    d.n_blocks = NB; d.max_ctx = 8; d.max_blocks_per_ctx = 16; d.max_batch = 8; d.device = 0;
    d.model_id = 7; d.config_hash = 9;
    d.layer_stride_bytes = (size_t)NB * 2 * BS * ROW;
    d.workspace_bytes = aaf_kv_pool_workspace_bytes(&d);
    if (d.workspace_bytes == 0) return 2;
    if (cudaMalloc(&d.pool_base, (size_t)L * d.layer_stride_bytes) != cudaSuccess) return 3;
    if (cudaMalloc(&d.workspace, d.workspace_bytes) != cudaSuccess) return 3;
    aaf_kv_pool *pool = NULL;
    CHECK(aaf_kv_pool_create(&d, &pool));

    cudaStream_t st;
    if (cudaStreamCreate(&st) != cudaSuccess) return 3;
    unsigned char *dev_buf = NULL, *dev_out = NULL;
    if (cudaMalloc((void **)&dev_buf, 64 * BPT) != cudaSuccess || cudaMalloc((void **)&dev_out, 64 * BPT) != cudaSuccess)
        return 3;
    unsigned char *host = (unsigned char *)malloc(64 * BPT), *want = (unsigned char *)malloc(64 * BPT);

    /* root context: tokens 0..5 (one full block and a half-full tail) */
    int root_ids[6] = {0, 1, 2, 3, 4, 5};
    encode(host, root_ids, 6);
    cudaMemcpyAsync(dev_buf, host, 6 * BPT, cudaMemcpyHostToDevice, st);
    aaf_kv_xfer_desc xd = {7, 9, L, H, D, E, 0, 6};
    aaf_ctx_t root = -1, kids[2] = {-1, -1}, merged = -1;
    CHECK(aaf_kv_import(pool, dev_buf, &xd, &root, st));
    xd.model_id = 8; /* a descriptor of another model must be refused */
    if (aaf_kv_import(pool, dev_buf, &xd, &merged, st) != AAF_ERR_INCOMPAT) return 4;
    CHECK(aaf_kv_fork(pool, root, 2, kids, st));

    /* child 0 appends tokens 100, 101, 102: its shared tail is copied on write */
    int new_ids[3] = {100, 101, 102};
    encode(host, new_ids, 3);
    cudaStreamSynchronize(st);
    unsigned char *dev_new = dev_buf + 32 * BPT;
    cudaMemcpyAsync(dev_new, host, 3 * BPT, cudaMemcpyHostToDevice, st);
    int32_t n_new = 3;
    const void *srcs[1] = {dev_new};
    CHECK(aaf_kv_append(pool, 1, &kids[0], &n_new, srcs, st));

    /* merged = child 0 || child 1 = 0..5 100 101 102 0..5 */
    aaf_ctx_t segs[2] = {kids[0], kids[1]};
    CHECK(aaf_kv_compose(pool, 2, segs, AAF_COMPOSE_SHARE, &merged, st));
    int64_t len = 0;
    CHECK(aaf_kv_ctx_len(pool, merged, &len));
    if (len != 15) return 5;
    CHECK(aaf_kv_materialize(pool, merged, 0, 15, dev_out, 15 * BPT, &xd, st));
    cudaMemcpyAsync(host, dev_out, 15 * BPT, cudaMemcpyDeviceToHost, st);
    cudaStreamSynchronize(st);
    int all_ids[15] = {0, 1, 2, 3, 4, 5, 100, 101, 102, 0, 1, 2, 3, 4, 5};
    encode(want, all_ids, 15);
    if (memcmp(host, want, 15 * BPT) != 0) { fprintf(stderr, "merged context differs\n"); return 6; }
    if (xd.n_tokens != 15 || xd.model_id != 7) return 7;

    /* the parent is untouched by its child's append */
    CHECK(aaf_kv_materialize(pool, root, 0, 6, dev_out, 6 * BPT, NULL, st));
    cudaMemcpyAsync(host, dev_out, 6 * BPT, cudaMemcpyDeviceToHost, st);
    cudaStreamSynchronize(st);
    encode(want, root_ids, 6);
    if (memcmp(host, want, 6 * BPT) != 0) { fprintf(stderr, "parent changed\n"); return 8; }

    /* batched calls from C: two merges in one call, then both results gathered by one call into one buffer each */
    {
        const int32_t seg_off[3] = {0, 2, 3};
        const aaf_ctx_t bsegs[3] = {kids[1], kids[0], root}; /* merge 0 = child 1 || child 0, merge 1 = root alone */
        aaf_ctx_t outs[2] = {-1, -1};
        CHECK(aaf_kv_compose_batch(pool, 2, seg_off, bsegs, AAF_COMPOSE_SHARE, outs, st));
        const int64_t b0[2] = {0, 2}, b1[2] = {15, 6};
        void *dsts[2] = {dev_out, dev_out + 16 * BPT};
        const size_t caps[2] = {15 * BPT, 4 * BPT};
        CHECK(aaf_kv_materialize_batch(pool, 2, outs, b0, b1, dsts, caps, NULL, st));
        cudaMemcpyAsync(host, dev_out, 32 * BPT, cudaMemcpyDeviceToHost, st);
        cudaStreamSynchronize(st);
        int m0[15] = {0, 1, 2, 3, 4, 5, 0, 1, 2, 3, 4, 5, 100, 101, 102}, m1[4] = {2, 3, 4, 5};
        encode(want, m0, 15);
        if (memcmp(host, want, 15 * BPT) != 0) { fprintf(stderr, "batched merge 0 differs\n"); return 12; }
        encode(want, m1, 4);
        if (memcmp(host + 16 * BPT, want, 4 * BPT) != 0) { fprintf(stderr, "batched gather 1 differs\n"); return 13; }
        /* register both buffers as new contexts in one call, then drop the four batch products again */
        const void *srcs2[2] = {dev_out, dev_out + 16 * BPT};
        aaf_kv_xfer_desc xds[2] = {{7, 9, L, H, D, E, 0, 15}, {7, 9, L, H, D, E, 2, 4}};
        aaf_ctx_t regs[2] = {-1, -1};
        CHECK(aaf_kv_import_batch(pool, 2, srcs2, xds, regs, st));
        aaf_ctx_t drop[4] = {outs[0], outs[1], regs[0], regs[1]};
        CHECK(aaf_kv_evict(pool, 4, drop, st));
    }

    /* reference counts are conserved; evicting everything returns every block */
    int32_t rc[NB], fl[NB], nfree = 0, sum = 0;
    CHECK(aaf_kv_get_refcounts(pool, rc));
    for (int b = 0; b < NB; ++b) sum += rc[b];
    if (sum != 2 + 3 + 2 + 4) return 9; /* table lengths of root, child 0, child 1, merged */
    aaf_ctx_t all[4] = {root, kids[0], kids[1], merged};
    CHECK(aaf_kv_evict(pool, 4, all, st));
    CHECK(aaf_kv_get_free_list(pool, fl, &nfree));
    if (nfree != NB) return 10;
    if (aaf_kv_sync_status(pool) != AAF_OK) return 11;
    CHECK(aaf_kv_pool_destroy(pool));
    cudaFree(d.pool_base); cudaFree(d.workspace); cudaFree(dev_buf); cudaFree(dev_out);
    free(host); free(want);
    printf("c abi ok\n");
    return 0;
}
