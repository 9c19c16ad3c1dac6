/* libgk from plain C, without Python or torch: device memory from the CUDA runtime's C API,
 * a save, a clean load, a load of a damaged record.  Prints "roundtrip ok" on success. */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "../../include/gk.h"

#define CHECK(x) do { if ((x) != cudaSuccess) { printf("cuda error at line %d\n", __LINE__); return 10; } } while (0)

int main(void)
{
    gk_geom g = {4, 4, 64, 16, GK_BF16, 0, 0, 0};
    const uint32_t n_tokens = 3 * 16 + 5; /* a partial last page */
    const uint64_t slab = 16ull * 4 * 64 * 2;
    const uint64_t N = 9;
    const uint64_t cache_bytes = 2ull * g.layers * N * slab;
    uint64_t blob_bytes = 0;
    uint32_t P = 0;
    if (gk_blob_size(&g, n_tokens, &blob_bytes, &P) != GK_OK || P != 4) return 1;

    uint8_t *h_src = malloc(cache_bytes), *h_dst = malloc(cache_bytes), *h_back = malloc(cache_bytes);
    for (uint64_t i = 0; i < cache_bytes; ++i) {
        h_src[i] = (uint8_t)(i * 2654435761u >> 13);
        h_dst[i] = (uint8_t)(0xA5u ^ (i >> 3));
    }
    uint8_t *d_src, *d_dst, *d_blob, *d_mask;
    uint64_t *d_sums;
    int32_t *d_spt, *d_dpt, *d_fb;
    CHECK(cudaMalloc((void **)&d_src, cache_bytes));
    CHECK(cudaMalloc((void **)&d_dst, cache_bytes));
    CHECK(cudaMalloc((void **)&d_blob, blob_bytes));
    CHECK(cudaMalloc((void **)&d_sums, P * 8));
    CHECK(cudaMalloc((void **)&d_spt, P * 4));
    CHECK(cudaMalloc((void **)&d_dpt, P * 4));
    CHECK(cudaMalloc((void **)&d_mask, 1));
    CHECK(cudaMalloc((void **)&d_fb, 4));
    const int32_t spt[4] = {7, 2, 5, 0}, dpt[4] = {1, 8, 3, 6};
    CHECK(cudaMemcpy(d_src, h_src, cache_bytes, cudaMemcpyHostToDevice));
    CHECK(cudaMemcpy(d_dst, h_dst, cache_bytes, cudaMemcpyHostToDevice));
    CHECK(cudaMemcpy(d_spt, spt, sizeof spt, cudaMemcpyHostToDevice));
    CHECK(cudaMemcpy(d_dpt, dpt, sizeof dpt, cudaMemcpyHostToDevice));

    gk_ctx *ctx = NULL;
    if (gk_ctx_create(&ctx, &g, 0) != GK_OK) return 2;
    gk_cache src = {d_src, N, 2 * N * slab, N * slab, slab, NULL, 0, 0, 0};
    gk_cache dst = {d_dst, N, 2 * N * slab, N * slab, slab, NULL, 0, 0, 0};
    if (gk_pack(ctx, &src, d_spt, n_tokens, d_blob, d_sums, NULL, NULL) != GK_OK) return 3;

    /* a damaged copy of the record first: it must be reported and must write nothing */
    uint8_t *h_blob = malloc(blob_bytes);
    CHECK(cudaMemcpy(h_blob, d_blob, blob_bytes, cudaMemcpyDeviceToHost));
    h_blob[blob_bytes / 2] ^= 0x01;
    uint8_t *d_bad;
    CHECK(cudaMalloc((void **)&d_bad, blob_bytes));
    CHECK(cudaMemcpy(d_bad, h_blob, blob_bytes, cudaMemcpyHostToDevice));
    gk_job job = {d_bad, d_sums, d_dpt, n_tokens, 0};
    if (gk_restore(ctx, &job, 1, &dst, d_mask, d_fb, NULL) != GK_OK) return 4;
    CHECK(cudaDeviceSynchronize());
    uint8_t mask = 0xff;
    int32_t fb = -7;
    CHECK(cudaMemcpy(&mask, d_mask, 1, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(&fb, d_fb, 4, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(h_back, d_dst, cache_bytes, cudaMemcpyDeviceToHost));
    if (mask != GK_JOB_CHECKSUM || fb != 1 || memcmp(h_back, h_dst, cache_bytes) != 0) return 5;

    /* the intact record */
    job.blob = d_blob;
    if (gk_restore(ctx, &job, 1, &dst, d_mask, d_fb, NULL) != GK_OK) return 6;
    CHECK(cudaDeviceSynchronize());
    CHECK(cudaMemcpy(&mask, d_mask, 1, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(h_back, d_dst, cache_bytes, cudaMemcpyDeviceToHost));
    if (mask != GK_JOB_OK) return 7;
    const uint64_t row = 4ull * 64 * 2;
    for (uint32_t l = 0; l < g.layers; ++l)
        for (uint32_t kv = 0; kv < 2; ++kv)
            for (uint64_t page = 0; page < N; ++page) {
                int p = -1;
                for (int q = 0; q < 4; ++q)
                    if ((uint64_t)dpt[q] == page) p = q;
                const uint64_t off = (2ull * l + kv) * N * slab + page * slab;
                const uint64_t valid = p < 0 ? 0 : (p < 3 ? 16 : 5) * row; /* tokens of the page that were saved */
                if (p >= 0 && memcmp(h_back + off, h_src + (2ull * l + kv) * N * slab + (uint64_t)spt[p] * slab, valid) != 0)
                    return 8;
                if (memcmp(h_back + off + valid, h_dst + off + valid, slab - valid) != 0) return 9;
            }
    gk_stats st;
    if (gk_get_stats(ctx, &st) != GK_OK || st.device_wait_expired != 0 || st.calls_restore != 2) return 11;
    gk_ctx_destroy(ctx);
    printf("roundtrip ok\n");
    return 0;
}
