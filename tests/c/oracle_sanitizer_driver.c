/* Drives the CPU oracle under AddressSanitizer / UBSan: round trips with ragged
 * sizes, every result code, and buffers allocated at their exact sizes so that
 * any read or write one byte outside a blob, a checksum array, a page table or a
 * cache shows up.  (The paper reports that a pass with address sanitizers found
 * an out-of-bounds read in its library; this is the same kind of pass for the
 * oracle.)  Exit code 0 = clean. */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "../../oracle/gk_oracle.h"
#include "../../oracle/gk_sha256_oracle.h"

static uint64_t rng_state = 0x9E3779B97F4A7C15ull;
static uint8_t rnd(void)
{
    rng_state ^= rng_state << 13;
    rng_state ^= rng_state >> 7;
    rng_state ^= rng_state << 17;
    return (uint8_t)(rng_state >> 32);
}

static int run(const ok_geom *g, uint32_t n_src, uint32_t n_dst, uint32_t n_tokens)
{
    uint64_t row = (uint64_t)g->kv_heads * g->head_dim * g->elem_bytes;
    uint64_t slab = row * g->page_tokens;
    uint64_t h4 = (uint64_t)g->kv_heads * 4;
    ok_cache src = {0}, dst = {0};
    src.num_pages = n_src; src.page_stride = slab; src.kv_stride = n_src * slab; src.layer_stride = 2 * n_src * slab;
    dst.num_pages = n_dst; dst.page_stride = slab; dst.kv_stride = n_dst * slab; dst.layer_stride = 2 * n_dst * slab;
    size_t sb = (size_t)(g->layers * 2 * n_src * slab), db = (size_t)(g->layers * 2 * n_dst * slab);
    src.data = malloc(sb); dst.data = malloc(db);
    for (size_t i = 0; i < sb; ++i) src.data[i] = rnd();
    for (size_t i = 0; i < db; ++i) dst.data[i] = rnd();
    if (g->scale_kv) {
        src.s_page_stride = h4; src.s_kv_stride = n_src * h4; src.s_layer_stride = g->scale_kv * n_src * h4;
        dst.s_page_stride = h4; dst.s_kv_stride = n_dst * h4; dst.s_layer_stride = g->scale_kv * n_dst * h4;
        size_t ss = (size_t)(g->layers * g->scale_kv * n_src * h4), ds = (size_t)(g->layers * g->scale_kv * n_dst * h4);
        src.scales = malloc(ss); dst.scales = malloc(ds);
        for (size_t i = 0; i < ss; ++i) src.scales[i] = rnd();
        for (size_t i = 0; i < ds; ++i) dst.scales[i] = rnd();
    }
    uint64_t nbytes; uint32_t P;
    if (ok_blob_size(g, n_tokens, &nbytes, &P) != 0) return 1;
    int32_t *spt = malloc(P * sizeof(int32_t)), *dpt = malloc(P * sizeof(int32_t));
    for (uint32_t p = 0; p < P; ++p) { spt[p] = (int32_t)(rnd() % n_src); dpt[p] = (int32_t)((p * 7u + 3u) % n_dst); }
    uint8_t *blob = malloc((size_t)nbytes);
    uint64_t *sums = malloc(P * sizeof(uint64_t));
    int32_t bad;
    if (ok_pack(g, &src, spt, n_tokens, blob, sums, &bad) != OK_CODE_OK) return 2;

    uint8_t *blob_bad = malloc((size_t)nbytes);
    memcpy(blob_bad, blob, (size_t)nbytes);
    blob_bad[nbytes - 1] ^= 0x80;
    int32_t *oob = malloc(P * sizeof(int32_t));
    memcpy(oob, dpt, P * sizeof(int32_t));
    oob[P - 1] = (int32_t)n_dst;
    ok_job jobs[4] = {
        {blob, sums, dpt, n_tokens},          /* ok (pages distinct when P <= n_dst) */
        {blob_bad, sums, dpt, n_tokens},      /* same pages: both claimants -> page table code */
        {NULL, sums, dpt, n_tokens},          /* missing */
        {blob, sums, oob, n_tokens},          /* out of range */
    };
    uint8_t mask[4]; int32_t fb[4];
    ok_restore(g, &dst, jobs, 4, 0, mask, fb);
    if (!(mask[0] == OK_CODE_PAGE_TABLE && mask[1] == OK_CODE_PAGE_TABLE && mask[2] == OK_CODE_MISSING &&
          mask[3] == OK_CODE_PAGE_TABLE)) return 3;
    ok_restore(g, &dst, jobs, 1, 0, mask, fb);
    if (mask[0] != OK_CODE_OK) return 4;
    ok_restore(g, &dst, jobs + 1, 1, 0, mask, fb);
    if (mask[0] != OK_CODE_CHECKSUM || fb[0] != (int32_t)P - 1) return 5;
    ok_restore(g, &dst, jobs + 1, 1, OK_FLAG_SKIP_VERIFY, mask, fb);
    if (mask[0] != OK_CODE_OK) return 6;
    /* round trip through the destination */
    uint8_t *blob2 = malloc((size_t)nbytes);
    uint64_t *sums2 = malloc(P * sizeof(uint64_t));
    ok_restore(g, &dst, jobs, 1, 0, mask, fb);
    if (ok_pack(g, &dst, dpt, n_tokens, blob2, sums2, &bad) != OK_CODE_OK) return 7;
    if (memcmp(blob, blob2, (size_t)nbytes) != 0 || memcmp(sums, sums2, P * sizeof(uint64_t)) != 0) return 8;
    if (ok_crc64(blob, (size_t)nbytes) != ok_crc64_bitwise(blob, (size_t)nbytes)) return 9;

    free(blob2); free(sums2); free(oob); free(blob_bad); free(sums); free(blob); free(dpt); free(spt);
    free(src.data); free(dst.data); free(src.scales); free(dst.scales);
    return 0;
}

/* fingerprints and digests on exact-size heap buffers */
static int run_sha(const ok_geom *g, uint32_t n_tokens)
{
    uint8_t out[32];
    for (size_t len = 0; len < 130; ++len) {
        uint8_t *m = malloc(len ? len : 1);
        for (size_t i = 0; i < len; ++i) m[i] = (uint8_t)(i * 7u + len);
        ok_sha256(len ? m : NULL, len, out);
        free(m);
    }
    uint64_t offsets[5] = {0, 0, 7, 64, 200};
    int32_t parent[4] = {-1, 0, 1, -1};
    uint8_t *data = malloc(200);
    for (int i = 0; i < 200; ++i) data[i] = (uint8_t)(i * 3);
    uint8_t model[32] = {1}, tenant[32] = {2};
    uint8_t *keys = malloc(4 * 32);
    if (ok_fingerprints(4, data, offsets, parent, model, tenant, keys) != 0) return 20;
    parent[2] = 2;
    if (ok_fingerprints(4, data, offsets, parent, model, tenant, keys) != -1) return 21;

    uint64_t nbytes = 0;
    uint32_t P = 0;
    ok_blob_size(g, n_tokens, &nbytes, &P);
    uint8_t *blob = malloc((size_t)nbytes);
    for (uint64_t i = 0; i < nbytes; ++i) blob[i] = (uint8_t)(i ^ (i >> 8));
    uint8_t *pages = malloc((size_t)P * 32);
    ok_blob_digest(g, blob, n_tokens, keys, pages, out);
    ok_blob_digest(g, blob, n_tokens, keys + 32, NULL, out);
    free(pages); free(blob); free(keys); free(data);
    return 0;
}

/* layer-wise save and load on exact-size buffers: 3 groups of g->layers layers */
static int run_layerwise(const ok_geom *g, uint32_t n_tokens)
{
    const uint32_t G = 3, N = 6;
    uint64_t slab = (uint64_t)g->page_tokens * g->kv_heads * g->head_dim * g->elem_bytes;
    uint32_t L = g->layers * G;
    ok_cache src = {0}, dst = {0};
    src.num_pages = dst.num_pages = N;
    src.page_stride = dst.page_stride = slab;
    src.kv_stride = dst.kv_stride = N * slab;
    src.layer_stride = dst.layer_stride = 2 * N * slab;
    src.data = malloc((size_t)(L * 2 * N * slab));
    dst.data = calloc((size_t)(L * 2 * N * slab), 1);
    for (uint64_t i = 0; i < L * 2 * N * slab; ++i) src.data[i] = (uint8_t)(i * 13u + 5u);
    if (g->scale_kv) {
        uint64_t h4 = g->kv_heads * 4u;
        src.s_page_stride = dst.s_page_stride = h4;
        src.s_kv_stride = dst.s_kv_stride = N * h4;
        src.s_layer_stride = dst.s_layer_stride = g->scale_kv * N * h4;
        src.scales = malloc((size_t)(L * g->scale_kv * N * h4));
        dst.scales = calloc((size_t)(L * g->scale_kv * N * h4), 1);
        for (uint64_t i = 0; i < L * g->scale_kv * N * h4; ++i) src.scales[i] = (uint8_t)(i * 7u);
    }
    uint64_t gbytes = 0;
    uint32_t P = 0;
    ok_blob_size(g, n_tokens, &gbytes, &P);
    int32_t *pt = malloc(P * sizeof(int32_t));
    for (uint32_t p = 0; p < P; ++p) pt[p] = (int32_t)((p * 5u + 1u) % N);
    uint8_t *blob = malloc((size_t)(G * gbytes));
    uint64_t *sums = malloc((size_t)G * P * sizeof(uint64_t));
    int32_t bad = 0;
    if (ok_pack_layerwise(g, G, &src, pt, n_tokens, blob, sums, &bad) != OK_CODE_OK) return 30;
    blob[gbytes + 1] ^= 0x10; /* damage in group 1 */
    ok_job job = {blob, sums, pt, n_tokens};
    uint8_t mask[1], gm[3];
    int32_t fb[1];
    ok_restore_layerwise(g, G, &dst, &job, 1, 0, mask, fb, gm, NULL, NULL);
    if (mask[0] != OK_CODE_CHECKSUM || gm[0] != 0 || gm[1] != OK_CODE_CHECKSUM || gm[2] != 0 || fb[0] != 0) return 31;
    free(sums); free(blob); free(pt); free(src.data); free(dst.data); free(src.scales); free(dst.scales);
    return 0;
}

int main(void)
{
    ok_geom bf16 = {3, 2, 8, 4, 2, 0};
    ok_geom fp8 = {2, 4, 8, 8, 1, 2};
    ok_geom fp8_shared = {2, 4, 8, 8, 1, 1};
    uint32_t lens[] = {1, 3, 4, 5, 17, 32};
    for (unsigned i = 0; i < sizeof(lens) / sizeof(lens[0]); ++i) {
        int rc;
        if ((rc = run(&bf16, 5, 11, lens[i])) != 0) { printf("bf16 len %u: %d\n", lens[i], rc); return 1; }
        if ((rc = run(&fp8, 5, 11, lens[i])) != 0) { printf("fp8 len %u: %d\n", lens[i], rc); return 1; }
        if ((rc = run(&fp8_shared, 5, 11, lens[i])) != 0) { printf("fp8/1 len %u: %d\n", lens[i], rc); return 1; }
    }
    ok_geom wide = {6, 4, 32, 8, 1, 2};   /* records of 12,480 bytes: three full digest chunks and a short one */
    if (run_layerwise(&bf16, 9) != 0 || run_layerwise(&fp8, 13) != 0) { printf("layerwise\n"); return 1; }
    if (run_sha(&bf16, 9) != 0 || run_sha(&wide, 17) != 0) { printf("sha\n"); return 1; }
    printf("clean\n");
    return 0;
}
