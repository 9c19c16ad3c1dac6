/*
 * gk_oracle.c -- CPU oracle (test infrastructure only; see gk_oracle.h).
 *
 * Written for checking by eye: one loop nest per definition, no blocking, no
 * threads, no SIMD.  Nothing here is shared with, or derived from, the CUDA
 * path.
 */
#include "gk_oracle.h"

#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------
 * CRC-64/XZ.  Catalogue parameters: width 64, polynomial 0x42F0E1EBA9EA3693,
 * init all ones, input and output reflected, final xor all ones.  In the
 * reflected formulation the register shifts right and the polynomial constant
 * is the bit-reversed one.
 * ---------------------------------------------------------------------- */
#define OK_POLY_REFLECTED 0xC96C5795D7870F42ull

static uint64_t crc_step_byte(uint64_t reg, uint8_t byte)
{
    reg ^= (uint64_t)byte;
    for (int bit = 0; bit < 8; ++bit) {
        if (reg & 1ull)
            reg = (reg >> 1) ^ OK_POLY_REFLECTED;
        else
            reg = reg >> 1;
    }
    return reg;
}

uint64_t ok_crc64_bitwise(const uint8_t *data, size_t len)
{
    uint64_t reg = ~0ull;
    for (size_t i = 0; i < len; ++i)
        reg = crc_step_byte(reg, data[i]);
    return ~reg;
}

static uint64_t g_table[256];
static int g_table_ready = 0;

static void table_init(void)
{
    /* entry b = the register after feeding byte b into an all-zero register */
    for (int b = 0; b < 256; ++b)
        g_table[b] = crc_step_byte(0ull, (uint8_t)b);
    g_table_ready = 1;
}

uint64_t ok_crc64_continue(uint64_t crc_so_far, const uint8_t *data, size_t len)
{
    if (!g_table_ready)
        table_init();
    uint64_t reg = ~crc_so_far; /* undo the final xor to get the register back */
    for (size_t i = 0; i < len; ++i)
        reg = g_table[(uint8_t)(reg ^ data[i])] ^ (reg >> 8);
    return ~reg;
}

uint64_t ok_crc64(const uint8_t *data, size_t len)
{
    /* the CRC of the empty string is 0, whose register is all ones = init */
    return ok_crc64_continue(0ull, data, len);
}

/* ------------------------------------------------------------------------
 * Geometry.
 * ---------------------------------------------------------------------- */
static uint64_t row_bytes(const ok_geom *g)
{
    return (uint64_t)g->kv_heads * g->head_dim * g->elem_bytes;
}

static uint64_t scale_section_bytes(const ok_geom *g)
{
    return (uint64_t)g->layers * g->scale_kv * g->kv_heads * 4u;
}

static uint32_t page_count(const ok_geom *g, uint32_t n_tokens)
{
    /* ceil(n / T), in 64 bits so that n close to 2^32 does not wrap */
    return (uint32_t)(((uint64_t)n_tokens + g->page_tokens - 1u) / g->page_tokens);
}

/* tokens held by logical page p of a block of n_tokens */
static uint32_t tokens_in_page(const ok_geom *g, uint32_t n_tokens, uint32_t p)
{
    uint32_t P = page_count(g, n_tokens);
    if (p + 1u < P)
        return g->page_tokens;
    return n_tokens - (P - 1u) * g->page_tokens;
}

uint64_t ok_record_bytes(const ok_geom *g, uint32_t n_tokens, uint32_t p)
{
    return scale_section_bytes(g) +
           (uint64_t)tokens_in_page(g, n_tokens, p) * 2u * g->layers * row_bytes(g);
}

uint64_t ok_record_offset(const ok_geom *g, uint32_t p)
{
    /* every earlier page is full */
    uint64_t full = scale_section_bytes(g) + (uint64_t)g->page_tokens * 2u * g->layers * row_bytes(g);
    return (uint64_t)p * full;
}

int ok_blob_size(const ok_geom *g, uint32_t n_tokens, uint64_t *blob_bytes, uint32_t *n_pages)
{
    if (!g || n_tokens == 0 || g->page_tokens == 0)
        return -1;
    uint32_t P = page_count(g, n_tokens);
    uint64_t total = 0;
    for (uint32_t p = 0; p < P; ++p)
        total += ok_record_bytes(g, n_tokens, p);
    if (blob_bytes)
        *blob_bytes = total;
    if (n_pages)
        *n_pages = P;
    return 0;
}

static uint8_t *slab_ptr(const ok_cache *c, uint32_t l, uint32_t kv, int32_t page)
{
    return c->data + (uint64_t)l * c->layer_stride + (uint64_t)kv * c->kv_stride +
           (uint64_t)page * c->page_stride;
}

static uint8_t *scale_ptr(const ok_cache *c, uint32_t l, uint32_t kv, int32_t page, uint32_t h)
{
    return c->scales + (uint64_t)l * c->s_layer_stride + (uint64_t)kv * c->s_kv_stride +
           (uint64_t)page * c->s_page_stride + 4ull * h;
}

/* Copies the valid part of one slab (the first t tokens) between a cache slab and
 * a record: one contiguous prefix for a token-major slab, one prefix per head for
 * a head-major slab.  to_record != 0: slab -> record, else record -> slab. */
static uint64_t copy_slab_prefix(const ok_geom *g, uint8_t *slab, uint8_t *rec, uint32_t t, int to_record)
{
    uint64_t row = row_bytes(g);
    if (!g->head_major) {
        if (to_record)
            memcpy(rec, slab, (size_t)(t * row));
        else
            memcpy(slab, rec, (size_t)(t * row));
        return t * row;
    }
    uint64_t tok = (uint64_t)g->head_dim * g->elem_bytes;       /* one token of one head */
    uint64_t head_block = (uint64_t)g->page_tokens * tok;       /* one head's part of the slab */
    for (uint32_t h = 0; h < g->kv_heads; ++h) {
        if (to_record)
            memcpy(rec + h * t * tok, slab + h * head_block, (size_t)(t * tok));
        else
            memcpy(slab + h * head_block, rec + h * t * tok, (size_t)(t * tok));
    }
    return t * row;
}

static int32_t lowest_out_of_range(const int32_t *pt, uint32_t P, uint64_t num_pages)
{
    for (uint32_t p = 0; p < P; ++p)
        if (pt[p] < 0 || (uint64_t)pt[p] >= num_pages)
            return (int32_t)p;
    return -1;
}

/* ------------------------------------------------------------------------
 * Save (pack).
 * ---------------------------------------------------------------------- */
int ok_pack(const ok_geom *g, const ok_cache *src, const int32_t *page_table,
            uint32_t n_tokens, uint8_t *blob, uint64_t *checksums, int32_t *bad_index)
{
    uint32_t P = page_count(g, n_tokens);
    int32_t bad = lowest_out_of_range(page_table, P, src->num_pages);
    if (bad_index)
        *bad_index = bad;
    if (bad >= 0)
        return OK_CODE_PAGE_TABLE;

    for (uint32_t p = 0; p < P; ++p) {
        uint8_t *rec = blob + ok_record_offset(g, p);
        uint8_t *w = rec;
        int32_t page = page_table[p];
        uint32_t t = tokens_in_page(g, n_tokens, p);

        for (uint32_t l = 0; l < g->layers; ++l)
            for (uint32_t kv = 0; kv < g->scale_kv; ++kv)
                for (uint32_t h = 0; h < g->kv_heads; ++h) {
                    memcpy(w, scale_ptr(src, l, kv, page, h), 4);
                    w += 4;
                }
        for (uint32_t l = 0; l < g->layers; ++l)
            for (uint32_t kv = 0; kv < 2; ++kv)
                w += copy_slab_prefix(g, slab_ptr(src, l, kv, page), w, t, 1);
        checksums[p] = ok_crc64(rec, (size_t)(w - rec));
    }
    return OK_CODE_OK;
}

/* ------------------------------------------------------------------------
 * Load (restore): verify everything, then commit what passed.
 * ---------------------------------------------------------------------- */
void ok_restore(const ok_geom *g, const ok_cache *dst, const ok_job *jobs, uint32_t n_jobs,
                uint32_t flags, uint8_t *mask, int32_t *first_bad)
{
    uint32_t *claims = (uint32_t *)calloc(dst->num_pages ? dst->num_pages : 1, sizeof(uint32_t));

    /* ---- phase 1a: missing records, ids out of range ---- */
    for (uint32_t j = 0; j < n_jobs; ++j) {
        const ok_job *job = &jobs[j];
        mask[j] = OK_CODE_OK;
        first_bad[j] = -1;
        if (job->blob == NULL || job->checksums == NULL) {
            mask[j] = OK_CODE_MISSING;
            continue;
        }
        int32_t bad = lowest_out_of_range(job->page_table, page_count(g, job->n_tokens), dst->num_pages);
        if (bad >= 0) {
            mask[j] = OK_CODE_PAGE_TABLE;
            first_bad[j] = bad;
        }
    }
    /* ---- phase 1b: a destination page may be claimed once per call ---- */
    for (uint32_t j = 0; j < n_jobs; ++j) {
        if (mask[j] != OK_CODE_OK)
            continue;
        uint32_t P = page_count(g, jobs[j].n_tokens);
        for (uint32_t p = 0; p < P; ++p)
            claims[jobs[j].page_table[p]] += 1u;
    }
    for (uint32_t j = 0; j < n_jobs; ++j) {
        if (mask[j] != OK_CODE_OK)
            continue;
        uint32_t P = page_count(g, jobs[j].n_tokens);
        for (uint32_t p = 0; p < P; ++p)
            if (claims[jobs[j].page_table[p]] > 1u) {
                mask[j] = OK_CODE_PAGE_TABLE;
                first_bad[j] = (int32_t)p;
                break;
            }
    }
    /* ---- phase 1c: every page record against its stored checksum ---- */
    if (!(flags & OK_FLAG_SKIP_VERIFY)) {
        for (uint32_t j = 0; j < n_jobs; ++j) {
            if (mask[j] != OK_CODE_OK)
                continue;
            uint32_t P = page_count(g, jobs[j].n_tokens);
            for (uint32_t p = 0; p < P; ++p) {
                const uint8_t *rec = jobs[j].blob + ok_record_offset(g, p);
                uint64_t crc = ok_crc64(rec, (size_t)ok_record_bytes(g, jobs[j].n_tokens, p));
                if (crc != jobs[j].checksums[p]) {
                    mask[j] = OK_CODE_CHECKSUM;
                    first_bad[j] = (int32_t)p;
                    break;
                }
            }
        }
    }
    /* ---- phase 2: commit the jobs that passed; nothing else is written ----
     * (single-pass reading: a job whose only fault is a checksum mismatch is written too) */
    for (uint32_t j = 0; j < n_jobs; ++j) {
        int write_it = mask[j] == OK_CODE_OK ||
                       ((flags & OK_FLAG_SINGLE_PASS) && mask[j] == OK_CODE_CHECKSUM);
        if (!write_it)
            continue;
        uint32_t P = page_count(g, jobs[j].n_tokens);
        for (uint32_t p = 0; p < P; ++p) {
            const uint8_t *r = jobs[j].blob + ok_record_offset(g, p);
            int32_t page = jobs[j].page_table[p];
            uint32_t t = tokens_in_page(g, jobs[j].n_tokens, p);

            for (uint32_t l = 0; l < g->layers; ++l)
                for (uint32_t kv = 0; kv < g->scale_kv; ++kv)
                    for (uint32_t h = 0; h < g->kv_heads; ++h) {
                        memcpy(scale_ptr(dst, l, kv, page, h), r, 4);
                        r += 4;
                    }
            for (uint32_t l = 0; l < g->layers; ++l)
                for (uint32_t kv = 0; kv < 2; ++kv)
                    r += copy_slab_prefix(g, slab_ptr(dst, l, kv, page), (uint8_t *)r, t, 0);
        }
    }
    free(claims);
}

/* ------------------------------------------------------------------------
 * Streaming load: windows of consecutive jobs through one small cache.
 * ---------------------------------------------------------------------- */
int ok_restore_stream(const ok_geom *g, const ok_cache *ring, const ok_job *jobs, uint32_t n_jobs,
                      uint32_t flags, uint8_t *mask, int32_t *first_bad, ok_window_fn consume, void *user)
{
    for (uint32_t j = 0; j < n_jobs; ++j)
        if ((uint64_t)page_count(g, jobs[j].n_tokens) > ring->num_pages)
            return -1;

    int32_t *ids = (int32_t *)malloc((size_t)(ring->num_pages ? ring->num_pages : 1) * sizeof(int32_t));
    for (uint64_t i = 0; i < ring->num_pages; ++i)
        ids[i] = (int32_t)i;
    ok_job *wjobs = (ok_job *)malloc((size_t)(n_jobs ? n_jobs : 1) * sizeof(ok_job));
    uint32_t *first_page = (uint32_t *)malloc((size_t)(n_jobs ? n_jobs : 1) * sizeof(uint32_t));

    uint32_t j0 = 0;
    while (j0 < n_jobs) {
        /* the longest run of jobs from j0 that fits */
        uint64_t used = 0;
        uint32_t j1 = j0;
        while (j1 < n_jobs && used + page_count(g, jobs[j1].n_tokens) <= ring->num_pages) {
            first_page[j1 - j0] = (uint32_t)used;
            wjobs[j1 - j0] = jobs[j1];
            wjobs[j1 - j0].page_table = ids + used;
            used += page_count(g, jobs[j1].n_tokens);
            ++j1;
        }
        ok_restore(g, ring, wjobs, j1 - j0, flags, mask + j0, first_bad + j0);
        if (consume)
            consume(user, j0, j1 - j0, first_page);
        j0 = j1;
    }
    free(first_page);
    free(wjobs);
    free(ids);
    return 0;
}

/* ------------------------------------------------------------------------
 * Layer-wise save and load: the ordinary format, once per group of layers.
 * ---------------------------------------------------------------------- */
static ok_cache layer_view(const ok_geom *g, const ok_cache *c, uint32_t group)
{
    ok_cache v = *c;
    v.data = c->data + (uint64_t)group * g->layers * c->layer_stride;
    if (c->scales)
        v.scales = c->scales + (uint64_t)group * g->layers * c->s_layer_stride;
    return v;
}

int ok_pack_layerwise(const ok_geom *g, uint32_t n_groups, const ok_cache *src, const int32_t *page_table,
                      uint32_t n_tokens, uint8_t *blob, uint64_t *checksums, int32_t *bad_index)
{
    uint64_t group_bytes = 0;
    uint32_t P = 0;
    ok_blob_size(g, n_tokens, &group_bytes, &P);
    for (uint32_t k = 0; k < n_groups; ++k) {
        ok_cache view = layer_view(g, src, k);
        int code = ok_pack(g, &view, page_table, n_tokens, blob + k * group_bytes, checksums + (uint64_t)k * P,
                           bad_index);
        if (code != OK_CODE_OK)
            return code; /* a bad table is bad for every group: group 0 reports it, nothing was written */
    }
    return OK_CODE_OK;
}

void ok_restore_layerwise(const ok_geom *g, uint32_t n_groups, const ok_cache *dst, const ok_job *jobs,
                          uint32_t n_jobs, uint32_t flags, uint8_t *mask, int32_t *first_bad,
                          uint8_t *group_mask, ok_group_fn consume, void *user)
{
    ok_job *gjobs = (ok_job *)malloc((size_t)(n_jobs ? n_jobs : 1) * sizeof(ok_job));
    uint8_t *gm = (uint8_t *)malloc(n_jobs ? n_jobs : 1);
    int32_t *gfb = (int32_t *)malloc((size_t)(n_jobs ? n_jobs : 1) * sizeof(int32_t));
    for (uint32_t j = 0; j < n_jobs; ++j) {
        mask[j] = OK_CODE_OK;
        first_bad[j] = -1;
    }
    for (uint32_t k = 0; k < n_groups; ++k) {
        for (uint32_t j = 0; j < n_jobs; ++j) {
            uint64_t group_bytes = 0;
            uint32_t P = 0;
            ok_blob_size(g, jobs[j].n_tokens, &group_bytes, &P);
            gjobs[j] = jobs[j];
            if (jobs[j].blob)
                gjobs[j].blob = jobs[j].blob + k * group_bytes;
            if (jobs[j].checksums)
                gjobs[j].checksums = jobs[j].checksums + (uint64_t)k * P;
        }
        ok_cache view = layer_view(g, dst, k);
        ok_restore(g, &view, gjobs, n_jobs, flags, gm, gfb);
        for (uint32_t j = 0; j < n_jobs; ++j) {
            if (group_mask)
                group_mask[(uint64_t)k * n_jobs + j] = gm[j];
            if (mask[j] == OK_CODE_OK && gm[j] != OK_CODE_OK)
                first_bad[j] = gfb[j]; /* the lowest failing group decides the reported page */
            if (gm[j] > mask[j])
                mask[j] = gm[j];
        }
        if (consume)
            consume(user, k, k * g->layers, g->layers);
    }
    free(gfb);
    free(gm);
    free(gjobs);
}
