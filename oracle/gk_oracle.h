/*
 * gk_oracle.h -- CPU oracle for the save/restore path of a block's KV state.
 *
 * TEST INFRASTRUCTURE ONLY.  This is the slow, plain definition that the CUDA
 * library is compared against.  It shares no source, header, table or helper
 * with the CUDA path; only tests, the smoke check and the benchmark's CPU
 * baseline may call it.
 *
 * What it follows (paper, Section 2.2 "Taliesin: KV memory"): the KV state of a
 * block of prompt text is written to storage after it is computed, loaded again
 * when the same block recurs, checked when loaded, and -- by that section's
 * design rule that wrong stored state must never be served -- any record that is
 * missing, damaged or fails a check is not used: the block is recomputed.  Section 3
 * (Table 1) demands that what is restored is bit-identical to what was saved;
 * Section 5 states that reuse is at whole-block granularity and that the design
 * is fail-closed.  The paper withholds its storage format (end of Section 1),
 * so the page-record layout, the checksum (CRC-64/XZ per page record) and the
 * result codes below are this build's own definitions.
 *
 * Layout definitions
 *   cache   : opaque bytes.  The slab of (layer l, kv, page g) starts at
 *             data + l*layer_stride + kv*kv_stride + g*page_stride and holds
 *             page_tokens rows of row = kv_heads*head_dim*elem_bytes bytes,
 *             token-major ([t][h][d]).  kv = 0 is K, kv = 1 is V.  With
 *             head_major = 1 the slab is [h][t][d] instead: head h owns
 *             page_tokens*head_dim*elem_bytes contiguous bytes.
 *   scales  : (fp8 caches only) fp32 per (l, kv < scale_kv, page g, head h) at
 *             scales + l*s_layer_stride + kv*s_kv_stride + g*s_page_stride + 4*h.
 *   blob    : page records 0..P-1 back to back, no header, no padding.  Record
 *             p = [scale section: for l, for kv < scale_kv, for h: 4 bytes]
 *             then for l: K prefix (t_p*row bytes), V prefix (t_p*row bytes),
 *             where t_p = page_tokens except for a shorter last page.  The
 *             prefix of a head-major slab is, head by head, the first t_p
 *             tokens of that head (for a full page: the whole slab as it is).
 *   checksum: CRC-64/XZ over the bytes of record p, one uint64 per page.
 *
 * All pins for these functions are listed in tests/test_oracle_pins.py.
 */
#ifndef GK_ORACLE_H
#define GK_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    uint32_t layers;
    uint32_t kv_heads;
    uint32_t head_dim;
    uint32_t page_tokens;
    uint32_t elem_bytes; /* 2 for bf16, 1 for fp8 e4m3 */
    uint32_t scale_kv;   /* 0: no scale section; 1: one scale per (l,page,h); 2: K and V scales */
    uint32_t head_major; /* 0: a slab is [token][head][dim]; 1: a slab is [head][token][dim] */
} ok_geom;

typedef struct {
    uint8_t *data;
    uint64_t num_pages;
    uint64_t layer_stride, kv_stride, page_stride; /* bytes */
    uint8_t *scales; /* NULL when scale_kv == 0 */
    uint64_t s_layer_stride, s_kv_stride, s_page_stride; /* bytes */
} ok_cache;

typedef struct {
    const uint8_t *blob;       /* NULL: the record is missing */
    const uint64_t *checksums; /* NULL: the record is missing */
    const int32_t *page_table; /* P logical -> physical page ids */
    uint32_t n_tokens;
} ok_job;

/* result codes per job */
enum {
    OK_CODE_OK = 0,        /* verified and committed */
    OK_CODE_CHECKSUM = 1,  /* some page record failed its checksum */
    OK_CODE_PAGE_TABLE = 2,/* id out of range, or a page claimed twice in the call */
    OK_CODE_MISSING = 3    /* no record */
};

#define OK_FLAG_SKIP_VERIFY 1u /* sabotage tests: switch the checksum defence off */
/* Single-pass load.  Section 2.2 has the runtime recompute a block whose record
 * fails a check, which overwrites the block's pages anyway; under this optional
 * reading a block whose only fault is a checksum mismatch is still reported with
 * code 1, but its destination pages receive the record bytes as they are
 * (unverified).  Blocks with code 2 or 3 still write nothing, and nothing
 * outside the reported block's own pages changes.  Off by default. */
#define OK_FLAG_SINGLE_PASS 4u

/* CRC-64/XZ by its bit-at-a-time definition. */
uint64_t ok_crc64_bitwise(const uint8_t *data, size_t len);
/* Same value, one table lookup per byte; the table is generated from the
 * bit-at-a-time step on first use. */
uint64_t ok_crc64(const uint8_t *data, size_t len);
/* Continue a CRC: ok_crc64_continue(ok_crc64(A), B) == ok_crc64(A || B). */
uint64_t ok_crc64_continue(uint64_t crc_so_far, const uint8_t *data, size_t len);

/* Sizes of a block of n_tokens: pages P = ceil(n/T), blob bytes = P*S + n*tokB. */
int ok_blob_size(const ok_geom *g, uint32_t n_tokens, uint64_t *blob_bytes, uint32_t *n_pages);
/* Bytes of page record p of a block of n_tokens, and its offset in the blob. */
uint64_t ok_record_bytes(const ok_geom *g, uint32_t n_tokens, uint32_t p);
uint64_t ok_record_offset(const ok_geom *g, uint32_t p);

/* Save: gather the block's pages into blob and checksum each record.
 * Returns OK_CODE_OK, or OK_CODE_PAGE_TABLE (nothing written) if an id is
 * outside [0, num_pages); *bad_index then holds the lowest offending index. */
int ok_pack(const ok_geom *g, const ok_cache *src, const int32_t *page_table,
            uint32_t n_tokens, uint8_t *blob, uint64_t *checksums, int32_t *bad_index);

/* Load: phase 1 validates and verifies every job without writing; phase 2
 * commits the jobs whose code is 0.  mask[j] gets the code, first_bad[j] the
 * lowest failing page index (codes 1, 2) or -1. */
void ok_restore(const ok_geom *g, const ok_cache *dst, const ok_job *jobs, uint32_t n_jobs,
                uint32_t flags, uint8_t *mask, int32_t *first_bad);

/* Streaming load through a cache that is smaller than the corpus (Section 4.3,
 * the long-window paragraph: saved blocks are streamed in and dropped after
 * use, so that the size of the corpus is bounded by storage, not GPU memory).
 * The jobs' own page tables are ignored.  Jobs are taken in order and grouped
 * into windows: a window is the longest run of consecutive jobs whose pages fit
 * the cache together; inside a window the jobs get consecutive page ids from 0
 * (every job takes ceil(n_tokens/page_tokens) pages, whatever its result).  Each
 * window is one ok_restore; after it `consume` (may be NULL) is called with the
 * index of the window's first job, its job count, and each job's first page id;
 * then the pages are reused by the next window.  mask and first_bad cover all
 * jobs.  Returns 0, or -1 (nothing done) if a single job has more pages than
 * the cache. */
typedef void (*ok_window_fn)(void *user, uint32_t first_job, uint32_t n_jobs, const uint32_t *first_page);
int ok_restore_stream(const ok_geom *g, const ok_cache *ring, const ok_job *jobs, uint32_t n_jobs,
                      uint32_t flags, uint8_t *mask, int32_t *first_bad, ok_window_fn consume, void *user);

/* Layer-wise save and load.  A block's record is cut by layer groups so that a
 * consumer that walks the layers in order can start on the first layers while
 * the later ones are still arriving from storage (the streaming of saved state
 * in Section 4.3; the paper gives no format).  g describes ONE GROUP (g->layers
 * = layers per group); the cache holds n_groups * g->layers layers.  The
 * layer-wise blob of a block is the concatenation, for group k = 0..n_groups-1,
 * of the ordinary blob (as ok_pack makes it) of the cache restricted to the
 * layers [k*g->layers, (k+1)*g->layers); the checksums are those blobs'
 * checksums, group after group (n_groups * P values).
 * ok_restore_layerwise loads group after group, each as one ok_restore of all
 * jobs over the restricted cache: fail-closed holds per (job, group).  mask[j]
 * is the largest code over the groups, first_bad[j] the page of the lowest
 * failing group (or -1); group_mask (n_groups * n_jobs, may be NULL) receives
 * every group's codes.  `consume` (may be NULL) is called after each group. */
typedef void (*ok_group_fn)(void *user, uint32_t group, uint32_t first_layer, uint32_t n_layers);
int ok_pack_layerwise(const ok_geom *g, uint32_t n_groups, const ok_cache *src, const int32_t *page_table,
                      uint32_t n_tokens, uint8_t *blob, uint64_t *checksums, int32_t *bad_index);
void ok_restore_layerwise(const ok_geom *g, uint32_t n_groups, const ok_cache *dst, const ok_job *jobs,
                          uint32_t n_jobs, uint32_t flags, uint8_t *mask, int32_t *first_bad,
                          uint8_t *group_mask, ok_group_fn consume, void *user);

#ifdef __cplusplus
}
#endif
#endif
