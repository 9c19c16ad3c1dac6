/*
 * gk.h -- C ABI of libgk: save and restore of a text block's KV state on one
 * NVIDIA B200 (sm_100a).
 *
 * The operations are those of the paper's KV memory (Section 2.2, "Taliesin: KV
 * memory"): after the runtime has computed the KV state of a block of prompt
 * text the state is written out; when the same block recurs it is loaded
 * instead of recomputed; what was stored is checked when it is loaded; and that
 * section's design rule puts correctness before reuse -- a request can always do
 * without stored state, but wrong stored state must never reach it -- so a record
 * that is absent, damaged or fails a check is not used at all: the block is
 * reported for recompute.  Restored state must be bit-identical to what was saved
 * (Section 3, Table 1), reuse is per whole block (Section 5, first item) and the design is
 * fail-closed (Section 5, second item).  The paper does not disclose its record
 * format (end of Section 1); the format below is this library's own.
 *
 * Data model
 *   paged cache  Opaque bytes.  The slab of (layer l, kv, physical page g)
 *                starts at data + l*layer_stride + kv*kv_stride + g*page_stride
 *                and holds page_tokens rows of row = kv_heads*head_dim*elem
 *                bytes, token-major ([t][h][d]); kv 0 is K, 1 is V.  One page id
 *                addresses all layers and both K and V.  With GK_FLAG_HEAD_MAJOR
 *                the slab is head-major instead ([h][t][d]: kv_heads runs of
 *                page_tokens*head_dim*elem bytes).
 *   scales       fp8 caches only: one fp32 per (l, kv < scale_kv, page, head) at
 *                scales + l*s_layer_stride + kv*s_kv_stride + g*s_page_stride + 4*h.
 *   blob         Page records 0..P-1 (P = ceil(n_tokens/page_tokens)) back to
 *                back, no header, no padding.  Record p = scale section (for l,
 *                for kv < scale_kv, for h: 4 bytes; absent for bf16), then for
 *                each layer the K prefix and the V prefix of the page, each
 *                t_p*row bytes, where t_p = page_tokens except for a shorter
 *                last page.  blob_bytes = P*S + n_tokens*2*layers*row.  A prefix
 *                of a head-major slab is, head by head, the first t_p tokens of
 *                that head (t_p*head_dim*elem bytes each): a full page is the
 *                slab as it lies in either layout, and the sizes do not change.
 *   checksums    uint64 per page: CRC-64/XZ of the bytes of its record.
 *
 * Conventions
 *   Every pointer called "device" must be device memory of the context's GPU;
 *   "host" means ordinary host memory unless "pinned" is stated.  The caller owns
 *   every buffer it passes.  A context owns only its internal workspace.
 *   Functions return GK_OK or a negative GK_ERR_* value; they never abort.  A
 *   checksum mismatch is NOT an error: the call returns GK_OK and the job's mask
 *   entry reports it.  Kernels are enqueued on the given stream; outputs are
 *   valid once that stream has been synchronised.  A context's workspace is
 *   shared by its calls: calls on one context must be issued in stream order on
 *   one stream at a time (use one context per concurrent stream).  gk_pack,
 *   gk_pack_batch, gk_restore, gk_verify and gk_commit calls of at most 64 jobs
 *   and 2,048 pages make no host-device copy and no synchronisation once the
 *   workspace has its size, and may be captured in a CUDA graph and replayed;
 *   the other entry points and larger calls may not.
 *   Requirements: row % 16 == 0, scale section bytes % 16 == 0, all base
 *   pointers and strides of data 16-byte aligned (scale pointers 4-byte), blob
 *   pointers 16-byte aligned, checksum pointers 8-byte aligned; otherwise
 *   GK_ERR_UNSUPPORTED.
 */
#ifndef GK_H
#define GK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GK_OK 0
#define GK_ERR_ARG (-1)         /* null pointer, zero tokens, bad geometry */
#define GK_ERR_UNSUPPORTED (-2) /* unknown dtype, alignment rules above not met */
#define GK_ERR_NOT_PINNED (-3)  /* host tier: blob or checksums not in pinned host memory */
#define GK_ERR_CUDA (-4)        /* a CUDA call failed; see gk_last_error */
#define GK_ERR_NOMEM (-5)       /* workspace allocation failed */
#define GK_ERR_DEVICE_WAIT (-6) /* reported by gk_get_stats: a bounded device wait ran out */
#define GK_ERR_TOO_LARGE (-7)   /* gk_page_checksums_noalloc: request exceeds its fixed scratch */

#define GK_BF16 0u
#define GK_FP8_E4M3 1u

/* Per-job result codes (mask entries).  Codes 1 to 3 mean that not one byte of
 * that job was written to the destination; the commit decision of a job is taken
 * once, for the whole job, so a job is never reported OK and written in part. */
#define GK_JOB_OK 0u          /* every page verified; block committed */
#define GK_JOB_CHECKSUM 1u    /* a page record failed its checksum */
#define GK_JOB_PAGE_TABLE 2u  /* page id out of [0,num_pages), or a destination page
                                 claimed more than once within the call */
#define GK_JOB_MISSING 3u     /* blob or checksums pointer is null */
#define GK_JOB_TIMEOUT 4u     /* a bounded wait inside a kernel ran out before this job was known
                                 to have verified (or the context still carries an earlier such
                                 failure, see gk_ctx_clear_error): the job is NOT restored.  Its
                                 destination pages are untouched, except in the one case described
                                 at gk_stats.device_wait_expired */

/* Test hook for sabotage tests (Section 3, sabotage-testing paragraph): switches the
 * checksum defence off so that a test can show the attack succeeds without it.
 * Page-table validation stays on. */
#define GK_FLAG_SKIP_VERIFY 1u

/* Slabs are head-major ([h][t][d]) instead of token-major.  Needs head_dim*elem to
 * be a multiple of 16 bytes (else GK_ERR_UNSUPPORTED).  A layout choice of this
 * library (the paper leaves the cache layout to the runtime it wraps). */
#define GK_FLAG_HEAD_MAJOR 2u

/* Single-pass restore.  NOT fail-closed: unverified bytes are written (into the
 * failing block's own pages); a departure from the block-level rule, off by default.
 * Section 2.2 has the runtime recompute every block whose
 * record fails a check, which rewrites that block's pages; a caller that does so
 * may set this flag: gk_restore* then checks and scatters each record in ONE pass
 * over the blob (2 bytes of memory traffic per blob byte instead of 3).  A block
 * whose only fault is a checksum mismatch is reported exactly as without the flag
 * (GK_JOB_CHECKSUM, same first bad page), but its OWN destination pages have
 * received the unverified record bytes and must not be used.  Blocks with
 * GK_JOB_PAGE_TABLE or GK_JOB_MISSING still write nothing, and no byte outside a
 * reported block's own pages (valid token range) changes.  Off by default: without
 * it nothing of a failing block is written.  gk_verify and gk_commit ignore it. */
#define GK_FLAG_SINGLE_PASS 4u

typedef struct gk_ctx gk_ctx;

typedef struct {
    uint32_t layers;
    uint32_t kv_heads;
    uint32_t head_dim;
    uint32_t page_tokens;
    uint32_t dtype;    /* GK_BF16 or GK_FP8_E4M3 */
    uint32_t scale_kv; /* fp8: 2 = a K scale and a V scale per (layer, head, page), 1 = one
                          shared scale; bf16: 0 */
    uint32_t flags;    /* 0 or an OR of GK_FLAG_SKIP_VERIFY, GK_FLAG_HEAD_MAJOR, GK_FLAG_SINGLE_PASS */
    uint32_t reserved; /* must be 0 */
} gk_geom;

typedef struct {
    void *data;         /* device */
    uint64_t num_pages; /* physical pages addressable through a page table */
    uint64_t layer_stride, kv_stride, page_stride; /* bytes */
    void *scales;       /* device; NULL when scale_kv == 0 */
    uint64_t s_layer_stride, s_kv_stride, s_page_stride; /* bytes */
} gk_cache;

/* One block.  For gk_pack*, blob and checksums are outputs; for gk_restore* they
 * are inputs.  page_table always points to DEVICE memory holding
 * ceil(n_tokens/page_tokens) int32 physical page ids. */
typedef struct {
    void *blob;                /* device (pinned host for gk_restore_host); NULL = missing */
    uint64_t *checksums;       /* device (pinned host for gk_restore_host); NULL = missing */
    const int32_t *page_table; /* device */
    uint32_t n_tokens;         /* > 0 */
    uint32_t request_id;       /* carried for the caller; not interpreted */
} gk_job;

typedef struct {
    uint64_t calls_pack, calls_restore, calls_restore_host;
    uint64_t jobs, pages, bytes_blob; /* submitted so far */
    uint64_t kernels_launched;        /* kernels enqueued by this context so far */
    uint32_t device_wait_expired;     /* non-zero once a bounded wait inside a kernel has run out.
                                         In the call that hit it, every job is either committed whole
                                         and reported GK_JOB_OK (it had verified before) or reported
                                         GK_JOB_TIMEOUT with nothing of it written.  The one exception:
                                         a wait on the kernel's own copy pipeline (a bulk copy that
                                         never completes, i.e. a hardware fault) leaves the jobs that
                                         had tiles in flight in that CTA partly written; they are
                                         reported GK_JOB_TIMEOUT, never GK_JOB_OK.  Every later call of
                                         the context reports GK_JOB_TIMEOUT for all jobs and writes
                                         nothing until gk_ctx_clear_error */
    uint32_t allocations;             /* device or pinned-host (re)allocations made so far by calls on this
                                         context (each one synchronises the device): stays constant once
                                         gk_ctx_reserve has sized everything */
    uint64_t calls_restore_stream;    /* its windows are counted in calls_restore_host as well */
    uint64_t quartet_launches;        /* packing and fused-restore launches that reduced one page record per
                                         warp, four pages to a work item (small records in large calls; tuning
                                         key "quad") */
} gk_stats;

/* Sizes of a block of n_tokens (Section 2.2: one record per block).  Either output may be NULL. */
int gk_blob_size(const gk_geom *geom, uint32_t n_tokens, uint64_t *blob_bytes, uint32_t *n_pages);

/* Creates a context for one geometry on one device.  Allocates constant tables
 * and a small workspace with cudaMalloc / cudaMallocHost; the workspace grows
 * (with a device synchronisation) when a later call needs more. */
int gk_ctx_create(gk_ctx **out, const gk_geom *geom, int device);
int gk_ctx_destroy(gk_ctx *ctx);
/* Text of the last error of this context (never NULL; empty if none). */
const char *gk_last_error(const gk_ctx *ctx);

/* Sizes everything a context allocates lazily, so that no later call within the
 * stated bounds allocates, frees or synchronises the device (a serving engine
 * calls this once at start-up; Section 2.2 has a request complete normally
 * whatever happens to stored state, which a mid-request device synchronisation
 * would not honour).  Bounds, per call: max_jobs jobs, max_pages page records in
 * total, a destination (or source) cache of num_pages pages and, for the host
 * tier, max_host_batch_bytes of blob bytes per staging slot (two slots are kept;
 * 0 = the host tier is not used; a host-tier call stages min(the call's blobs,
 * 256 MiB) per slot, or its largest single blob if that is larger).  Covers
 * gk_pack*, gk_restore*, gk_verify, gk_commit, gk_page_checksums and the
 * layer-wise and streaming calls; gk_fingerprints and gk_blob_digests size their
 * own scratch on first use.  Synchronises the device.  gk_get_stats().allocations
 * tells whether a later call had to grow something after all. */
int gk_ctx_reserve(gk_ctx *ctx, uint32_t max_jobs, uint64_t max_pages, uint64_t num_pages,
                   uint64_t max_host_batch_bytes);

/* Clears the context's record of a device wait that ran out (Section 5, second
 * item, and Section 2.2: a failed load is a miss, the block is recomputed and the
 * request completes; the store stays usable).  A wait can run out without any
 * fault, e.g. on a GPU that is time-sliced with another process.  Enqueued on
 * `stream`: calls issued after it on that stream commit again.  The caller should
 * first have treated every job reported GK_JOB_TIMEOUT as not restored. */
int gk_ctx_clear_error(gk_ctx *ctx, void *stream);

/* Save (Section 2.2: the block's state is written out once it has been computed;
 * here: gathered into one contiguous record with checksums).  jobs is a HOST array of n_jobs entries;
 * each job's blob (gk_blob_size bytes) and checksums (n_pages entries) are
 * device outputs.  Duplicate page ids are legal when packing.  A job whose table
 * holds an id outside [0, src->num_pages) writes neither blob nor checksums and
 * gets status GK_JOB_PAGE_TABLE; status_dev (device, n_jobs bytes, may be NULL)
 * receives 0 or that code.  n_jobs == 0 is a no-op. */
int gk_pack_batch(gk_ctx *ctx, const gk_cache *src, const gk_job *jobs, uint32_t n_jobs,
                  uint8_t *status_dev, void *stream);

/* One block; same as gk_pack_batch with a single job. */
int gk_pack(gk_ctx *ctx, const gk_cache *src, const int32_t *page_table_dev, uint32_t n_tokens,
            void *blob_dev, uint64_t *checksums_dev, uint8_t *status_dev, void *stream);

/* Save to the host tier (Section 2.2: stored state goes to storage; Section 4.3,
 * footprint and long-window paragraphs: the store is bounded by storage, not by
 * GPU memory).  As gk_pack_batch, but each job's blob and checksums are outputs
 * in PINNED host memory.  Batches of blocks are packed into the internal device
 * staging ring on `stream` while the previous batch is copied to the host on an
 * internal copy stream.  The call returns after enqueuing; `stream` is made to
 * wait for the last copy, so the host buffers are valid once `stream` has been
 * synchronised.  For a job with status GK_JOB_PAGE_TABLE the host blob and
 * checksums are unspecified and must not be used. */
int gk_pack_host(gk_ctx *ctx, const gk_cache *src, const gk_job *jobs, uint32_t n_jobs,
                 uint8_t *status_dev, void *stream);

/* Page checksums of an existing device blob (the check-on-load of Section 2.2
 * rests on them): checksums_dev[p] = CRC-64/XZ of record p. */
int gk_page_checksums(gk_ctx *ctx, const void *blob_dev, uint32_t n_tokens,
                      uint64_t *checksums_dev, void *stream);

/* Load (Section 2.2, and the fail-closed item of Section 5).  jobs is a HOST array;
 * blob, checksums and page_table of each job are device pointers.  Phase 1
 * validates every page table and verifies every page record of every job and
 * writes nothing to dst; phase 2 scatters the jobs whose code is GK_JOB_OK into
 * dst through their page tables (valid token prefix of each page only; fp8 scale
 * sections to dst->scales).  mask_dev (device, n_jobs bytes) receives the code of
 * each job, first_bad_page_dev (device, n_jobs int32) the lowest failing logical
 * page index for codes 1 and 2, else -1.  Destination bytes outside the committed
 * jobs' valid ranges are never written. */
int gk_restore(gk_ctx *ctx, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst,
               uint8_t *mask_dev, int32_t *first_bad_page_dev, void *stream);

/* The two halves of gk_restore as separate calls, for callers that must put a
 * step of their own between "checked" and "written" -- above all tensor-parallel
 * serving (Section 3 and Section 4.4 report tensor-parallel runs), where every
 * rank holds its own shard of a block and a block may be committed only if it
 * verified on ALL ranks: gk_verify on each rank, a max-reduction of the masks
 * across ranks, gk_commit with the reduced mask.
 *
 * gk_verify validates the page tables against dst (which it does not write) and
 * verifies every page record; mask_dev / first_bad_page_dev receive what gk_restore
 * would report, and nothing is committed.  gk_commit validates the tables again
 * and scatters exactly the jobs whose entry in mask_dev (device, n_jobs bytes,
 * input) is GK_JOB_OK and whose own table check passes; it verifies no checksum,
 * so the mask must come from a gk_verify of the same jobs. */
int gk_verify(gk_ctx *ctx, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst, uint8_t *mask_dev,
              int32_t *first_bad_page_dev, void *stream);
int gk_commit(gk_ctx *ctx, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst,
              const uint8_t *mask_dev, void *stream);

/* Load from the host tier (Section 4.3, long-window paragraph: saved blocks are
 * streamed in from storage and dropped after use).  As gk_restore, but each job's blob and checksums lie
 * in PINNED host memory.  Blobs are copied in batches into an internal device
 * staging ring on an internal copy stream while the previous batch is verified
 * and committed on `stream`; the checksum is taken over the bytes as they arrived
 * in device memory.  All page tables are validated on `stream` before anything is
 * verified or committed (the copies, on their own stream, may start earlier).  The
 * call returns after the last stage has been enqueued; results are valid after
 * `stream` has been synchronised.  The host buffers must stay valid until then.
 * The first copy starts only when the work already enqueued on `stream` has
 * finished, so the host buffers may be filled by earlier work on that stream. */
int gk_restore_host(gk_ctx *ctx, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst,
                    uint8_t *mask_dev, int32_t *first_bad_page_dev, void *stream);

/* Streaming load of a corpus that is larger than the cache (Section 4.3,
 * long-window paragraph: blocks are streamed in, used and dropped, so that GPU
 * memory stays flat while the corpus grows).  `ring` is a small cache whose pages
 * are handed out by this call; the jobs' own page_table fields are ignored.  Jobs
 * are taken in order and grouped into windows: a window is the longest run of
 * consecutive jobs whose pages fit `ring` together, and inside a window the jobs
 * get consecutive page ids from 0 (every job takes ceil(n_tokens/page_tokens)
 * pages, whatever its result).  Each window is loaded as by gk_restore_host
 * (blobs and checksums in PINNED host memory; verify, then commit, fail-closed per
 * job); then `consume` (may be NULL) is called ON THE HOST with the window's
 * blocks, and the next window reuses the pages.  Everything is ordered on
 * `stream`: the callback must only enqueue its work on `stream` (it may also
 * synchronise it); it must not call into this context.  While the consumer's
 * work runs, the copies of the next window are already in flight.
 * `blocks[i].page_table` is device memory owned by the context, valid until the
 * next call on the context; mask_dev / first_bad_page_dev (device, n_jobs
 * entries) cover the whole call and are indexed by blocks[i].job.
 * Returns GK_ERR_TOO_LARGE, having done nothing, if one job alone has more pages
 * than `ring`.  Device memory held: the ring, two staging slots (each the size of
 * the largest blob, or up to 256 MiB of smaller ones) and a workspace of a few
 * bytes per page of a window. */
typedef struct {
    uint32_t job;              /* index into the call's job array */
    uint32_t n_tokens;
    const int32_t *page_table; /* device: ids of the ring pages that hold the block */
} gk_window_block;
typedef void (*gk_window_fn)(void *user, const gk_window_block *blocks, uint32_t n_blocks,
                             const uint8_t *mask_dev, void *stream);
int gk_restore_stream(gk_ctx *ctx, const gk_job *jobs, uint32_t n_jobs, const gk_cache *ring,
                      uint8_t *mask_dev, int32_t *first_bad_page_dev, gk_window_fn consume, void *user,
                      void *stream);

/* Layer-wise save and load.  Fail-closed per (block, group of layers), not per
 * block: a departure from the block-level rule that the caller opts into by using
 * these calls; never the default format.  A consumer that walks the layers in order (a
 * forward pass) can start on the first layers of a block while the later ones
 * are still arriving from the host tier, if the block's record is cut by layer
 * groups (Section 4.3 streams saved state in from storage; the paper gives no
 * format).  Here the context's geometry describes ONE GROUP (geom.layers = layers
 * per group) and the cache holds n_groups * geom.layers layers.  The layer-wise
 * blob of a block is the concatenation, for group k = 0 .. n_groups-1, of the
 * ordinary blob (as gk_pack_batch makes it) of the cache restricted to the layers
 * [k*geom.layers, (k+1)*geom.layers); its checksums are those blobs' checksums,
 * group after group.  So jobs[j].blob holds n_groups * gk_blob_size() bytes and
 * jobs[j].checksums n_groups * n_pages entries.
 *
 * gk_pack_layerwise / gk_pack_layerwise_host: one gk_pack_batch / gk_pack_host
 * per group (status_dev as there).
 *
 * gk_restore_layerwise / gk_restore_layerwise_host: group after group, each as
 * one gk_restore / gk_restore_host of all jobs over the restricted cache, so
 * fail-closed holds per (job, group): of a block that fails in one group, the
 * groups that verified HAVE been written to the block's own pages and the failing
 * ones have not; the block as a whole is usable only if mask_dev[j] == GK_JOB_OK.
 * mask_dev[j] (device, n_jobs bytes) is the largest code over the groups,
 * first_bad_page_dev[j] the page reported by the lowest failing group (or -1);
 * group_mask_dev (device, n_groups * n_jobs bytes, group-major; may be NULL)
 * receives every group's codes.  After the work of group k has been enqueued,
 * on_group (may be NULL) is called ON THE HOST; it must only enqueue work on
 * `stream` (e.g. layer k's attention); group_mask points at group k's codes (NULL
 * if group_mask_dev is NULL).  In the host tier the copies of group k+1 run while
 * group k is verified, committed and consumed.  On the device tier the groups
 * (which touch different layers of the cache and different parts of the blobs)
 * go in turn to this context and to a second, internal one on two internal
 * streams, so that the first launches of a group overlap the last ones of the
 * group before; `stream` waits for each group in order before on_group sees it,
 * and for all of them before the call's work on `stream` is complete.  The
 * internal context is created at the first such call (or by gk_ctx_reserve);
 * its counters and its error word are part of this context's (gk_get_stats,
 * gk_ctx_clear_error). */
typedef void (*gk_group_fn)(void *user, uint32_t group, uint32_t first_layer, uint32_t n_layers,
                            const uint8_t *group_mask, void *stream);
int gk_pack_layerwise(gk_ctx *ctx, uint32_t n_groups, const gk_cache *src, const gk_job *jobs, uint32_t n_jobs,
                      uint8_t *status_dev, void *stream);
int gk_pack_layerwise_host(gk_ctx *ctx, uint32_t n_groups, const gk_cache *src, const gk_job *jobs,
                           uint32_t n_jobs, uint8_t *status_dev, void *stream);
int gk_restore_layerwise(gk_ctx *ctx, uint32_t n_groups, const gk_job *jobs, uint32_t n_jobs,
                         const gk_cache *dst, uint8_t *mask_dev, int32_t *first_bad_page_dev,
                         uint8_t *group_mask_dev, gk_group_fn on_group, void *user, void *stream);
int gk_restore_layerwise_host(gk_ctx *ctx, uint32_t n_groups, const gk_job *jobs, uint32_t n_jobs,
                              const gk_cache *dst, uint8_t *mask_dev, int32_t *first_bad_page_dev,
                              uint8_t *group_mask_dev, gk_group_fn on_group, void *user, void *stream);

/* Block fingerprints (Section 2.2: the lookup key of a block's state is derived
 * from the block's input, byte for byte, and from the identities of model and
 * tenant; Section 2.1: records of one model or tenant stay out of another's reach;
 * Section 2.2 and Section 5: a block is reused only at identical token positions).
 * The paper gives no format; this
 * library's keys are, with SHA-256 (FIPS 180-4), || for concatenation and
 * little-endian integers,
 *     inner_i = SHA-256( bytes_i || model[32] || tenant[32] || u64(len_i) || "GKF1" )
 *     key_i   = SHA-256( parent_key || inner_i || "GKF2" )
 * where bytes_i = data_dev[offsets_dev[i] .. offsets_dev[i+1]) (device; any
 * alignment, 16-byte aligned starts are fastest) and parent_key is key_{parent[i]},
 * or 32 zero bytes if parent[i] == -1: the key of a block depends on every block
 * before it in its prompt.  parent is a HOST array of n entries with
 * -1 <= parent[i] < i (else GK_ERR_ARG), or NULL for no chains; model and tenant
 * are HOST arrays of 32 bytes.  keys_dev: device, n*32 bytes, 16-byte aligned.
 * One thread hashes one message, so a call takes as long as its longest message
 * (about 40 ns per 64 bytes) however many messages it has. */
int gk_fingerprints(gk_ctx *ctx, const void *data_dev, const uint64_t *offsets_dev, const int32_t *parent,
                    uint32_t n, const uint8_t *model, const uint8_t *tenant, uint8_t *keys_dev, void *stream);

/* Confirmation hash of stored blocks (Section 3, sabotage-testing paragraph, lists
 * a confirmation hash among the safety mechanisms; Section 7 names hashes, besides
 * comparing bytes, as the judge of loaded state).  A three-level SHA-256 tree
 * over each blob, bound to the key the block is filed under:
 *     leaf   = SHA-256( chunk || "GKL0" )      chunk = 4096 record bytes, the last may be shorter
 *     page_p = SHA-256( leaf_0 || ... || leaf_{m-1} || u64(record bytes) || "GKP0" )
 *     digest = SHA-256( page_0 || ... || page_{P-1} || key[32] || u32(n_tokens) || u32(P) || "GKB0" )
 * jobs[j].blob: device, not NULL (else GK_ERR_ARG); checksums and page_table are
 * ignored.  keys_dev: device, n_jobs*32 bytes.  digests_dev: device, n_jobs*32
 * bytes, 16-byte aligned.  page_digests_dev: NULL, or device, 32 bytes per page of
 * the call in job order, 16-byte aligned (tells which page of a blob changed).
 * This is integer arithmetic, about 22 instructions per byte: an order of
 * magnitude slower than the CRC path, meant as a second tier. */
int gk_blob_digests(gk_ctx *ctx, const gk_job *jobs, uint32_t n_jobs, const uint8_t *keys_dev,
                    uint8_t *digests_dev, uint8_t *page_digests_dev, void *stream);

/* Bounds-checked build.  Section 3's sabotage paragraph reports that an address
 * sanitizer found the one out-of-bounds read of the paper's own code; a GPU
 * library cannot lean on such a tool everywhere, so this one can be compiled
 * with -DGK_DEBUG (libgk_debug.so): every access of a streaming kernel to caller
 * memory -- bulk copies from and to caches and blobs, scale values, checksum
 * words -- is then compared with the extent of the object it belongs to (cache
 * extents from the strides and num_pages, blob and checksum extents from
 * n_tokens).  An access that falls outside is skipped, never made, and the first
 * one is recorded; nothing traps and the context stays usable.
 * gk_debug_status copies the record out (blocking): out[0] = 0 if every access so
 * far was inside, else role << 8 | kind (kind 1 cache, 2 blob, 3 scales, 4
 * checksums, 5 staging tile; role 0 loader, 1 commit loader, 2 finisher, 3
 * storer), out[1..2] = offset of the refused access from its object's base,
 * out[3] = its size.  In the ordinary build it returns GK_ERR_UNSUPPORTED.
 * gk_debug_range_ok is the predicate itself, for host tests: 1 if
 * [addr, addr+bytes) lies inside [base, base+extent), else 0. */
int gk_debug_status(gk_ctx *ctx, uint32_t out[4]);
int gk_debug_range_ok(uint64_t addr, uint64_t bytes, uint64_t base, uint64_t extent);

/* Counters of this context.  Reads the device error word with a blocking copy. */
int gk_get_stats(gk_ctx *ctx, gk_stats *out);

/* Tuning knobs, for tests and measurements; defaults are chosen from the
 * geometry.  Keys: "seg_granules" (length of a checksum segment in units of
 * 32 KiB; 0 = one segment per page), "commit_seg_tiles" (length of a commit work
 * item in 16 KiB tiles), "grid_cap" (upper bound on CTAs per kernel; 0 = fill
 * the GPU), "profile" (1 = time every streaming kernel, see gk_get_kernel_times),
 * "fused" (1, the default: gk_restore verifies and commits in one launch; 0: a
 * verify launch, a checksum-compare launch and a commit launch), "wait_limit_ms"
 * (time limit of every wait inside a kernel, default 2000), "commit_reverse" (1,
 * the default: the commit side reads a job's records from the last to the first,
 * so that what was verified last is still in L2), "l2_hints" (bit 0: verify loads
 * ask L2 to keep the lines, bit 1: commit loads ask it to drop them, bit 2: commit
 * stores ask it to drop the written lines first; default 0),
 * "test_drop_verify" (tests only: with value k > 0 the fused restore kernel
 * verifies nothing of the jobs k-1, k, ..., so that the commit waits of exactly
 * those jobs run into their limit and the time-out handling can be checked
 * without hanging or faulting the GPU), "quad" (page quartets: 0, the default:
 * packing and verifying launches whose page records are at most 96 KiB and that
 * have at least 3.5 pages per resident CTA (verifying launches also with records
 * of up to 128 KiB from 12 pages per resident CTA on) reduce one record per warp
 * instead of one per CTA -- a quarter of the per-thread checksum epilogues per
 * byte; 1 = never;
 * 2 = in every such launch, whatever its size), and in the bounds-checked build only
 * "debug_extent_cut" (tests: cache extents are taken to be this many bytes smaller
 * than they are, so that a perfectly valid access to the last page is refused and
 * the reporting can be checked without any access outside an object). */
int gk_ctx_set_tuning(gk_ctx *ctx, const char *key, uint32_t value);

/* Page checksums of a device blob for callers that must not allocate.  (The
 * paper has no counterpart to this entry point; it exists for integration.)
 *
 * Everything else in this library works through a gk_ctx, and creating or
 * growing a context calls cudaMalloc and cudaMallocHost.  Some callers cannot
 * afford that: a serving engine that has already handed all free HBM to its own
 * KV-cache pool (a late cudaMalloc can fail there, and it synchronises the whole
 * device in the middle of serving), or a background scrubber that re-checks
 * stored blobs beside a running engine and has to stay out of its memory
 * budget.  For them this call computes checksums_dev[p] = CRC-64/XZ of page record
 * p of the blob -- the same values gk_page_checksums writes -- and allocates
 * nothing: no cudaMalloc, cudaFree, cudaMallocHost or any other allocating
 * routine, no context.  Its scratch is one fixed array of about 133 KiB inside the
 * library's device image, which every GPU that loads the library holds until the
 * process exits.
 *
 * Limits: at most GK_NOALLOC_MAX_PAGES pages per call (n_tokens <=
 * GK_NOALLOC_MAX_PAGES * page_tokens) and page_tokens <= GK_NOALLOC_MAX_PAGE_TOKENS;
 * beyond either the call does nothing and returns GK_ERR_TOO_LARGE.  geom->flags
 * is ignored.  Other returns: GK_ERR_ARG, GK_ERR_UNSUPPORTED (alignment rules as
 * above; device not sm_100), GK_ERR_CUDA.
 *
 * The first call on a device looks up the scratch array's device address and
 * sets the kernel's shared-memory attribute, once, with that device current;
 * make that first call before any stream capture is begun.  All calls on a
 * device share the one scratch array, which still holds the previous call's
 * contents when a call starts (the call resets what it needs): two calls that
 * overlap on the GPU -- different streams, or the same blob checked from two
 * threads -- race on it and may both return wrong checksums, so serialise them.
 * Work is enqueued on `stream`; checksums_dev is valid once it has been
 * synchronised.  Should a bounded wait inside the kernel run out (it cannot be
 * reported here: the call has returned), NO entry of checksums_dev is written:
 * a caller that must tell fills checksums_dev with a value of its own first
 * (a CRC-64 can take any value, so compare with the stored checksums: an
 * unwritten array fails that comparison like damage does). */
#define GK_NOALLOC_MAX_PAGES 8192u
#define GK_NOALLOC_MAX_PAGE_TOKENS 256u
int gk_page_checksums_noalloc(const gk_geom *geom, const void *blob_dev, uint32_t n_tokens,
                              uint64_t *checksums_dev, int device, void *stream);

/* Measurement aid (the paper has no counterpart): the rate at which this GPU
 * executes three-input logic operations, the instruction the checksum kernels
 * are made of -- lane operations per second over all SMs, from one kernel of
 * independent lop3 chains timed with CUDA events (best of three launches).  The
 * roofline of the checksum-bound kernels is this rate divided by their
 * instructions per byte.  Blocks until the measurement is done. */
int gk_measure_logic_rate(gk_ctx *ctx, double *lane_ops_per_second, void *stream);

/* Per-kernel device time of the streaming kernels, for measurements.  With the
 * tuning key "profile" set to 1 every launch of a streaming kernel is bracketed
 * by CUDA events on its stream.  This call waits for the recorded events, and
 * returns and then clears the totals since the previous call: index 0 = verify
 * alone, 1 = pack, 2 = commit alone, 3 = fused verify+commit (the restore kernel);
 * ms = summed duration, launches = count. */
int gk_get_kernel_times(gk_ctx *ctx, double ms[4], uint64_t launches[4]);

#ifdef __cplusplus
}
#endif
#endif
