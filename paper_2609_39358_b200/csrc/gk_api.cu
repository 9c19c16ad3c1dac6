// gk_api.cu -- host side of libgk: the C ABI declared in include/gk.h.
//
// Argument checking, per-call job tables, workspace management, kernel
// launches and the host-tier staging pipeline.  Every step of the data path
// runs in the kernels of gk_kernels.cuh; there is no CPU fallback.
#include "../../include/gk.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "gk_kernels.cuh"
#include "gk_sha256.cuh"

#ifndef GK_CRC_NT
#define GK_CRC_NT 128
#endif
// Ring shapes below are measured on B200.  Packing with 16 KiB x 5 stages (8 GiB of 2 MiB records:
// 2.62 ms against 2.65 ms with 3 stages; 4 GiB of 64 KiB records as page quartets: 1.30 against
// 1.43 ms -- the loader's look-ups at the start of every item need the deeper ring); the verifying
// kernels are bound by the integer pipe and do with 3.
#ifndef GK_CRC_STAGE
#define GK_CRC_STAGE 16384
#endif
#ifndef GK_CRC_STAGES
#define GK_CRC_STAGES 3
#endif
#ifndef GK_PACK_STAGE
#define GK_PACK_STAGE GK_CRC_STAGE
#endif
#ifndef GK_PACK_STAGES
#define GK_PACK_STAGES 5
#endif
#ifndef GK_VERIFY_MINB
#define GK_VERIFY_MINB 2
#endif
#ifndef GK_PACK_MINB
#define GK_PACK_MINB 2
#endif
#ifndef GK_COPY_STAGE
#define GK_COPY_STAGE 16384
#endif
#ifndef GK_COPY_STAGES
#define GK_COPY_STAGES 4
#endif
#ifndef GK_COPY_MINB
#define GK_COPY_MINB 3
#endif
// fused restore kernel: verify ring and commit ring of one CTA
#ifndef GK_FUSED_VSTAGES
#define GK_FUSED_VSTAGES 3
#endif
#ifndef GK_FUSED_CSTAGES
#define GK_FUSED_CSTAGES 4
#endif
#ifndef GK_FUSED_MINB
#define GK_FUSED_MINB 2
#endif

using namespace gk;

namespace {

using VerifyCfg = StreamCfg<kVerify, GK_CRC_NT, GK_CRC_STAGE, GK_CRC_STAGES>;
using PackCfg = StreamCfg<kPack, GK_CRC_NT, GK_PACK_STAGE, GK_PACK_STAGES>;
using CommitCfg = StreamCfg<kCommit, 0, GK_COPY_STAGE, GK_COPY_STAGES>;
using SingleCfg = StreamCfg<kSingle, GK_CRC_NT, GK_PACK_STAGE, GK_PACK_STAGES>;
using FusedCfg = RestoreCfg<GK_CRC_NT, GK_CRC_STAGE, GK_FUSED_VSTAGES, GK_COPY_STAGE, GK_FUSED_CSTAGES>;

constexpr int kSlots = 2;  // host-tier staging ring

uint64_t gf_xpow(uint64_t n)
{
    uint64_t r = 1, base = 2;
    while (n) {
        if (n & 1ull) r = gf_mul(r, base);
        base = gf_mul(base, base);
        n >>= 1;
    }
    return r;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// pages of a block; 64-bit so that n_tokens near 2^32 does not wrap
uint32_t pages_of(uint32_t n_tokens, uint32_t page_tokens)
{
    return (uint32_t)(((uint64_t)n_tokens + page_tokens - 1) / page_tokens);
}

}  // namespace

struct gk_ctx {
    gk_geom geom{};
    GeomDev gd{};
    int device = 0;
    int sm_count = 0;
    int occ_verify = 0, occ_pack = 0, occ_commit = 0, occ_fused = 0, occ_single = 0;
    uint32_t quad_mode = 0;      // page quartets: 0 = where they pay, 1 = never, 2 = wherever they are possible
    uint64_t *d_thread_const = nullptr;
    bool fused = true;           // restore runs verify and commit in one launch
    unsigned long long wait_limit_ns = kWaitLimitNs;
    uint32_t ctr_next[2] = {0, 0};  // what the device work counters will read when the next launch of
                                    // the current call starts (the first kernel of a call zeroes them)
    uint32_t test_drop_verify = 0;  // test hook: see gk_ctx_set_tuning
    bool commit_reverse = true;     // commit side walks a job's pages from the last to the first
    uint32_t l2_hints = 0;          // bit 0: verify loads evict_last, bit 1: commit loads evict_first
    uint32_t commit_items_per_cta = 3;       // small calls: commit work items wanted per resident CTA
    uint64_t debug_extent_cut = 0;  // bounds-checked build, tests: cache extents are reported this much smaller
    unsigned long long *trace = nullptr;  // builds with GK_TRACE: device buffer for time stamps (tuning keys)
    uint32_t seg_granules = 0;   // segment length in granules for the CRC modes
    uint32_t commit_seg_tiles = 0;
    uint32_t grid_cap = 0;       // 0: SMs * occupancy

    // constant tables + sticky error word
    uint64_t *d_init_term = nullptr;
    uint32_t *d_error = nullptr;

    // growing device workspace and pinned staging for job tables
    uint8_t *d_ws = nullptr;
    size_t ws_cap = 0;
    // pinned staging for job tables, two halves used in turn: the host fills one while the
    // upload of the previous call may still be reading the other
    uint8_t *h_stage = nullptr;      // 2 * h_stage_cap bytes
    size_t h_stage_cap = 0;          // bytes of one half
    cudaEvent_t ev_stage[2] = {nullptr, nullptr};  // upload from that half has been consumed
    uint32_t stage_next = 0;
    cudaEvent_t ev_entry = nullptr;  // host tier: where the caller's stream stood when the call came in

    // host tier
    cudaStream_t copy_stream = nullptr;
    uint8_t *d_slot[kSlots] = {nullptr, nullptr};
    size_t slot_cap = 0;
    cudaEvent_t ev_slot_free[kSlots] = {nullptr, nullptr};
    cudaEvent_t ev_copied[kSlots] = {nullptr, nullptr};
    bool slot_used[kSlots] = {false, false};
    uint32_t slot_next = 0;  // the slot the next batch goes to (carried across calls)
    bool pdl_next = false;   // the kernel just enqueued lets the next one start early (small calls)

    // layer-wise restore: the codes and pages of the group in flight
    uint8_t *d_group_tmp = nullptr;
    size_t group_tmp_cap = 0;
    // layer-wise calls on the device tier: the groups go in turn to this context and to a twin of it, each on a
    // stream of its own, so that the first launches of a group overlap the last ones of the group before
    gk_ctx *twin = nullptr;
    bool is_twin = false;
    cudaStream_t lw_stream[2] = {nullptr, nullptr};
    cudaEvent_t lw_entry = nullptr;
    cudaEvent_t lw_done[2] = {nullptr, nullptr};    // the group's work on its stream has been enqueued
    cudaEvent_t lw_merged[2] = {nullptr, nullptr};  // the group's result arrays have been read (caller's stream)

    // streaming restore: the ids 0..iota_cap-1, from which window page tables are cut
    int32_t *d_iota = nullptr;
    uint64_t iota_cap = 0;

    // optional per-kernel timing (tuning key "profile")
    bool profile = false;
    struct ProfSlot { cudaEvent_t a, b; int cls; };
    std::vector<ProfSlot> prof_pool;
    size_t prof_used = 0;
    double prof_ms[4] = {0, 0, 0, 0};
    uint64_t prof_launches[4] = {0, 0, 0, 0};

    // powers of x^(8 * segment bytes) for the segment lengths used recently (host arithmetic
    // of a few microseconds per length, which small calls would otherwise pay every time)
    struct SegPowers { uint64_t seg_bytes = 0; uint64_t x_seg = 0; std::vector<uint64_t> pw; uint64_t used = 0; };
    SegPowers seg_cache[4];
    uint64_t seg_cache_clock = 0;

    // host tier: buffers already seen to be pinned host memory (exact start addresses)
    std::vector<const void *> pinned_seen;

    gk_stats stats{};
    char err[512] = {0};
};

namespace {

int fail(gk_ctx *c, int code, const char *fmt, ...)
{
    if (c) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(c->err, sizeof(c->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

#define GK_CUDA(c, call)                                                                      \
    do {                                                                                      \
        cudaError_t e_ = (call);                                                              \
        if (e_ != cudaSuccess)                                                                \
            return fail((c), GK_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));    \
    } while (0)

int check_geom(const gk_geom *g, GeomDev *out)
{
    if (!g) return GK_ERR_ARG;
    if (g->layers == 0 || g->kv_heads == 0 || g->head_dim == 0 || g->page_tokens == 0) return GK_ERR_ARG;
    if (g->reserved != 0 || (g->flags & ~(GK_FLAG_SKIP_VERIFY | GK_FLAG_HEAD_MAJOR | GK_FLAG_SINGLE_PASS)))
        return GK_ERR_ARG;
    uint32_t elem;
    if (g->dtype == GK_BF16) {
        elem = 2;
        if (g->scale_kv != 0) return GK_ERR_ARG;
    } else if (g->dtype == GK_FP8_E4M3) {
        elem = 1;
        if (g->scale_kv != 1 && g->scale_kv != 2) return GK_ERR_ARG;
    } else {
        return GK_ERR_UNSUPPORTED;
    }
    const uint64_t row = (uint64_t)g->kv_heads * g->head_dim * elem;
    const uint64_t S = (uint64_t)g->layers * g->scale_kv * g->kv_heads * 4u;
    if (row % 16 != 0 || S % 16 != 0) return GK_ERR_UNSUPPORTED;
    const bool head_major = (g->flags & GK_FLAG_HEAD_MAJOR) != 0;
    if (head_major && ((uint64_t)g->head_dim * elem) % 16 != 0) return GK_ERR_UNSUPPORTED;
    if (row * g->page_tokens > (1ull << 30) || S > (1ull << 30)) return GK_ERR_UNSUPPORTED;
    if (out) {
        out->layers = g->layers;
        out->kv_heads = g->kv_heads;
        out->page_tokens = g->page_tokens;
        out->scale_kv = g->scale_kv;
        out->row = (uint32_t)row;
        out->S = (uint32_t)S;
        out->h4 = g->kv_heads * 4u;
        out->flags = g->flags;
        out->hrow = g->head_dim * elem;
        out->head_major = head_major ? 1u : 0u;
        out->tokB = 2ull * g->layers * row;
        out->R = S + (uint64_t)g->page_tokens * out->tokB;
    }
    return GK_OK;
}

int check_cache(gk_ctx *c, const gk_cache *k, CacheDev *out)
{
    if (!k || !k->data || k->num_pages == 0) return fail(c, GK_ERR_ARG, "cache: null data or zero pages");
    if (k->num_pages > 0x7fffffffull) return fail(c, GK_ERR_ARG, "cache: too many pages");
    if (((uintptr_t)k->data | k->layer_stride | k->kv_stride | k->page_stride) & 15u)
        return fail(c, GK_ERR_UNSUPPORTED, "cache: data pointer and strides must be multiples of 16 bytes");
    if (c->gd.scale_kv) {
        if (!k->scales) return fail(c, GK_ERR_ARG, "cache: fp8 geometry needs a scale tensor");
        if (((uintptr_t)k->scales | k->s_layer_stride | k->s_kv_stride | k->s_page_stride) & 3u)
            return fail(c, GK_ERR_UNSUPPORTED, "cache: scale pointer and strides must be multiples of 4 bytes");
    }
    out->data = (uint8_t *)k->data;
    out->num_pages = k->num_pages;
    out->layer_stride = k->layer_stride;
    out->kv_stride = k->kv_stride;
    out->page_stride = k->page_stride;
    out->scales = (uint8_t *)k->scales;
    out->s_layer_stride = k->s_layer_stride;
    out->s_kv_stride = k->s_kv_stride;
    out->s_page_stride = k->s_page_stride;
    // where the last byte that a page table of this geometry can address lies (the bounds-checked build
    // compares every access with these)
    const uint64_t slab = (uint64_t)c->gd.page_tokens * c->gd.row;
    out->data_extent = (uint64_t)(c->gd.layers - 1u) * k->layer_stride + k->kv_stride + (k->num_pages - 1u) * k->page_stride + slab;
    out->scales_extent = c->gd.scale_kv ? (uint64_t)(c->gd.layers - 1u) * k->s_layer_stride +
                                              (uint64_t)(c->gd.scale_kv - 1u) * k->s_kv_stride +
                                              (k->num_pages - 1u) * k->s_page_stride + 4ull * c->gd.kv_heads
                                        : 0u;
    out->data_extent -= c->debug_extent_cut < out->data_extent ? c->debug_extent_cut : out->data_extent;
    return GK_OK;
}

// Work items wanted per launch: two per resident CTA, so that small calls still fill the GPU
// (measured: verify of 64 and of 325 GQA pages is fastest with 1-2 and 2-4 items per CTA).
uint64_t items_wanted(const gk_ctx *c, int occ) { return 2ull * (uint64_t)c->sm_count * (uint64_t)occ; }

// Tiling of the CRC modes for a call of total_pages pages.  Large calls use one
// segment per page (the per-thread epilogue is paid once per page); small calls
// cut pages into segments of at least two granules so that every SM gets work.
//
// Page quartets (`quad_for`: the call packs, or verifies -- alone or in a fused restore): small records in a
// call with enough quartets for every resident CTA are reduced one per WARP instead of one per CTA, four pages
// to a work item (see Tiling).  Where they pay (B200, gqa7b geometry with 1, 2, 4 layers per record): 64 KiB
// records from about 1,000 pages on (8 GiB: save 0.82 -> 1.03 of the copy peak, restore 0.88 -> 1.03; 512
// pages: 35 us as single pages, 39 us as quartets); 128 KiB records only where the kernel verifies, and from
// about 4,000 pages on (8 GiB: restore 1.01 -> 1.03, save 1.02 either way); 256 KiB records nowhere.
enum QuadUse { kNoQuad = 0, kQuadPack = 1, kQuadRestore = 2 };

bool quad_wanted(const gk_ctx *c, QuadUse quad_for, uint64_t total_pages, int occ)
{
    if (quad_for == kNoQuad || c->quad_mode == 1u || c->seg_granules) return false;
    if (quad_for == kQuadPack && c->gd.S != 0u) return false;  // scale values are gathered by a whole warp per record
    if (c->quad_mode == 2u) return true;
    const uint64_t resident = (uint64_t)c->sm_count * (uint64_t)occ;
    if (c->gd.R <= (96u << 10)) return 2ull * total_pages >= 7ull * resident;
    return quad_for == kQuadRestore && c->gd.R <= (128u << 10) && total_pages >= 12ull * resident;
}

uint32_t crc_items(const Tiling &tl, uint64_t pages)
{
    return tl.quad ? (uint32_t)((pages + 3) / 4) : (uint32_t)pages * tl.nseg_max;
}

Tiling crc_tiling(const gk_ctx *c, uint32_t stage_bytes, uint64_t total_pages, int occ, bool overlap_jobs = false,
                  QuadUse quad_for = kNoQuad)
{
    Tiling t;
    if (quad_wanted(c, quad_for, total_pages, occ)) {
        t.quad = 1u;
        t.stage_bytes = stage_bytes / 4;   // one record's part of a stage
        t.gran_bytes = 32u * 256u;         // 8 shift-register steps of 8 words for each of 32 threads
        t.seg_tiles = (uint32_t)((c->gd.R + t.gran_bytes - 1) / t.gran_bytes) * (t.gran_bytes / t.stage_bytes);
        t.nseg_max = 1;
        return t;
    }
    t.stage_bytes = stage_bytes;
    t.gran_bytes = VerifyCfg::kGran;
    const uint32_t gran_full = (uint32_t)((c->gd.R + t.gran_bytes - 1) / t.gran_bytes);
    uint32_t sg = gran_full;
    if (c->seg_granules) {
        sg = c->seg_granules;
    } else if (total_pages > 0 && total_pages < items_wanted(c, occ)) {
        // Small call: cut pages into k segments each.  Estimated time = rounds * (segment time +
        // per-item overhead), rounds = ceil(items / resident CTAs); constants fitted to measurements
        // on B200 (a CTA sharing its SM streams about 15 GB/s through the CRC; ring refill, item
        // look-up and the per-segment epilogue cost about 20 us per item).
        const double grid = (double)c->sm_count * occ;
        const double page_us = (double)c->gd.R / 15e3;
        const double item_us = 20.0;
        double best = 1e30;
        uint32_t best_k = 1;
        uint32_t kmax = gran_full > 1 ? gran_full / 2 : 1;  // at least two granules per segment
        if (kmax > kPrepMaxSeg) kmax = kPrepMaxSeg;               // and the table must fit the preparation launch
        for (uint32_t k = 1; k <= kmax; ++k) {
            const uint32_t g = (gran_full + k - 1) / k;            // granules per segment
            const uint32_t nseg = (gran_full + g - 1) / g;
            const double rounds = std::ceil((double)total_pages * nseg / grid);
            const double cost = rounds * (page_us / nseg + item_us);
            if (cost < best * 0.999) {
                best = cost;
                best_k = k;
            }
        }
        if (overlap_jobs) {
            // fused restore of several jobs: finer items let the first jobs finish verifying early,
            // so that their commit overlaps the verification of the rest (8 jobs x 512 tokens:
            // 310 us with whole pages, 273 us with three segments per page)
            const uint64_t per_page = (items_wanted(c, occ) + total_pages - 1) / total_pages;
            if (per_page > best_k) best_k = (uint32_t)(per_page < kmax ? per_page : kmax);
        }
        sg = (gran_full + best_k - 1) / best_k;
    }
    if (sg > gran_full) sg = gran_full;
    if (sg < 1) sg = 1;
    t.seg_tiles = sg * (t.gran_bytes / stage_bytes);
    t.nseg_max = (gran_full + sg - 1) / sg;
    return t;
}

Tiling commit_tiling(const gk_ctx *c, uint32_t stage_bytes, uint64_t total_pages, int occ)
{
    Tiling t;
    t.stage_bytes = stage_bytes;
    t.gran_bytes = stage_bytes;
    const uint32_t tiles_full = (uint32_t)((c->gd.R + t.stage_bytes - 1) / t.stage_bytes);
    uint32_t st = (256u << 10) / stage_bytes;  // 256 KiB per commit item
    if (c->commit_seg_tiles) {
        st = c->commit_seg_tiles;
    } else if (total_pages > 0) {
        const uint64_t items = total_pages * ((tiles_full + st - 1) / st);
        const uint64_t want = (uint64_t)c->commit_items_per_cta * c->sm_count * occ;
        if (items < want) {
            const uint64_t per_page = (want + total_pages - 1) / total_pages;
            st = (uint32_t)((tiles_full + per_page - 1) / per_page);
        }
    }
    if (st > tiles_full) st = tiles_full;
    if (st < 1) st = 1;
    t.seg_tiles = st;
    t.nseg_max = (tiles_full + st - 1) / st;
    return t;
}

// Views into the workspace for one call.
struct WsLayout {
    size_t jobs, page_job, page_acc, bad_range, bad_dup, bad_crc, page_cnt, job_done, job_latch, claims, total;
};

WsLayout ws_layout(uint32_t n_jobs, uint64_t total_pages, uint32_t nseg_max, uint64_t num_pages)
{
    WsLayout l;
    size_t o = 0;
    l.jobs = o;      o = align_up(o + (size_t)n_jobs * sizeof(JobDev) + (size_t)nseg_max * 16, 256);  // + seg_pow
    l.page_job = o;  o = align_up(o + (size_t)total_pages * 4, 256);
    l.page_acc = o;  o = align_up(o + (size_t)total_pages * 8, 256);
    l.bad_range = o; o = align_up(o + (size_t)n_jobs * 4, 256);
    l.bad_dup = o;   o = align_up(o + (size_t)n_jobs * 4, 256);
    l.bad_crc = o;   o = align_up(o + (size_t)n_jobs * 4, 256);
    l.page_cnt = o;  o = align_up(o + (size_t)total_pages * 4, 256);
    l.job_done = o;  o = align_up(o + (size_t)n_jobs * 4, 256);
    l.job_latch = o; o = align_up(o + (size_t)n_jobs * 4, 256);
    l.claims = o;    o = align_up(o + (size_t)num_pages * 8, 256);
    l.total = o;
    return l;
}

int ensure_workspace(gk_ctx *c, size_t need)
{
    if (need <= c->ws_cap) return GK_OK;
    GK_CUDA(c, cudaDeviceSynchronize());  // earlier calls may still use the old block
    if (c->d_ws) cudaFree(c->d_ws);
    c->d_ws = nullptr;
    c->ws_cap = 0;
    const size_t cap = align_up(need + need / 2, 1 << 20);
    if (cudaMalloc(&c->d_ws, cap) != cudaSuccess) {
        cudaGetLastError();
        return fail(c, GK_ERR_NOMEM, "workspace of %zu bytes", cap);
    }
    c->ws_cap = cap;
    c->stats.allocations++;
    return GK_OK;
}

int ensure_host_stage(gk_ctx *c, size_t need)
{
    if (need <= c->h_stage_cap) return GK_OK;
    for (int i = 0; i < 2; ++i) GK_CUDA(c, cudaEventSynchronize(c->ev_stage[i]));
    if (c->h_stage) cudaFreeHost(c->h_stage);
    c->h_stage = nullptr;
    c->h_stage_cap = 0;
    const size_t cap = align_up(need * 2, 1 << 16);
    if (cudaMallocHost(&c->h_stage, 2 * cap) != cudaSuccess) {
        cudaGetLastError();
        return fail(c, GK_ERR_NOMEM, "pinned staging of %zu bytes", 2 * cap);
    }
    c->h_stage_cap = cap;
    c->stats.allocations++;
    return GK_OK;
}

// The half of the pinned staging area that the next upload may fill: waits only for the
// upload that used this half two calls ago.
int next_host_stage(gk_ctx *c, size_t need, uint8_t **out, cudaEvent_t *ev)
{
    int rc = ensure_host_stage(c, need);
    if (rc != GK_OK) return rc;
    const uint32_t h = c->stage_next;
    c->stage_next ^= 1u;
    GK_CUDA(c, cudaEventSynchronize(c->ev_stage[h]));
    *out = c->h_stage + (size_t)h * c->h_stage_cap;
    *ev = c->ev_stage[h];
    return GK_OK;
}

// x^(8*seg_bytes) and its powers 0..n-1 mod P, from the context's cache
const gk_ctx::SegPowers &seg_powers(gk_ctx *c, uint64_t seg_bytes, uint32_t n)
{
    gk_ctx::SegPowers *e = nullptr, *oldest = &c->seg_cache[0];
    for (auto &s : c->seg_cache) {
        if (s.seg_bytes == seg_bytes && s.x_seg != 0) e = &s;
        if (s.used < oldest->used) oldest = &s;
    }
    if (!e) {
        e = oldest;
        e->seg_bytes = seg_bytes;
        e->x_seg = gf_xpow(8ull * seg_bytes);
        e->pw.assign({1ull, 1ull << 32});
    }
    while (e->pw.size() < 2 * (size_t)n) {
        const uint64_t next = gf_mul(e->pw[e->pw.size() - 2], e->x_seg);
        e->pw.push_back(next);
        e->pw.push_back(gf_mul(next, 1ull << 32));
    }
    e->used = ++c->seg_cache_clock;
    return *e;
}

WorkDev make_work(gk_ctx *c, const WsLayout &l, uint32_t n_jobs, uint32_t total_pages, const Tiling &crc)
{
    WorkDev w{};
    w.jobs = (const JobDev *)(c->d_ws + l.jobs);
    w.n_jobs = n_jobs;
    w.page_begin = 0;
    w.total_pages = total_pages;
    w.page_job = (int32_t *)(c->d_ws + l.page_job);
    w.page_acc = (uint64_t *)(c->d_ws + l.page_acc);
    w.bad_range = (int32_t *)(c->d_ws + l.bad_range);
    w.bad_dup = (int32_t *)(c->d_ws + l.bad_dup);
    w.bad_crc = (int32_t *)(c->d_ws + l.bad_crc);
    w.page_cnt = (uint32_t *)(c->d_ws + l.page_cnt);
    w.job_done = (uint32_t *)(c->d_ws + l.job_done);
    w.job_latch = (uint32_t *)(c->d_ws + l.job_latch);
    w.claims = (unsigned long long *)(c->d_ws + l.claims);
    w.error = c->d_error;
    w.work_ctr = c->d_error + 16;
    w.init_term = c->d_init_term;
    w.thread_const = c->d_thread_const;
    w.seg_pow = (const uint64_t *)(c->d_ws + l.jobs + (size_t)n_jobs * sizeof(JobDev));
    w.wait_limit_ns = c->wait_limit_ns;
    return w;
}

// Job records of a call from the caller's gk_job array.  blob_override /
// sums_override (may be null) replace the callers' pointers, for the host tier.
int fill_job_table(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, JobDev *h, uint8_t *const *blob_override,
                   uint64_t *const *sums_override, bool need_tables, uint64_t *total_pages_out,
                   uint64_t *total_bytes_out)
{
    uint64_t pages = 0, bytes = 0;
    for (uint32_t j = 0; j < n_jobs; ++j) {
        const gk_job &jb = jobs[j];
        if (jb.n_tokens == 0) return fail(c, GK_ERR_ARG, "job %u: n_tokens == 0", j);
        if (need_tables && !jb.page_table) return fail(c, GK_ERR_ARG, "job %u: null page table", j);
        const uint32_t np = pages_of(jb.n_tokens, c->gd.page_tokens);
        h[j].blob = blob_override ? blob_override[j] : (uint8_t *)jb.blob;
        h[j].checksums = sums_override ? sums_override[j] : jb.checksums;
        h[j].page_table = jb.page_table;
        h[j].n_tokens = jb.n_tokens;
        h[j].n_pages = np;
        h[j].page_base = (uint32_t)pages;
        h[j].missing = (jb.blob == nullptr || jb.checksums == nullptr) ? 1u : 0u;
        if (!h[j].missing) {
            if (((uintptr_t)h[j].blob & 15u) || ((uintptr_t)h[j].checksums & 7u))
                return fail(c, GK_ERR_UNSUPPORTED, "job %u: blob must be 16-byte and checksums 8-byte aligned", j);
        }
        pages += np;
        bytes += (uint64_t)np * c->gd.S + (uint64_t)jb.n_tokens * c->gd.tokB;
        if (pages > 0x7fffffffull) return fail(c, GK_ERR_ARG, "too many pages in one call");
    }
    *total_pages_out = pages;
    if (total_bytes_out) *total_bytes_out = bytes;
    return GK_OK;
}

// powers of x^(8 * segment bytes), which place segment remainders inside their page: for every
// power k the pair (power, power * x^32), one factor for each 32-bit half of a remainder
void fill_seg_pow(gk_ctx *c, const Tiling &crc, uint64_t *pw)
{
    if (crc.nseg_max == 0) return;
    const gk_ctx::SegPowers &sp = seg_powers(c, (uint64_t)crc.seg_tiles * crc.stage_bytes, crc.nseg_max);
    std::memcpy(pw, sp.pw.data(), (size_t)crc.nseg_max * 16);
}

// Fills the pinned job table (and the segment powers behind it) and enqueues the upload.
int upload_jobs(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const WsLayout &l, const Tiling &crc,
                uint8_t *const *blob_override, uint64_t *const *sums_override, bool need_tables, cudaStream_t st,
                uint64_t *total_pages_out, uint64_t *total_bytes_out)
{
    const size_t table_bytes = (size_t)n_jobs * sizeof(JobDev) + (size_t)crc.nseg_max * 16;
    uint8_t *stage = nullptr;
    cudaEvent_t ev = nullptr;
    int rc = next_host_stage(c, table_bytes, &stage, &ev);
    if (rc != GK_OK) return rc;
    JobDev *h = (JobDev *)stage;
    if ((rc = fill_job_table(c, jobs, n_jobs, h, blob_override, sums_override, need_tables, total_pages_out,
                             total_bytes_out)) != GK_OK)
        return rc;
    fill_seg_pow(c, crc, reinterpret_cast<uint64_t *>(stage + (size_t)n_jobs * sizeof(JobDev)));
    GK_CUDA(c, cudaMemcpyAsync(c->d_ws + l.jobs, h, table_bytes, cudaMemcpyHostToDevice, st));
    GK_CUDA(c, cudaEventRecord(ev, st));
    return GK_OK;
}

// Small calls: job table and segment powers travel as kernel arguments of the one
// preparation launch (no staging copy, no separate validate / claim launches).
bool is_small_call(uint32_t n_jobs, uint64_t pages, const Tiling &crc)
{
    // one CTA walks all pages of the call three times: beyond two pages per thread the parallel
    // validation and claim kernels are faster, staging copy included
    return n_jobs <= kPrepMaxJobs && crc.nseg_max <= kPrepMaxSeg && pages <= 2048;
}

int launch_prep_small(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const Tiling &crc, const WorkDev &w,
                      uint64_t num_pages, bool need_tables, bool do_claims, cudaStream_t st, uint64_t *pages_out,
                      uint64_t *bytes_out, uint8_t *status_out = nullptr)
{
    PrepSmallParams pp{};
    int rc = fill_job_table(c, jobs, n_jobs, pp.jobs, nullptr, nullptr, need_tables, pages_out, bytes_out);
    if (rc != GK_OK) return rc;
    fill_seg_pow(c, crc, pp.seg_pow);
    pp.n_seg_pow = 2 * crc.nseg_max;
    pp.do_claims = do_claims ? 1u : 0u;
    pp.num_pages = num_pages;
    pp.status_out = status_out;
    c->ctr_next[0] = c->ctr_next[1] = 0;  // the kernel zeroes the device counters
    prep_small_kernel<<<1, 1024, 0, st>>>(pp, w);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched++;
    c->pdl_next = !c->profile;  // timing events between the two launches would break the pairing
    return GK_OK;
}

// Draws from a work counter in one launch.  A loader draws once per item it meets and stops at
// the first number that is past the end; taking the first item without drawing (the CTA's own
// number) saves one draw per CTA.  The host adds these up so that it can tell every later
// launch of the call what its counter starts from.
uint32_t draws_of(uint32_t n_items, uint32_t grid, bool static_first)
{
    return n_items + (static_first ? 0u : grid);
}

uint32_t stream_grid(const gk_ctx *c, int occ, uint32_t n_items)
{
    uint32_t g = (uint32_t)(c->sm_count * occ);
    if (c->grid_cap && g > c->grid_cap) g = c->grid_cap;
    if (g > n_items) g = n_items;
    return g ? g : 1u;
}

// Per-kernel timing (tuning key "profile"): takes a pair of events from the pool, records the
// first one, and hands the pair back; the caller records the second one behind its launch.
int prof_begin(gk_ctx *c, int cls, cudaStream_t st, gk_ctx::ProfSlot **slot)
{
    *slot = nullptr;
    if (!c->profile) return GK_OK;
    if (c->prof_used == c->prof_pool.size()) {
        gk_ctx::ProfSlot ns{};
        GK_CUDA(c, cudaEventCreate(&ns.a));
        GK_CUDA(c, cudaEventCreate(&ns.b));
        c->prof_pool.push_back(ns);
    }
    *slot = &c->prof_pool[c->prof_used++];
    (*slot)->cls = cls;
    GK_CUDA(c, cudaEventRecord((*slot)->a, st));
    return GK_OK;
}

// Launches a streaming kernel; right behind the small-call preparation kernel it is
// launched as a programmatic dependent, so that its CTAs are resident and their
// rings set up by the time the preparation kernel ends.
template <class Kernel>
cudaError_t launch_streaming(gk_ctx *c, Kernel kernel, uint32_t grid, int threads, size_t smem, cudaStream_t st,
                             const StreamParams &Q)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = c->pdl_next ? 1u : 0u;
    c->pdl_next = false;
    return cudaLaunchKernelEx(&cfg, kernel, Q);
}

template <class Cfg, int MODE, int NT, int SB, int ST, int MINB, bool QUAD = false>
int launch_stream(gk_ctx *c, int occ, const StreamParams &P, cudaStream_t st)
{
    const uint32_t items = MODE == kCommit ? P.n_items_c : P.n_items;
    if (items == 0) {
        c->pdl_next = false;
        return GK_OK;
    }
    const uint32_t grid = stream_grid(c, occ, items);
    gk_ctx::ProfSlot *slot = nullptr;
    int rc_prof = prof_begin(c, MODE, st, &slot);  // kSingle == 3: booked with the fused restore kernel
    if (rc_prof != GK_OK) return rc_prof;
    StreamParams Q = P;
    const int ci = MODE == kCommit ? 1 : 0;
    if (ci) Q.ctr_base_c = c->ctr_next[1];
    else Q.ctr_base_v = c->ctr_next[0];
    Q.trace = c->trace;
    c->ctr_next[ci] += draws_of(items, grid, true);
    GK_CUDA(c, launch_streaming(c, stream_kernel<MODE, NT, SB, ST, MINB, QUAD>, grid, Cfg::kThreads, Cfg::kSmemBytes, st, Q));
    if (slot) GK_CUDA(c, cudaEventRecord(slot->b, st));
    c->stats.kernels_launched++;
    if (QUAD) c->stats.quartet_launches++;
    return GK_OK;
}

int launch_verify(gk_ctx *c, const StreamParams &P, cudaStream_t st)
{
    if (P.tl.quad)
        return launch_stream<VerifyCfg, kVerify, GK_CRC_NT, GK_CRC_STAGE, GK_CRC_STAGES, GK_VERIFY_MINB, true>(
            c, c->occ_verify, P, st);
    return launch_stream<VerifyCfg, kVerify, GK_CRC_NT, GK_CRC_STAGE, GK_CRC_STAGES, GK_VERIFY_MINB>(c, c->occ_verify, P, st);
}
int launch_pack(gk_ctx *c, const StreamParams &P, cudaStream_t st)
{
    if (P.tl.quad)
        return launch_stream<PackCfg, kPack, GK_CRC_NT, GK_PACK_STAGE, GK_PACK_STAGES, GK_PACK_MINB, true>(c, c->occ_pack, P,
                                                                                                            st);
    return launch_stream<PackCfg, kPack, GK_CRC_NT, GK_PACK_STAGE, GK_PACK_STAGES, GK_PACK_MINB>(c, c->occ_pack, P, st);
}
// single-pass restore; per-kernel timing books it under "restore" (index 3)
int launch_single(gk_ctx *c, const StreamParams &P, cudaStream_t st)
{
    return launch_stream<SingleCfg, kSingle, GK_CRC_NT, GK_PACK_STAGE, GK_PACK_STAGES, GK_PACK_MINB>(c, c->occ_single, P, st);
}
int launch_commit(gk_ctx *c, const StreamParams &P, cudaStream_t st)
{
    return launch_stream<CommitCfg, kCommit, 0, GK_COPY_STAGE, GK_COPY_STAGES, GK_COPY_MINB>(c, c->occ_commit, P, st);
}

// verify + commit in one launch; per-kernel timing books it under "commit" (index 2)
int launch_fused(gk_ctx *c, const StreamParams &P, cudaStream_t st)
{
    const uint32_t items = P.n_items > P.n_items_c ? P.n_items : P.n_items_c;
    if (items == 0) {
        c->pdl_next = false;
        return GK_OK;
    }
    uint32_t grid = stream_grid(c, c->occ_fused, items);
    // Large records without scale sections in a large call: the kernel is bound by DRAM, the checksum needs
    // only half the integer lanes, and one CTA per SM is a little faster than two (8 GiB of 2 MiB records:
    // 3.80 against 3.83 ms; 3 MiB records 8.41 against 8.50 ms; 768 KiB records and fp8 records, whose scale
    // values the loader's and storer's lanes move one by one, are slower that way).
    // Not for a call of one or two blocks: a block is committed only after all of it has verified, so its two
    // phases follow one another, and the verifying phase alone wants both CTAs of an SM (one block of 24,018
    // tokens: 1.62 ms with two CTAs per SM, 1.77 ms with one).
    if (!c->grid_cap && c->gd.S == 0 && c->gd.R >= (1u << 20) && P.n_items >= 8u * (uint32_t)c->sm_count &&
        P.w.n_jobs >= 4u && grid > (uint32_t)c->sm_count) {
        grid = (uint32_t)c->sm_count;
        // not as a programmatic dependent: CTAs that arrive while the kernel before is still on some SMs
        // double up on the others and stay there (96 blocks of 3 MiB records: 8.62 instead of 8.41 ms)
        c->pdl_next = false;
    }
    gk_ctx::ProfSlot *slot = nullptr;
    int rc_prof = prof_begin(c, 3, st, &slot);
    if (rc_prof != GK_OK) return rc_prof;
    StreamParams Q = P;
    Q.ctr_base_v = c->ctr_next[0];
    Q.ctr_base_c = c->ctr_next[1];
    Q.trace = c->trace;
    // the verify side draws every item, the commit side takes the first one of each CTA without drawing
    c->ctr_next[0] += draws_of(P.n_items, grid, false);
    c->ctr_next[1] += draws_of(P.n_items_c, grid, true);
    if (P.tl.quad)
        GK_CUDA(c, launch_streaming(c, restore_kernel<GK_CRC_NT, GK_CRC_STAGE, GK_FUSED_VSTAGES, GK_COPY_STAGE,
                                                      GK_FUSED_CSTAGES, GK_FUSED_MINB, true>,
                                    grid, FusedCfg::kThreads, FusedCfg::kSmemBytes, st, Q));
    else
        GK_CUDA(c, launch_streaming(c, restore_kernel<GK_CRC_NT, GK_CRC_STAGE, GK_FUSED_VSTAGES, GK_COPY_STAGE,
                                                      GK_FUSED_CSTAGES, GK_FUSED_MINB>,
                                    grid, FusedCfg::kThreads, FusedCfg::kSmemBytes, st, Q));
    if (slot) GK_CUDA(c, cudaEventRecord(slot->b, st));
    c->stats.kernels_launched++;
    if (P.tl.quad) c->stats.quartet_launches++;
    return GK_OK;
}

int launch_validate(gk_ctx *c, const WorkDev &w, uint64_t num_pages, int clear_claims, cudaStream_t st,
                    uint8_t *status_out = nullptr)
{
    uint32_t grid = w.n_jobs;
    if (clear_claims) {
        uint32_t g2 = (uint32_t)((num_pages + 1023) / 1024);
        if (g2 > 2048) g2 = 2048;
        if (g2 > grid) grid = g2;
    }
    c->ctr_next[0] = c->ctr_next[1] = 0;  // the kernel zeroes the device counters
    validate_kernel<<<grid, 1024, 0, st>>>(w, num_pages, clear_claims, status_out);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched++;
    return GK_OK;
}

// Large calls of at most kPrepMaxJobs jobs: the job table rides in the validation kernel's arguments instead of
// a staging copy in front of it (one stream operation less per call: layer-wise calls make one call per group).
bool table_fits_args(uint32_t n_jobs, const Tiling &crc)
{
    return n_jobs <= kPrepMaxJobs && crc.nseg_max <= kPrepMaxSeg;
}

int launch_validate_args(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const Tiling &crc, const WorkDev &w,
                         uint64_t num_pages, int clear_claims, bool need_tables, cudaStream_t st, uint64_t *pages_out,
                         uint64_t *bytes_out, uint8_t *status_out = nullptr)
{
    PrepSmallParams pp{};
    int rc = fill_job_table(c, jobs, n_jobs, pp.jobs, nullptr, nullptr, need_tables, pages_out, bytes_out);
    if (rc != GK_OK) return rc;
    fill_seg_pow(c, crc, pp.seg_pow);
    pp.n_seg_pow = 2 * crc.nseg_max;
    uint32_t grid = n_jobs;
    if (clear_claims) {
        uint32_t g2 = (uint32_t)((num_pages + 1023) / 1024);
        if (g2 > 2048) g2 = 2048;
        if (g2 > grid) grid = g2;
    }
    c->ctr_next[0] = c->ctr_next[1] = 0;  // the kernel zeroes the device counters
    validate_args_kernel<<<grid, 1024, 0, st>>>(pp, w, num_pages, clear_claims, status_out);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched++;
    return GK_OK;
}

int launch_claim(gk_ctx *c, const WorkDev &w, cudaStream_t st)
{
    claim_kernel<<<(w.total_pages + 255) / 256, 256, 0, st>>>(w);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched++;
    return GK_OK;
}

int launch_finalize(gk_ctx *c, const WorkDev &w, const Tiling &tl, int write_mode, uint8_t *status, cudaStream_t st)
{
    finalize_kernel<<<(w.total_pages + 127) / 128, 128, 0, st>>>(c->gd, w, tl, write_mode, status);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched++;
    return GK_OK;
}

// Host tier (both directions): sizes of every job, the pinned-memory check, the
// two device staging slots, the place of every job in a slot and the batches.
struct HostPlan {
    struct Plan { uint64_t blob_bytes, sums_bytes, need; uint32_t pages; };
    std::vector<Plan> plan;
    std::vector<uint8_t *> blob_dev;
    std::vector<uint64_t *> sums_dev;
    std::vector<uint32_t> batch_end;  // exclusive job index per batch
    uint64_t pages = 0;
};

// The two device staging slots of the host tier, each of at least `want` bytes.
int ensure_slots(gk_ctx *c, uint64_t want)
{
    if (want < 256) want = 256;
    if (want <= c->slot_cap) return GK_OK;
    GK_CUDA(c, cudaDeviceSynchronize());
    for (int i = 0; i < kSlots; ++i) {
        if (c->d_slot[i]) cudaFree(c->d_slot[i]);
        c->d_slot[i] = nullptr;
        c->slot_used[i] = false;
    }
    c->slot_cap = 0;
    c->slot_next = 0;
    for (int i = 0; i < kSlots; ++i) {
        if (cudaMalloc(&c->d_slot[i], want) != cudaSuccess) {
            cudaGetLastError();
            return fail(c, GK_ERR_NOMEM, "host-tier staging slot of %llu bytes", (unsigned long long)want);
        }
    }
    c->slot_cap = want;
    c->stats.allocations++;
    return GK_OK;
}

// The page ids 0..num_pages-1 on the device; the windows of a streaming restore take their
// page tables as slices of them.
int ensure_iota(gk_ctx *c, uint64_t num_pages, cudaStream_t st)
{
    if (c->iota_cap >= num_pages) return GK_OK;
    GK_CUDA(c, cudaDeviceSynchronize());  // an earlier call's consumer may still read the old array
    if (c->d_iota) cudaFree(c->d_iota);
    c->d_iota = nullptr;
    c->iota_cap = 0;
    if (cudaMalloc(&c->d_iota, num_pages * sizeof(int32_t)) != cudaSuccess) {
        cudaGetLastError();
        return fail(c, GK_ERR_NOMEM, "page id array of %llu entries", (unsigned long long)num_pages);
    }
    c->iota_cap = num_pages;
    c->stats.allocations++;
    iota_kernel<<<(unsigned)((num_pages + 255) / 256), 256, 0, st>>>(c->d_iota, (uint32_t)num_pages);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched++;
    return GK_OK;
}

// Layer-wise restore: per-group result arrays (pages always, codes unless the caller keeps them).
int ensure_group_tmp(gk_ctx *c, uint32_t n_jobs)
{
    const size_t need = align_up((size_t)n_jobs * 4, 256) + (size_t)n_jobs;
    if (need <= c->group_tmp_cap) return GK_OK;
    GK_CUDA(c, cudaDeviceSynchronize());
    if (c->d_group_tmp) cudaFree(c->d_group_tmp);
    c->d_group_tmp = nullptr;
    c->group_tmp_cap = 0;
    if (cudaMalloc(&c->d_group_tmp, need * 2) != cudaSuccess) {
        cudaGetLastError();
        return fail(c, GK_ERR_NOMEM, "layer-wise result arrays of %zu bytes", need * 2);
    }
    c->group_tmp_cap = need * 2;
    c->stats.allocations++;
    return GK_OK;
}

// Pinned-memory check of the host tier.  The driver is asked once per buffer: start addresses
// that passed are remembered (sorted, at most 65,536 of them; the list starts afresh when full),
// so a call over thousands of blocks that were seen before costs no driver call at all.
bool is_pinned(gk_ctx *c, const void *ptr)
{
    auto it = std::lower_bound(c->pinned_seen.begin(), c->pinned_seen.end(), ptr);
    if (it != c->pinned_seen.end() && *it == ptr) return true;
    cudaPointerAttributes a{};
    if (cudaPointerGetAttributes(&a, ptr) != cudaSuccess || a.type != cudaMemoryTypeHost) {
        cudaGetLastError();
        return false;
    }
    if (c->pinned_seen.size() >= 65536) {
        c->pinned_seen.clear();
        it = c->pinned_seen.end();
    }
    c->pinned_seen.insert(it, ptr);
    return true;
}

int make_host_plan(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, bool allow_missing, HostPlan &hp)
{
    std::vector<HostPlan::Plan> &plan = hp.plan;
    plan.resize(n_jobs);
    uint64_t max_need = 0, total_need = 0, pages = 0;
    for (uint32_t j = 0; j < n_jobs; ++j) {
        if (jobs[j].n_tokens == 0) return fail(c, GK_ERR_ARG, "job %u: n_tokens == 0", j);
        const uint32_t np = pages_of(jobs[j].n_tokens, c->gd.page_tokens);
        plan[j].pages = np;
        plan[j].blob_bytes = (uint64_t)np * c->gd.S + (uint64_t)jobs[j].n_tokens * c->gd.tokB;
        plan[j].sums_bytes = (uint64_t)np * 8;
        plan[j].need = 0;
        pages += np;
        if (jobs[j].blob && jobs[j].checksums) {
            for (const void *ptr : {(const void *)jobs[j].blob, (const void *)jobs[j].checksums}) {
                if (!is_pinned(c, ptr))
                    return fail(c, GK_ERR_NOT_PINNED, "job %u: blob and checksums must be pinned host memory", j);
            }
            plan[j].need = align_up(plan[j].blob_bytes, 256) + align_up(plan[j].sums_bytes, 256);
        } else if (!allow_missing) {
            return fail(c, GK_ERR_ARG, "job %u: null blob or checksums", j);
        }
        if (plan[j].need > max_need) max_need = plan[j].need;
        total_need += plan[j].need;
    }
    hp.pages = pages;
    // staging slots: room for the largest job, and for batches of small jobs up to 256 MiB
    uint64_t want = max_need;
    const uint64_t batch_target = 256ull << 20;
    if (want < batch_target) want = total_need < batch_target ? total_need : batch_target;
    int rc_slots = ensure_slots(c, want);
    if (rc_slots != GK_OK) return rc_slots;
    // assign every job a place in a slot
    hp.blob_dev.assign(n_jobs, nullptr);
    hp.sums_dev.assign(n_jobs, nullptr);
    uint64_t used = 0;
    uint32_t b = 0;
    for (uint32_t j = 0; j < n_jobs; ++j) {
        if (used + plan[j].need > c->slot_cap && used > 0) {
            hp.batch_end.push_back(j);
            ++b;
            used = 0;
        }
        if (plan[j].need) {
            uint8_t *base = c->d_slot[(c->slot_next + b) % kSlots] + used;
            hp.blob_dev[j] = base;
            hp.sums_dev[j] = (uint64_t *)(base + align_up(plan[j].blob_bytes, 256));
            used += plan[j].need;
        }
    }
    hp.batch_end.push_back(n_jobs);
    return GK_OK;
}

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev)
    {
        cudaGetDevice(&prev);
        if (prev != dev) cudaSetDevice(dev);
        else prev = -1;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

}  // namespace

extern "C" {

int gk_blob_size(const gk_geom *geom, uint32_t n_tokens, uint64_t *blob_bytes, uint32_t *n_pages)
{
    GeomDev gd;
    const int rc = check_geom(geom, &gd);
    if (rc != GK_OK) return rc;
    if (n_tokens == 0) return GK_ERR_ARG;
    const uint32_t np = pages_of(n_tokens, gd.page_tokens);
    if (blob_bytes) *blob_bytes = (uint64_t)np * gd.S + (uint64_t)n_tokens * gd.tokB;
    if (n_pages) *n_pages = np;
    return GK_OK;
}

int gk_ctx_create(gk_ctx **out, const gk_geom *geom, int device)
{
    if (!out) return GK_ERR_ARG;
    *out = nullptr;
    GeomDev gd;
    int rc = check_geom(geom, &gd);
    if (rc != GK_OK) return rc;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        cudaGetLastError();
        return GK_ERR_CUDA;
    }
    gk_ctx *c = new (std::nothrow) gk_ctx();
    if (!c) return GK_ERR_NOMEM;
    c->geom = *geom;
    c->gd = gd;
    c->device = device;
    DeviceGuard guard(device);

    auto bail = [&](int code) {
        gk_ctx_destroy(c);
        return code;
    };
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return bail(GK_ERR_CUDA);
    if (prop.major != 10) return bail(GK_ERR_UNSUPPORTED);  // built for sm_100a only
    c->sm_count = prop.multiProcessorCount;

    // every streaming kernel: shared-memory size, then how many CTAs of it an SM holds
    int occ_quad[3] = {0, 0, 0};
    auto prepare = [&](auto *kernel, int threads, size_t smem, int *occ) {
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess &&
               cudaOccupancyMaxActiveBlocksPerMultiprocessor(occ, kernel, threads, smem) == cudaSuccess && *occ >= 1;
    };
    if (!prepare(stream_kernel<kVerify, GK_CRC_NT, GK_CRC_STAGE, GK_CRC_STAGES, GK_VERIFY_MINB>, VerifyCfg::kThreads,
                 VerifyCfg::kSmemBytes, &c->occ_verify) ||
        !prepare(stream_kernel<kPack, GK_CRC_NT, GK_PACK_STAGE, GK_PACK_STAGES, GK_PACK_MINB>, PackCfg::kThreads,
                 PackCfg::kSmemBytes, &c->occ_pack) ||
        !prepare(restore_kernel<GK_CRC_NT, GK_CRC_STAGE, GK_FUSED_VSTAGES, GK_COPY_STAGE, GK_FUSED_CSTAGES, GK_FUSED_MINB>,
                 FusedCfg::kThreads, FusedCfg::kSmemBytes, &c->occ_fused) ||
        !prepare(stream_kernel<kCommit, 0, GK_COPY_STAGE, GK_COPY_STAGES, GK_COPY_MINB>, CommitCfg::kThreads,
                 CommitCfg::kSmemBytes, &c->occ_commit) ||
        !prepare(stream_kernel<kSingle, GK_CRC_NT, GK_PACK_STAGE, GK_PACK_STAGES, GK_PACK_MINB>, SingleCfg::kThreads,
                 SingleCfg::kSmemBytes, &c->occ_single) ||
        // the page-quartet forms of the packing and of the fused kernel: same block shape, same occupancy
        !prepare(stream_kernel<kPack, GK_CRC_NT, GK_PACK_STAGE, GK_PACK_STAGES, GK_PACK_MINB, true>, PackCfg::kThreads,
                 PackCfg::kSmemBytes, &occ_quad[0]) ||
        !prepare(restore_kernel<GK_CRC_NT, GK_CRC_STAGE, GK_FUSED_VSTAGES, GK_COPY_STAGE, GK_FUSED_CSTAGES, GK_FUSED_MINB,
                                true>,
                 FusedCfg::kThreads, FusedCfg::kSmemBytes, &occ_quad[1]) ||
        !prepare(stream_kernel<kVerify, GK_CRC_NT, GK_CRC_STAGE, GK_CRC_STAGES, GK_VERIFY_MINB, true>, VerifyCfg::kThreads,
                 VerifyCfg::kSmemBytes, &occ_quad[2]) ||
        occ_quad[0] < c->occ_pack || occ_quad[1] < c->occ_fused || occ_quad[2] < c->occ_verify) {
        cudaGetLastError();
        return bail(GK_ERR_CUDA);
    }

    // tables: ones * x^(8*len(t)) for every page fill t, and the per-thread placement constants
    std::vector<uint64_t> init(gd.page_tokens + 1, 0);
    for (uint32_t t = 1; t <= gd.page_tokens; ++t)
        init[t] = gf_mul(~0ull, gf_xpow(8ull * (gd.S + (uint64_t)t * gd.tokB)));
    if (cudaMalloc(&c->d_init_term, init.size() * 8) != cudaSuccess || cudaMalloc(&c->d_error, 256) != cudaSuccess)
        return bail(GK_ERR_NOMEM);
    if (cudaMemcpy(c->d_init_term, init.data(), init.size() * 8, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(c->d_error, 0, 256) != cudaSuccess)
        return bail(GK_ERR_CUDA);
    std::vector<uint64_t> tc(QuadConst<GK_CRC_NT>::kOver0 + 2);
    for (int t = 0; t < GK_CRC_NT; ++t) tc[t] = gf_xpow(32ull * (GK_CRC_NT - 1 - t) + 64ull);
    for (int w = 0; w < GK_CRC_NT / 32; ++w)  // the two words that stick out above warp w
        for (int i = 0; i < 2; ++i) tc[GK_CRC_NT + 2 * w + i] = gf_xpow(1024ull * (GK_CRC_NT / 32 - w) + 64ull + 32ull * i);
    // page quartets: a record reduced by one warp alone
    for (int t = 0; t < 32; ++t) tc[QuadConst<GK_CRC_NT>::kLane0 + t] = gf_xpow(32ull * (31 - t) + 64ull);
    for (int i = 0; i < 2; ++i) tc[QuadConst<GK_CRC_NT>::kOver0 + i] = gf_xpow(1024ull + 64ull + 32ull * i);
    if (cudaMalloc(&c->d_thread_const, tc.size() * 8) != cudaSuccess) return bail(GK_ERR_NOMEM);
    if (cudaMemcpy(c->d_thread_const, tc.data(), tc.size() * 8, cudaMemcpyHostToDevice) != cudaSuccess)
        return bail(GK_ERR_CUDA);
    for (int i = 0; i < 2; ++i)
        if (cudaEventCreateWithFlags(&c->ev_stage[i], cudaEventDisableTiming) != cudaSuccess) return bail(GK_ERR_CUDA);
    if (cudaEventCreateWithFlags(&c->ev_entry, cudaEventDisableTiming) != cudaSuccess) return bail(GK_ERR_CUDA);
    for (int i = 0; i < kSlots; ++i) {
        if (cudaEventCreateWithFlags(&c->ev_slot_free[i], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_copied[i], cudaEventDisableTiming) != cudaSuccess)
            return bail(GK_ERR_CUDA);
    }
    if (cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return bail(GK_ERR_CUDA);
    *out = c;
    return GK_OK;
}

int gk_ctx_destroy(gk_ctx *c)
{
    if (!c) return GK_OK;
    DeviceGuard guard(c->device);
    cudaDeviceSynchronize();
    if (c->twin) gk_ctx_destroy(c->twin);
    for (int i = 0; i < 2; ++i) {
        if (c->lw_stream[i]) cudaStreamDestroy(c->lw_stream[i]);
        if (c->lw_done[i]) cudaEventDestroy(c->lw_done[i]);
        if (c->lw_merged[i]) cudaEventDestroy(c->lw_merged[i]);
    }
    if (c->lw_entry) cudaEventDestroy(c->lw_entry);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    for (auto &ps : c->prof_pool) {
        cudaEventDestroy(ps.a);
        cudaEventDestroy(ps.b);
    }
    for (int i = 0; i < kSlots; ++i) {
        if (c->d_slot[i]) cudaFree(c->d_slot[i]);
        if (c->ev_slot_free[i]) cudaEventDestroy(c->ev_slot_free[i]);
        if (c->ev_copied[i]) cudaEventDestroy(c->ev_copied[i]);
    }
    for (int i = 0; i < 2; ++i)
        if (c->ev_stage[i]) cudaEventDestroy(c->ev_stage[i]);
    if (c->ev_entry) cudaEventDestroy(c->ev_entry);
    if (c->h_stage) cudaFreeHost(c->h_stage);
    if (c->d_ws) cudaFree(c->d_ws);
    if (c->d_iota) cudaFree(c->d_iota);
    if (c->d_group_tmp) cudaFree(c->d_group_tmp);
    if (c->d_init_term) cudaFree(c->d_init_term);
    if (c->d_thread_const) cudaFree(c->d_thread_const);
    if (c->d_error) cudaFree(c->d_error);
    cudaGetLastError();
    delete c;
    return GK_OK;
}

const char *gk_last_error(const gk_ctx *c) { return c ? c->err : "null context"; }

int gk_ctx_set_tuning(gk_ctx *c, const char *key, uint32_t value)
{
    if (!c || !key) return GK_ERR_ARG;
    if (!strcmp(key, "seg_granules")) c->seg_granules = value;
    else if (!strcmp(key, "commit_seg_tiles")) c->commit_seg_tiles = value;
    else if (!strcmp(key, "grid_cap")) c->grid_cap = value;
    else if (!strcmp(key, "profile")) c->profile = value != 0;
    else if (!strcmp(key, "fused")) c->fused = value != 0;
    else if (!strcmp(key, "wait_limit_ms")) c->wait_limit_ns = (unsigned long long)(value ? value : 1u) * 1000000ull;
    else if (!strcmp(key, "test_drop_verify")) c->test_drop_verify = value;
    else if (!strcmp(key, "commit_reverse")) c->commit_reverse = value != 0;
    else if (!strcmp(key, "l2_hints")) c->l2_hints = value;
    else if (!strcmp(key, "commit_items_per_cta")) c->commit_items_per_cta = value ? value : 1u;
    else if (!strcmp(key, "quad")) c->quad_mode = value <= 2u ? value : 0u;
#ifdef GK_DEBUG
    else if (!strcmp(key, "debug_extent_cut")) c->debug_extent_cut = value;
#endif
#ifdef GK_TRACE
    else if (!strcmp(key, "trace_lo")) c->trace = (unsigned long long *)(((uintptr_t)c->trace & ~(uintptr_t)0xffffffffull) | value);
    else if (!strcmp(key, "trace_hi")) c->trace = (unsigned long long *)(((uintptr_t)c->trace & 0xffffffffull) | ((uintptr_t)value << 32));
#endif
    else return fail(c, GK_ERR_ARG, "unknown tuning key %s", key);
    if (c->twin) return gk_ctx_set_tuning(c->twin, key, value);
    return GK_OK;
}

// The twin of a context (layer-wise calls on the device tier): same geometry, same tuning, its own workspace,
// error word and counters; gk_get_stats, gk_ctx_clear_error and gk_debug_status of the context cover both.
static int ensure_twin(gk_ctx *c)
{
    if (c->twin) return GK_OK;
    gk_ctx *t = nullptr;
    int rc = gk_ctx_create(&t, &c->geom, c->device);
    if (rc != GK_OK) return fail(c, rc, "layer-wise: no second context");
    t->seg_granules = c->seg_granules;
    t->commit_seg_tiles = c->commit_seg_tiles;
    t->grid_cap = c->grid_cap;
    t->fused = c->fused;
    t->wait_limit_ns = c->wait_limit_ns;
    t->test_drop_verify = c->test_drop_verify;
    t->commit_reverse = c->commit_reverse;
    t->l2_hints = c->l2_hints;
    t->commit_items_per_cta = c->commit_items_per_cta;
    t->quad_mode = c->quad_mode;
    t->debug_extent_cut = c->debug_extent_cut;
    t->trace = c->trace;
    for (int i = 0; i < 2; ++i) {
        if (cudaStreamCreateWithFlags(&c->lw_stream[i], cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->lw_done[i], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->lw_merged[i], cudaEventDisableTiming) != cudaSuccess) {
            gk_ctx_destroy(t);
            return fail(c, GK_ERR_CUDA, "layer-wise: streams and events");
        }
    }
    if (cudaEventCreateWithFlags(&c->lw_entry, cudaEventDisableTiming) != cudaSuccess) {
        gk_ctx_destroy(t);
        return fail(c, GK_ERR_CUDA, "layer-wise: streams and events");
    }
    t->is_twin = true;
    c->twin = t;
    c->stats.allocations++;
    return GK_OK;
}

int gk_ctx_reserve(gk_ctx *c, uint32_t max_jobs, uint64_t max_pages, uint64_t num_pages, uint64_t max_host_batch_bytes)
{
    if (!c) return GK_ERR_ARG;
    if (max_pages > 0x7fffffffull || num_pages > 0x7fffffffull) return fail(c, GK_ERR_ARG, "too many pages");
    DeviceGuard guard(c->device);
    // the largest tables any call within these bounds builds: a page cut into as many segments as it has granules
    const uint32_t seg_max = (uint32_t)((c->gd.R + VerifyCfg::kGran - 1) / VerifyCfg::kGran);
    const WsLayout l = ws_layout(max_jobs, max_pages, seg_max, num_pages);
    int rc;
    if ((rc = ensure_workspace(c, l.total)) != GK_OK) return rc;
    if ((rc = ensure_host_stage(c, (size_t)max_jobs * sizeof(JobDev) + (size_t)seg_max * 16)) != GK_OK) return rc;
    if (max_jobs && (rc = ensure_group_tmp(c, max_jobs)) != GK_OK) return rc;
    if (max_jobs && !c->profile && !c->is_twin) {  // layer-wise calls on the device tier use a second context
        if ((rc = ensure_twin(c)) != GK_OK) return rc;
        if ((rc = gk_ctx_reserve(c->twin, max_jobs, max_pages, num_pages, 0)) != GK_OK) return rc;
    }
    if (max_host_batch_bytes) {
        // room for the checksums beside the blobs, and for the alignment of every job's two parts
        const uint64_t want = max_host_batch_bytes + max_pages * 8 + (uint64_t)max_jobs * 512;
        if ((rc = ensure_slots(c, want)) != GK_OK) return rc;
        if (num_pages && (rc = ensure_iota(c, num_pages, 0)) != GK_OK) return rc;
    }
    GK_CUDA(c, cudaDeviceSynchronize());
    return GK_OK;
}

int gk_ctx_clear_error(gk_ctx *c, void *stream)
{
    if (!c) return GK_ERR_ARG;
    DeviceGuard guard(c->device);
    GK_CUDA(c, cudaMemsetAsync(c->d_error, 0, 4, (cudaStream_t)stream));
    if (c->twin) GK_CUDA(c, cudaMemsetAsync(c->twin->d_error, 0, 4, (cudaStream_t)stream));
    return GK_OK;
}

int gk_pack_batch(gk_ctx *c, const gk_cache *src, const gk_job *jobs, uint32_t n_jobs, uint8_t *status_dev,
                  void *stream)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0) return GK_OK;
    if (!jobs) return fail(c, GK_ERR_ARG, "null job array");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    CacheDev cd;
    int rc = check_cache(c, src, &cd);
    if (rc != GK_OK) return rc;
    for (uint32_t j = 0; j < n_jobs; ++j)
        if (!jobs[j].blob || !jobs[j].checksums) return fail(c, GK_ERR_ARG, "job %u: null output", j);

    uint64_t pages = 0, bytes = 0;
    for (uint32_t j = 0; j < n_jobs; ++j) pages += pages_of(jobs[j].n_tokens, c->gd.page_tokens);
    const Tiling tl = crc_tiling(c, GK_CRC_STAGE, pages, c->occ_pack, false, kQuadPack);
    const WsLayout l = ws_layout(n_jobs, pages, tl.nseg_max, 0);
    if ((rc = ensure_workspace(c, l.total)) != GK_OK) return rc;
    WorkDev w = make_work(c, l, n_jobs, (uint32_t)pages, tl);
    if (is_small_call(n_jobs, pages, tl)) {
        if ((rc = launch_prep_small(c, jobs, n_jobs, tl, w, cd.num_pages, true, false, st, &pages, &bytes,
                                    status_dev)) != GK_OK)
            return rc;
    } else {
        if (table_fits_args(n_jobs, tl)) {
            if ((rc = launch_validate_args(c, jobs, n_jobs, tl, w, cd.num_pages, 0, true, st, &pages, &bytes,
                                           status_dev)) != GK_OK)
                return rc;
        } else {
            if ((rc = upload_jobs(c, jobs, n_jobs, l, tl, nullptr, nullptr, true, st, &pages, &bytes)) != GK_OK)
                return rc;
            if ((rc = launch_validate(c, w, cd.num_pages, 0, st, status_dev)) != GK_OK) return rc;
        }
        c->pdl_next = !c->profile;  // the packing kernel sets its rings up while the validation runs
    }
    StreamParams P{};
    P.g = c->gd;
    P.cache = cd;
    P.w = w;
    P.tl = tl;
    P.n_items = crc_items(tl, pages);
    P.inline_final = 1u;  // checksums are written by the CTA that delivers a page's last segment
    if ((rc = launch_pack(c, P, st)) != GK_OK) return rc;
    c->stats.calls_pack++;
    c->stats.jobs += n_jobs;
    c->stats.pages += pages;
    c->stats.bytes_blob += bytes;
    return GK_OK;
}

int gk_pack(gk_ctx *c, const gk_cache *src, const int32_t *page_table_dev, uint32_t n_tokens, void *blob_dev,
            uint64_t *checksums_dev, uint8_t *status_dev, void *stream)
{
    gk_job jb{};
    jb.blob = blob_dev;
    jb.checksums = checksums_dev;
    jb.page_table = page_table_dev;
    jb.n_tokens = n_tokens;
    return gk_pack_batch(c, src, &jb, 1, status_dev, stream);
}

int gk_page_checksums(gk_ctx *c, const void *blob_dev, uint32_t n_tokens, uint64_t *checksums_dev, void *stream)
{
    if (!c) return GK_ERR_ARG;
    if (!blob_dev || !checksums_dev || n_tokens == 0) return fail(c, GK_ERR_ARG, "null blob/checksums or zero tokens");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    gk_job jb{};
    jb.blob = const_cast<void *>(blob_dev);
    jb.checksums = checksums_dev;
    jb.page_table = nullptr;
    jb.n_tokens = n_tokens;
    uint64_t pages = pages_of(n_tokens, c->gd.page_tokens), bytes = 0;
    const Tiling tl = crc_tiling(c, GK_CRC_STAGE, pages, c->occ_verify, false, kQuadRestore);
    const WsLayout l = ws_layout(1, pages, tl.nseg_max, 0);
    int rc;
    if ((rc = ensure_workspace(c, l.total)) != GK_OK) return rc;
    if ((rc = upload_jobs(c, &jb, 1, l, tl, nullptr, nullptr, false, st, &pages, &bytes)) != GK_OK) return rc;
    WorkDev w = make_work(c, l, 1, (uint32_t)pages, tl);
    if ((rc = launch_validate(c, w, 0, 0, st)) != GK_OK) return rc;
    StreamParams P{};
    P.g = c->gd;
    P.w = w;
    P.tl = tl;
    P.n_items = crc_items(tl, pages);
    if ((rc = launch_verify(c, P, st)) != GK_OK) return rc;
    if ((rc = launch_finalize(c, w, tl, 1, nullptr, st)) != GK_OK) return rc;
    c->stats.pages += pages;
    c->stats.bytes_blob += bytes;
    return GK_OK;
}

// verify + commit for the pages [page_begin, page_begin + n_pages) of the call
static int enqueue_verify_commit(gk_ctx *c, WorkDev w, const CacheDev &cd, const Tiling &tlv, const Tiling &tlc,
                                 uint32_t page_begin, uint32_t n_pages, uint8_t *mask_dev,
                                 int32_t *first_bad_dev, cudaStream_t st)
{
    int rc;
    w.page_begin = page_begin;
    w.total_pages = n_pages;
    StreamParams P{};
    P.g = c->gd;
    P.cache = cd;
    P.w = w;
    P.mask_out = mask_dev;
    P.first_bad_out = first_bad_dev;
    P.tl = tlv;
    P.tlc = tlc;
    P.n_items = crc_items(tlv, n_pages);
    P.n_items_c = n_pages * tlc.nseg_max;
    P.commit_reverse = c->commit_reverse ? 1u : 0u;
    P.l2_hints = c->l2_hints;
    if (c->gd.flags & GK_FLAG_SKIP_VERIFY) return launch_commit(c, P, st);
    if (c->gd.flags & GK_FLAG_SINGLE_PASS) {
        // one pass: every tile is checksummed and scattered from the same shared-memory stage;
        // the codes are known only when the launch has ended, so a small kernel reports them
        P.inline_final = 1u;
        if ((rc = launch_single(c, P, st)) != GK_OK) return rc;
        report_kernel<<<(w.n_jobs + 127) / 128, 128, 0, st>>>(w, mask_dev, first_bad_dev);
        GK_CUDA(c, cudaGetLastError());
        c->stats.kernels_launched++;
        return GK_OK;
    }
    if (c->fused) {
        P.fused = 1u;
        P.inline_final = 1u;
        P.test_drop_from = c->test_drop_verify;  // tests: the jobs from this one on are never verified
        return launch_fused(c, P, st);
    }
    if ((rc = launch_verify(c, P, st)) != GK_OK) return rc;
    if ((rc = launch_finalize(c, w, tlv, 0, nullptr, st)) != GK_OK) return rc;
    return launch_commit(c, P, st);
}

int gk_restore(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst, uint8_t *mask_dev,
               int32_t *first_bad_page_dev, void *stream)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0) return GK_OK;
    if (!jobs || !mask_dev || !first_bad_page_dev) return fail(c, GK_ERR_ARG, "null jobs, mask or first_bad_page");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    CacheDev cd;
    int rc = check_cache(c, dst, &cd);
    if (rc != GK_OK) return rc;

    uint64_t pages = 0, bytes = 0;
    for (uint32_t j = 0; j < n_jobs; ++j) pages += pages_of(jobs[j].n_tokens, c->gd.page_tokens);
    const bool single = (c->gd.flags & GK_FLAG_SINGLE_PASS) && !(c->gd.flags & GK_FLAG_SKIP_VERIFY);
    const bool fused = !single && c->fused && !(c->gd.flags & GK_FLAG_SKIP_VERIFY);
    const Tiling tlv = crc_tiling(c, GK_CRC_STAGE, pages,
                                  single ? c->occ_single : fused ? c->occ_fused : c->occ_verify, fused && n_jobs > 1,
                                  single ? kNoQuad : kQuadRestore);
    const Tiling tlc = commit_tiling(c, GK_COPY_STAGE, pages, fused ? c->occ_fused : c->occ_commit);
    const WsLayout l = ws_layout(n_jobs, pages, tlv.nseg_max, cd.num_pages);
    if ((rc = ensure_workspace(c, l.total)) != GK_OK) return rc;
    WorkDev w = make_work(c, l, n_jobs, (uint32_t)pages, tlv);
    if (is_small_call(n_jobs, pages, tlv)) {
        if ((rc = launch_prep_small(c, jobs, n_jobs, tlv, w, cd.num_pages, true, true, st, &pages, &bytes)) != GK_OK)
            return rc;
    } else {
        if (table_fits_args(n_jobs, tlv)) {
            if ((rc = launch_validate_args(c, jobs, n_jobs, tlv, w, cd.num_pages, 1, true, st, &pages, &bytes)) != GK_OK)
                return rc;
        } else {
            if ((rc = upload_jobs(c, jobs, n_jobs, l, tlv, nullptr, nullptr, true, st, &pages, &bytes)) != GK_OK)
                return rc;
            if ((rc = launch_validate(c, w, cd.num_pages, 1, st)) != GK_OK) return rc;
        }
        if ((rc = launch_claim(c, w, st)) != GK_OK) return rc;
        c->pdl_next = !c->profile;  // the first streaming kernel sets its rings up while the claims are made
    }
    if ((rc = enqueue_verify_commit(c, w, cd, tlv, tlc, 0, (uint32_t)pages, mask_dev, first_bad_page_dev, st)) != GK_OK)
        return rc;
    c->stats.calls_restore++;
    c->stats.jobs += n_jobs;
    c->stats.pages += pages;
    c->stats.bytes_blob += bytes;
    return GK_OK;
}

// shared front part of gk_verify / gk_commit: job table, page tables, claims
static int prepare_restore(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst, cudaStream_t st,
                           CacheDev *cd, Tiling *tlv, Tiling *tlc, WorkDev *w, uint64_t *pages_out, uint64_t *bytes_out)
{
    int rc = check_cache(c, dst, cd);
    if (rc != GK_OK) return rc;
    uint64_t pages = 0, bytes = 0;
    for (uint32_t j = 0; j < n_jobs; ++j) pages += pages_of(jobs[j].n_tokens, c->gd.page_tokens);
    *tlv = crc_tiling(c, GK_CRC_STAGE, pages, c->occ_verify, false, kQuadRestore);
    *tlc = commit_tiling(c, GK_COPY_STAGE, pages, c->occ_commit);
    const WsLayout l = ws_layout(n_jobs, pages, tlv->nseg_max, cd->num_pages);
    if ((rc = ensure_workspace(c, l.total)) != GK_OK) return rc;
    *w = make_work(c, l, n_jobs, (uint32_t)pages, *tlv);
    if (is_small_call(n_jobs, pages, *tlv)) {
        if ((rc = launch_prep_small(c, jobs, n_jobs, *tlv, *w, cd->num_pages, true, true, st, &pages, &bytes)) != GK_OK)
            return rc;
    } else {
        if ((rc = upload_jobs(c, jobs, n_jobs, l, *tlv, nullptr, nullptr, true, st, &pages, &bytes)) != GK_OK) return rc;
        if ((rc = launch_validate(c, *w, cd->num_pages, 1, st)) != GK_OK) return rc;
        if ((rc = launch_claim(c, *w, st)) != GK_OK) return rc;
    }
    *pages_out = pages;
    *bytes_out = bytes;
    return GK_OK;
}

int gk_verify(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst, uint8_t *mask_dev,
              int32_t *first_bad_page_dev, void *stream)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0) return GK_OK;
    if (!jobs || !mask_dev || !first_bad_page_dev) return fail(c, GK_ERR_ARG, "null jobs, mask or first_bad_page");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    CacheDev cd;
    Tiling tlv, tlc;
    WorkDev w;
    uint64_t pages, bytes;
    int rc = prepare_restore(c, jobs, n_jobs, dst, st, &cd, &tlv, &tlc, &w, &pages, &bytes);
    if (rc != GK_OK) return rc;
    if (!(c->gd.flags & GK_FLAG_SKIP_VERIFY)) {
        StreamParams P{};
        P.g = c->gd;
        P.w = w;
        P.tl = tlv;
        P.n_items = crc_items(tlv, pages);
        if ((rc = launch_verify(c, P, st)) != GK_OK) return rc;
        if ((rc = launch_finalize(c, w, tlv, 0, nullptr, st)) != GK_OK) return rc;
    }
    report_kernel<<<(n_jobs + 127) / 128, 128, 0, st>>>(w, mask_dev, first_bad_page_dev);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched++;
    c->stats.jobs += n_jobs;
    c->stats.pages += pages;
    c->stats.bytes_blob += bytes;
    return GK_OK;
}

int gk_commit(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst, const uint8_t *mask_dev,
              void *stream)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0) return GK_OK;
    if (!jobs || !mask_dev) return fail(c, GK_ERR_ARG, "null jobs or mask");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    CacheDev cd;
    Tiling tlv, tlc;
    WorkDev w;
    uint64_t pages, bytes;
    int rc = prepare_restore(c, jobs, n_jobs, dst, st, &cd, &tlv, &tlc, &w, &pages, &bytes);
    if (rc != GK_OK) return rc;
    w.ext_mask = mask_dev;
    StreamParams P{};
    P.g = c->gd;
    P.cache = cd;
    P.w = w;
    P.tl = tlv;
    P.tlc = tlc;
    P.n_items_c = (uint32_t)pages * tlc.nseg_max;
    if ((rc = launch_commit(c, P, st)) != GK_OK) return rc;
    c->stats.calls_restore++;
    return GK_OK;
}

// order_after_stream: the host buffers may still be being written by earlier work on the
// caller's stream, so the first copy must wait for that work.  The streaming restore passes
// false for every window but the first: its buffers were ready when the call came in, and the
// copies of a window are meant to run under the consumer of the window before it.
static int restore_host_impl(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst, uint8_t *mask_dev,
                             int32_t *first_bad_page_dev, void *stream, bool order_after_stream)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0) return GK_OK;
    if (!jobs || !mask_dev || !first_bad_page_dev) return fail(c, GK_ERR_ARG, "null jobs, mask or first_bad_page");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    CacheDev cd;
    int rc = check_cache(c, dst, &cd);
    if (rc != GK_OK) return rc;
    if (order_after_stream) {
        GK_CUDA(c, cudaEventRecord(c->ev_entry, st));
        GK_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->ev_entry, 0));
    }

    HostPlan hp;
    if ((rc = make_host_plan(c, jobs, n_jobs, true, hp)) != GK_OK) return rc;
    std::vector<HostPlan::Plan> &plan = hp.plan;
    std::vector<uint8_t *> &blob_dev = hp.blob_dev;
    std::vector<uint64_t *> &sums_dev = hp.sums_dev;
    std::vector<uint32_t> &batch_end = hp.batch_end;
    uint64_t pages = hp.pages;

    // batches are what is launched, so size the work items for a batch, not for the call
    const uint64_t pages_per_launch = (pages + batch_end.size() - 1) / batch_end.size();
    const bool single = (c->gd.flags & GK_FLAG_SINGLE_PASS) && !(c->gd.flags & GK_FLAG_SKIP_VERIFY);
    const bool fused = c->fused && !single && !(c->gd.flags & GK_FLAG_SKIP_VERIFY);
    const int occ = single ? c->occ_single : fused ? c->occ_fused : c->occ_verify;
    const Tiling tlv = crc_tiling(c, GK_CRC_STAGE, pages_per_launch, occ, fused && n_jobs > batch_end.size(),
                                  single ? kNoQuad : kQuadRestore);
    const Tiling tlc = commit_tiling(c, GK_COPY_STAGE, pages_per_launch, fused ? c->occ_fused : c->occ_commit);
    const WsLayout l = ws_layout(n_jobs, pages, tlv.nseg_max, cd.num_pages);
    if ((rc = ensure_workspace(c, l.total)) != GK_OK) return rc;
    uint64_t bytes = 0;
    if ((rc = upload_jobs(c, jobs, n_jobs, l, tlv, blob_dev.data(), sums_dev.data(), true, st, &pages, &bytes)) != GK_OK)
        return rc;
    WorkDev w = make_work(c, l, n_jobs, (uint32_t)pages, tlv);
    if ((rc = launch_validate(c, w, cd.num_pages, 1, st)) != GK_OK) return rc;
    if ((rc = launch_claim(c, w, st)) != GK_OK) return rc;

    uint32_t j0 = 0, page0 = 0;
    for (size_t b = 0; b < batch_end.size(); ++b) {
        const int slot = (int)((c->slot_next + b) % kSlots);
        const uint32_t j1 = batch_end[b];
        if (c->slot_used[slot]) GK_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->ev_slot_free[slot], 0));
        uint32_t npages = 0;
        for (uint32_t j = j0; j < j1; ++j) {
            npages += plan[j].pages;
            if (!plan[j].need) continue;
            GK_CUDA(c, cudaMemcpyAsync(blob_dev[j], jobs[j].blob, plan[j].blob_bytes, cudaMemcpyHostToDevice,
                                       c->copy_stream));
            GK_CUDA(c, cudaMemcpyAsync(sums_dev[j], jobs[j].checksums, plan[j].sums_bytes, cudaMemcpyHostToDevice,
                                       c->copy_stream));
        }
        GK_CUDA(c, cudaEventRecord(c->ev_copied[slot], c->copy_stream));
        GK_CUDA(c, cudaStreamWaitEvent(st, c->ev_copied[slot], 0));
        if ((rc = enqueue_verify_commit(c, w, cd, tlv, tlc, page0, npages, mask_dev, first_bad_page_dev, st)) != GK_OK)
            return rc;
        GK_CUDA(c, cudaEventRecord(c->ev_slot_free[slot], st));
        c->slot_used[slot] = true;
        j0 = j1;
        page0 += npages;
    }
    c->slot_next = (uint32_t)((c->slot_next + batch_end.size()) % kSlots);
    c->stats.calls_restore_host++;
    c->stats.jobs += n_jobs;
    c->stats.pages += pages;
    c->stats.bytes_blob += bytes;
    return GK_OK;
}

int gk_restore_host(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst, uint8_t *mask_dev,
                    int32_t *first_bad_page_dev, void *stream)
{
    return restore_host_impl(c, jobs, n_jobs, dst, mask_dev, first_bad_page_dev, stream, true);
}

int gk_restore_stream(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const gk_cache *ring, uint8_t *mask_dev,
                      int32_t *first_bad_page_dev, gk_window_fn consume, void *user, void *stream)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0) return GK_OK;
    if (!jobs || !mask_dev || !first_bad_page_dev) return fail(c, GK_ERR_ARG, "null jobs, mask or first_bad_page");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    CacheDev cd;
    int rc = check_cache(c, ring, &cd);
    if (rc != GK_OK) return rc;
    std::vector<uint32_t> np(n_jobs);
    for (uint32_t j = 0; j < n_jobs; ++j) {
        if (jobs[j].n_tokens == 0) return fail(c, GK_ERR_ARG, "job %u: n_tokens == 0", j);
        np[j] = pages_of(jobs[j].n_tokens, c->gd.page_tokens);
        if ((uint64_t)np[j] > cd.num_pages)
            return fail(c, GK_ERR_TOO_LARGE, "job %u: %u pages do not fit a ring of %llu", j, np[j],
                        (unsigned long long)cd.num_pages);
    }
    if ((rc = ensure_iota(c, cd.num_pages, st)) != GK_OK) return rc;
    std::vector<gk_job> wjobs;
    std::vector<gk_window_block> blocks;
    uint32_t j0 = 0;
    while (j0 < n_jobs) {
        uint64_t used = 0;
        uint32_t j1 = j0;
        wjobs.clear();
        blocks.clear();
        while (j1 < n_jobs && used + np[j1] <= cd.num_pages) {
            gk_job w = jobs[j1];
            w.page_table = c->d_iota + used;
            wjobs.push_back(w);
            blocks.push_back(gk_window_block{j1, jobs[j1].n_tokens, c->d_iota + used});
            used += np[j1];
            ++j1;
        }
        rc = restore_host_impl(c, wjobs.data(), j1 - j0, ring, mask_dev + j0, first_bad_page_dev + j0, stream, j0 == 0);
        if (rc != GK_OK) return rc;
        if (consume) consume(user, blocks.data(), j1 - j0, mask_dev, stream);
        j0 = j1;
    }
    c->stats.calls_restore_stream++;
    return GK_OK;
}

int gk_pack_host(gk_ctx *c, const gk_cache *src, const gk_job *jobs, uint32_t n_jobs, uint8_t *status_dev,
                 void *stream)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0) return GK_OK;
    if (!jobs) return fail(c, GK_ERR_ARG, "null job array");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    CacheDev cd;
    int rc = check_cache(c, src, &cd);
    if (rc != GK_OK) return rc;
    HostPlan hp;
    if ((rc = make_host_plan(c, jobs, n_jobs, false, hp)) != GK_OK) return rc;

    uint64_t pages = hp.pages, bytes = 0;
    const Tiling tl = crc_tiling(c, GK_CRC_STAGE, (pages + hp.batch_end.size() - 1) / hp.batch_end.size(), c->occ_pack,
                                 false, kQuadPack);
    const WsLayout l = ws_layout(n_jobs, pages, tl.nseg_max, 0);
    if ((rc = ensure_workspace(c, l.total)) != GK_OK) return rc;
    if ((rc = upload_jobs(c, jobs, n_jobs, l, tl, hp.blob_dev.data(), hp.sums_dev.data(), true, st, &pages, &bytes)) != GK_OK)
        return rc;
    WorkDev w = make_work(c, l, n_jobs, (uint32_t)pages, tl);
    if ((rc = launch_validate(c, w, cd.num_pages, 0, st, status_dev)) != GK_OK) return rc;

    uint32_t j0 = 0, page0 = 0;
    int last_slot[kSlots] = {0, 0};
    for (size_t b = 0; b < hp.batch_end.size(); ++b) {
        const int slot = (int)((c->slot_next + b) % kSlots);
        const uint32_t j1 = hp.batch_end[b];
        // the slot's previous contents must have left (earlier D2H, or an earlier restore reading it)
        if (c->slot_used[slot]) GK_CUDA(c, cudaStreamWaitEvent(st, c->ev_slot_free[slot], 0));
        uint32_t npages = 0;
        for (uint32_t j = j0; j < j1; ++j) npages += hp.plan[j].pages;
        WorkDev wb = w;
        wb.page_begin = page0;
        wb.total_pages = npages;
        StreamParams P{};
        P.g = c->gd;
        P.cache = cd;
        P.w = wb;
        P.tl = tl;
        P.n_items = crc_items(tl, npages);
        P.inline_final = 1u;
        if ((rc = launch_pack(c, P, st)) != GK_OK) return rc;
        GK_CUDA(c, cudaEventRecord(c->ev_copied[slot], st));
        GK_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->ev_copied[slot], 0));
        for (uint32_t j = j0; j < j1; ++j) {
            GK_CUDA(c, cudaMemcpyAsync(jobs[j].blob, hp.blob_dev[j], hp.plan[j].blob_bytes, cudaMemcpyDeviceToHost,
                                       c->copy_stream));
            GK_CUDA(c, cudaMemcpyAsync(jobs[j].checksums, hp.sums_dev[j], hp.plan[j].sums_bytes,
                                       cudaMemcpyDeviceToHost, c->copy_stream));
        }
        GK_CUDA(c, cudaEventRecord(c->ev_slot_free[slot], c->copy_stream));
        c->slot_used[slot] = true;
        last_slot[slot] = 1;
        j0 = j1;
        page0 += npages;
    }
    // the caller's stream is complete only when the last copies have landed
    for (int i = 0; i < kSlots; ++i)
        if (last_slot[i]) GK_CUDA(c, cudaStreamWaitEvent(st, c->ev_slot_free[i], 0));
    c->slot_next = (uint32_t)((c->slot_next + hp.batch_end.size()) % kSlots);
    c->stats.calls_pack++;
    c->stats.jobs += n_jobs;
    c->stats.pages += pages;
    c->stats.bytes_blob += bytes;
    return GK_OK;
}

// ---------------------------------------------------------------------------
// layer-wise save and load: the ordinary calls, once per group of layers, over
// the cache restricted to the group and the group's part of every blob
// ---------------------------------------------------------------------------
static gk_cache group_view(const gk_ctx *c, const gk_cache *k, uint32_t group)
{
    gk_cache v = *k;
    v.data = (uint8_t *)k->data + (uint64_t)group * c->gd.layers * k->layer_stride;
    if (k->scales) v.scales = (uint8_t *)k->scales + (uint64_t)group * c->gd.layers * k->s_layer_stride;
    return v;
}

static void group_jobs(const gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, uint32_t group, std::vector<gk_job> &out)
{
    out.assign(jobs, jobs + n_jobs);
    for (uint32_t j = 0; j < n_jobs; ++j) {
        const uint32_t np = pages_of(jobs[j].n_tokens, c->gd.page_tokens);
        const uint64_t bytes = (uint64_t)np * c->gd.S + (uint64_t)jobs[j].n_tokens * c->gd.tokB;
        if (out[j].blob) out[j].blob = (uint8_t *)jobs[j].blob + (uint64_t)group * bytes;
        if (out[j].checksums) out[j].checksums = jobs[j].checksums + (uint64_t)group * np;
    }
}

// Layer-wise calls on the device tier alternate between the context and its twin (see gk_ctx::twin); per-kernel
// timing keeps everything in one context, where its event pool is.
static bool lw_two_streams(const gk_ctx *c, uint32_t n_groups, bool host)
{
    return !host && n_groups > 1 && !c->profile;
}

static int pack_layerwise_impl(gk_ctx *c, uint32_t n_groups, const gk_cache *src, const gk_job *jobs, uint32_t n_jobs,
                               uint8_t *status_dev, void *stream, bool host)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0 || n_groups == 0) return GK_OK;
    if (!jobs || !src) return fail(c, GK_ERR_ARG, "null jobs or cache");
    for (uint32_t j = 0; j < n_jobs; ++j)
        if (jobs[j].n_tokens == 0) return fail(c, GK_ERR_ARG, "job %u: n_tokens == 0", j);
    std::vector<gk_job> gj;
    if (!lw_two_streams(c, n_groups, host)) {
        for (uint32_t k = 0; k < n_groups; ++k) {
            const gk_cache view = group_view(c, src, k);
            group_jobs(c, jobs, n_jobs, k, gj);
            const int rc = host ? gk_pack_host(c, &view, gj.data(), n_jobs, status_dev, stream)
                                : gk_pack_batch(c, &view, gj.data(), n_jobs, status_dev, stream);
            if (rc != GK_OK) return rc;
        }
        return GK_OK;
    }
    // device tier: the groups are independent of one another (their own layers of the cache, their own part of
    // every blob), so they go in turn to two contexts on two streams; every group writes the same status bytes
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    int rc = ensure_twin(c);
    if (rc != GK_OK) return rc;
    GK_CUDA(c, cudaEventRecord(c->lw_entry, st));
    for (int i = 0; i < 2; ++i) GK_CUDA(c, cudaStreamWaitEvent(c->lw_stream[i], c->lw_entry, 0));
    for (uint32_t k = 0; k < n_groups; ++k) {
        gk_ctx *ck = (k & 1u) ? c->twin : c;
        const gk_cache view = group_view(c, src, k);
        group_jobs(c, jobs, n_jobs, k, gj);
        rc = gk_pack_batch(ck, &view, gj.data(), n_jobs, status_dev, c->lw_stream[k & 1u]);
        if (rc != GK_OK) {
            if (ck != c) fail(c, rc, "%s", ck->err);
            break;
        }
    }
    // the caller's stream goes on when both streams are through (also after a failure: what was enqueued runs)
    for (int i = 0; i < 2; ++i) {
        GK_CUDA(c, cudaEventRecord(c->lw_done[i], c->lw_stream[i]));
        GK_CUDA(c, cudaStreamWaitEvent(st, c->lw_done[i], 0));
    }
    return rc;
}

static int restore_layerwise_impl(gk_ctx *c, uint32_t n_groups, const gk_job *jobs, uint32_t n_jobs,
                                  const gk_cache *dst, uint8_t *mask_dev, int32_t *first_bad_page_dev,
                                  uint8_t *group_mask_dev, gk_group_fn on_group, void *user, void *stream, bool host)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0 || n_groups == 0) return GK_OK;
    if (!jobs || !dst || !mask_dev || !first_bad_page_dev)
        return fail(c, GK_ERR_ARG, "null jobs, cache, mask or first_bad_page");
    for (uint32_t j = 0; j < n_jobs; ++j)
        if (jobs[j].n_tokens == 0) return fail(c, GK_ERR_ARG, "job %u: n_tokens == 0", j);
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    int rc_tmp = ensure_group_tmp(c, n_jobs);
    if (rc_tmp != GK_OK) return rc_tmp;
    int32_t *gfb = (int32_t *)c->d_group_tmp;
    uint8_t *gm_own = c->d_group_tmp + align_up((size_t)n_jobs * 4, 256);
    std::vector<gk_job> gj;
    if (!lw_two_streams(c, n_groups, host)) {
        for (uint32_t k = 0; k < n_groups; ++k) {
            const gk_cache view = group_view(c, dst, k);
            group_jobs(c, jobs, n_jobs, k, gj);
            uint8_t *gm = group_mask_dev ? group_mask_dev + (size_t)k * n_jobs : gm_own;
            const int rc = host ? restore_host_impl(c, gj.data(), n_jobs, &view, gm, gfb, stream, k == 0)
                                : gk_restore(c, gj.data(), n_jobs, &view, gm, gfb, stream);
            if (rc != GK_OK) return rc;
            merge_group_kernel<<<(n_jobs + 127) / 128, 128, 0, st>>>(mask_dev, first_bad_page_dev, gm, gfb, n_jobs,
                                                                     k == 0);
            GK_CUDA(c, cudaGetLastError());
            c->stats.kernels_launched++;
            if (on_group)
                on_group(user, k, k * c->gd.layers, c->gd.layers, group_mask_dev ? gm : nullptr, stream);
        }
        return GK_OK;
    }
    // Device tier: group k runs in context k & 1 on stream k & 1 (the groups touch different layers of the cache
    // and different parts of the blobs).  The caller's stream waits for group k, merges its codes into the
    // block-level result and is handed to on_group, in the order of the groups; a context's result arrays are
    // reused by group k + 2 only after the merge of group k has read them.
    int rc = ensure_twin(c);
    if (rc != GK_OK) return rc;
    if ((rc = ensure_group_tmp(c->twin, n_jobs)) != GK_OK) return fail(c, rc, "%s", c->twin->err);
    GK_CUDA(c, cudaEventRecord(c->lw_entry, st));
    for (int i = 0; i < 2; ++i) GK_CUDA(c, cudaStreamWaitEvent(c->lw_stream[i], c->lw_entry, 0));
    for (uint32_t k = 0; k < n_groups; ++k) {
        const uint32_t i = k & 1u;
        gk_ctx *ck = i ? c->twin : c;
        int32_t *gfb_k = (int32_t *)ck->d_group_tmp;
        uint8_t *gm_k = group_mask_dev ? group_mask_dev + (size_t)k * n_jobs
                                       : ck->d_group_tmp + align_up((size_t)n_jobs * 4, 256);
        const gk_cache view = group_view(c, dst, k);
        group_jobs(c, jobs, n_jobs, k, gj);
        if (k >= 2u) GK_CUDA(c, cudaStreamWaitEvent(c->lw_stream[i], c->lw_merged[i], 0));
        rc = gk_restore(ck, gj.data(), n_jobs, &view, gm_k, gfb_k, c->lw_stream[i]);
        if (rc != GK_OK) {
            if (ck != c) fail(c, rc, "%s", ck->err);
            break;
        }
        GK_CUDA(c, cudaEventRecord(c->lw_done[i], c->lw_stream[i]));
        GK_CUDA(c, cudaStreamWaitEvent(st, c->lw_done[i], 0));
        merge_group_kernel<<<(n_jobs + 127) / 128, 128, 0, st>>>(mask_dev, first_bad_page_dev, gm_k, gfb_k, n_jobs,
                                                                 k == 0);
        GK_CUDA(c, cudaGetLastError());
        c->stats.kernels_launched++;
        GK_CUDA(c, cudaEventRecord(c->lw_merged[i], st));
        if (on_group)
            on_group(user, k, k * c->gd.layers, c->gd.layers, group_mask_dev ? gm_k : nullptr, stream);
    }
    if (rc != GK_OK) {  // whatever was enqueued on the two streams still runs: the caller's stream waits for it
        for (int i = 0; i < 2; ++i) {
            cudaEventRecord(c->lw_done[i], c->lw_stream[i]);
            cudaStreamWaitEvent(st, c->lw_done[i], 0);
        }
    }
    return rc;
}

int gk_pack_layerwise(gk_ctx *c, uint32_t n_groups, const gk_cache *src, const gk_job *jobs, uint32_t n_jobs,
                      uint8_t *status_dev, void *stream)
{
    return pack_layerwise_impl(c, n_groups, src, jobs, n_jobs, status_dev, stream, false);
}

int gk_pack_layerwise_host(gk_ctx *c, uint32_t n_groups, const gk_cache *src, const gk_job *jobs, uint32_t n_jobs,
                           uint8_t *status_dev, void *stream)
{
    return pack_layerwise_impl(c, n_groups, src, jobs, n_jobs, status_dev, stream, true);
}

int gk_restore_layerwise(gk_ctx *c, uint32_t n_groups, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst,
                         uint8_t *mask_dev, int32_t *first_bad_page_dev, uint8_t *group_mask_dev, gk_group_fn on_group,
                         void *user, void *stream)
{
    return restore_layerwise_impl(c, n_groups, jobs, n_jobs, dst, mask_dev, first_bad_page_dev, group_mask_dev,
                                  on_group, user, stream, false);
}

int gk_restore_layerwise_host(gk_ctx *c, uint32_t n_groups, const gk_job *jobs, uint32_t n_jobs, const gk_cache *dst,
                              uint8_t *mask_dev, int32_t *first_bad_page_dev, uint8_t *group_mask_dev,
                              gk_group_fn on_group, void *user, void *stream)
{
    return restore_layerwise_impl(c, n_groups, jobs, n_jobs, dst, mask_dev, first_bad_page_dev, group_mask_dev,
                                  on_group, user, stream, true);
}

int gk_fingerprints(gk_ctx *c, const void *data_dev, const uint64_t *offsets_dev, const int32_t *parent, uint32_t n,
                    const uint8_t *model, const uint8_t *tenant, uint8_t *keys_dev, void *stream)
{
    if (!c) return GK_ERR_ARG;
    if (n == 0) return GK_OK;
    if (!offsets_dev || !model || !tenant || !keys_dev) return fail(c, GK_ERR_ARG, "null offsets, model, tenant or keys");
    if ((uintptr_t)keys_dev & 15u) return fail(c, GK_ERR_UNSUPPORTED, "keys must be 16-byte aligned");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    // workspace: [parent n][depth n] | inner n*32
    const size_t meta = align_up((size_t)n * 8, 256);
    int rc = ensure_workspace(c, meta + (size_t)n * 32);
    if (rc != GK_OK) return rc;
    FingerprintParams P{};
    P.data = (const uint8_t *)data_dev;
    P.offsets = offsets_dev;
    P.n = n;
    std::memcpy(P.model, model, 32);
    std::memcpy(P.tenant, tenant, 32);
    P.inner = c->d_ws + meta;
    P.keys = keys_dev;
    if (parent) {
        uint8_t *stage = nullptr;
        cudaEvent_t ev = nullptr;
        if ((rc = next_host_stage(c, (size_t)n * 8, &stage, &ev)) != GK_OK) return rc;
        int32_t *hp = (int32_t *)stage;
        uint32_t *hd = (uint32_t *)(stage + (size_t)n * 4);
        uint32_t max_depth = 0;
        for (uint32_t i = 0; i < n; ++i) {
            if (parent[i] < -1 || (parent[i] >= 0 && (uint32_t)parent[i] >= i))
                return fail(c, GK_ERR_ARG, "parent[%u] = %d: need -1 <= parent[i] < i", i, parent[i]);
            hp[i] = parent[i];
            hd[i] = parent[i] < 0 ? 0u : hd[parent[i]] + 1u;
            if (hd[i] > max_depth) max_depth = hd[i];
        }
        GK_CUDA(c, cudaMemcpyAsync(c->d_ws, stage, (size_t)n * 8, cudaMemcpyHostToDevice, st));
        GK_CUDA(c, cudaEventRecord(ev, st));
        P.parent = (const int32_t *)c->d_ws;
        P.depth = (const uint32_t *)(c->d_ws + (size_t)n * 4);
        P.max_depth = max_depth;
    }
    fingerprint_inner_kernel<<<(n + 63u) / 64u, 64, 0, st>>>(P);
    GK_CUDA(c, cudaGetLastError());
    fingerprint_chain_kernel<<<1, 1024, 0, st>>>(P);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched += 2;
    return GK_OK;
}

int gk_blob_digests(gk_ctx *c, const gk_job *jobs, uint32_t n_jobs, const uint8_t *keys_dev, uint8_t *digests_dev,
                    uint8_t *page_digests_dev, void *stream)
{
    if (!c) return GK_ERR_ARG;
    if (n_jobs == 0) return GK_OK;
    if (!jobs || !keys_dev || !digests_dev) return fail(c, GK_ERR_ARG, "null jobs, keys or digests");
    if (((uintptr_t)digests_dev | (uintptr_t)page_digests_dev) & 15u)
        return fail(c, GK_ERR_UNSUPPORTED, "digest arrays must be 16-byte aligned");
    for (uint32_t j = 0; j < n_jobs; ++j)
        if (!jobs[j].blob) return fail(c, GK_ERR_ARG, "job %u: null blob", j);
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    uint64_t pages = 0;
    for (uint32_t j = 0; j < n_jobs; ++j) {
        if (jobs[j].n_tokens == 0) return fail(c, GK_ERR_ARG, "job %u: n_tokens == 0", j);
        pages += pages_of(jobs[j].n_tokens, c->gd.page_tokens);
    }
    if (pages > 0x7fffffffull) return fail(c, GK_ERR_ARG, "too many pages in one call");
    const uint32_t m_max = (uint32_t)((c->gd.R + kDigestChunk - 1) / kDigestChunk);
    // workspace: job table | leaves | page digests (unless the caller wants them)
    WsLayout l{};
    l.jobs = 0;
    const size_t o_leaves = align_up((size_t)n_jobs * sizeof(JobDev), 256);
    const size_t o_pages = align_up(o_leaves + (size_t)pages * m_max * 32, 256);
    int rc = ensure_workspace(c, o_pages + (size_t)pages * 32);
    if (rc != GK_OK) return rc;
    Tiling none{};
    uint64_t bytes = 0;
    if ((rc = upload_jobs(c, jobs, n_jobs, l, none, nullptr, nullptr, false, st, &pages, &bytes)) != GK_OK) return rc;
    DigestParams P{};
    P.g = c->gd;
    P.jobs = (const JobDev *)c->d_ws;
    P.n_jobs = n_jobs;
    P.total_pages = (uint32_t)pages;
    P.m_max = m_max;
    P.leaves = c->d_ws + o_leaves;
    P.page_digests = page_digests_dev ? page_digests_dev : c->d_ws + o_pages;
    P.keys = keys_dev;
    P.digests = digests_dev;
    const uint64_t leaf_threads = pages * m_max;
    sha_leaf_kernel<<<(unsigned)((leaf_threads + 127) / 128), 128, 0, st>>>(P);
    GK_CUDA(c, cudaGetLastError());
    sha_page_kernel<<<(unsigned)((pages + 63) / 64), 64, 0, st>>>(P);
    GK_CUDA(c, cudaGetLastError());
    sha_blob_kernel<<<(n_jobs + 63u) / 64u, 64, 0, st>>>(P);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched += 3;
    return GK_OK;
}

int gk_get_kernel_times(gk_ctx *c, double ms[4], uint64_t launches[4])
{
    if (!c || !ms || !launches) return GK_ERR_ARG;
    DeviceGuard guard(c->device);
    for (size_t i = 0; i < c->prof_used; ++i) {
        gk_ctx::ProfSlot &ps = c->prof_pool[i];
        GK_CUDA(c, cudaEventSynchronize(ps.b));
        float t = 0.f;
        GK_CUDA(c, cudaEventElapsedTime(&t, ps.a, ps.b));
        c->prof_ms[ps.cls] += t;
        c->prof_launches[ps.cls]++;
    }
    c->prof_used = 0;
    for (int i = 0; i < 4; ++i) {
        ms[i] = c->prof_ms[i];
        launches[i] = c->prof_launches[i];
        c->prof_ms[i] = 0;
        c->prof_launches[i] = 0;
    }
    return GK_OK;
}

}  // extern "C"

namespace {
// Measurement aid: every thread runs `iters` rounds of 16 independent three-input logic
// operations (the instruction the checksum kernels are made of), enough warps per SM to fill
// the pipe; the result is stored so that nothing is optimised away.
__global__ void __launch_bounds__(256) logic_rate_kernel(uint32_t *sink, uint32_t iters, uint32_t seed)
{
    uint32_t r[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) r[i] = seed * (uint32_t)(i + 1) + threadIdx.x;
    for (uint32_t k = 0; k < iters; ++k) {
#pragma unroll
        for (int i = 0; i < 16; ++i)
            asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(r[i]) : "r"(r[(i + 5) & 15]), "r"(k));
    }
    uint32_t acc = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) acc ^= r[i];
    sink[blockIdx.x * blockDim.x + threadIdx.x] = acc;
}
}  // namespace

extern "C" {

int gk_measure_logic_rate(gk_ctx *c, double *lane_ops_per_second, void *stream)
{
    if (!c || !lane_ops_per_second) return GK_ERR_ARG;
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t grid = (uint32_t)c->sm_count * 8u, threads = 256u, iters = 1u << 14;
    int rc = ensure_workspace(c, (size_t)grid * threads * 4);
    if (rc != GK_OK) return rc;
    cudaEvent_t e0, e1;
    GK_CUDA(c, cudaEventCreate(&e0));
    GK_CUDA(c, cudaEventCreate(&e1));
    float best = 0.f;
    for (int rep = 0; rep < 4; ++rep) {  // the first launch warms up
        cudaEventRecord(e0, st);
        logic_rate_kernel<<<grid, threads, 0, st>>>(reinterpret_cast<uint32_t *>(c->d_ws), iters, 12345u + rep);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess) break;
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (rep > 0 && (best == 0.f || ms < best)) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    GK_CUDA(c, cudaGetLastError());
    c->stats.kernels_launched += 4;
    if (best <= 0.f) return fail(c, GK_ERR_CUDA, "logic rate measurement failed");
    *lane_ops_per_second = (double)grid * threads * iters * 16.0 / (best * 1e-3);
    return GK_OK;
}

int gk_debug_range_ok(uint64_t addr, uint64_t bytes, uint64_t base, uint64_t extent)
{
    return range_inside(addr, bytes, base, extent) ? 1 : 0;
}

int gk_debug_status(gk_ctx *c, uint32_t out[4])
{
    if (!c || !out) return GK_ERR_ARG;
#ifdef GK_DEBUG
    DeviceGuard guard(c->device);
    GK_CUDA(c, cudaMemcpy(out, c->d_error + 8, 16, cudaMemcpyDeviceToHost));
    if (out[0] == 0u && c->twin) GK_CUDA(c, cudaMemcpy(out, c->twin->d_error + 8, 16, cudaMemcpyDeviceToHost));
    return GK_OK;
#else
    out[0] = out[1] = out[2] = out[3] = 0u;
    return fail(c, GK_ERR_UNSUPPORTED, "this library was built without GK_DEBUG");
#endif
}

int gk_get_stats(gk_ctx *c, gk_stats *out)
{
    if (!c || !out) return GK_ERR_ARG;
    DeviceGuard guard(c->device);
    uint32_t e = 0;
    GK_CUDA(c, cudaMemcpy(&e, c->d_error, 4, cudaMemcpyDeviceToHost));
    c->stats.device_wait_expired = e;
    *out = c->stats;
    if (c->twin) {  // what the twin did counts as this context's own (its calls are counted here, not there)
        gk_stats t{};
        const int rc = gk_get_stats(c->twin, &t);
        if (rc != GK_OK) return rc;
        out->calls_pack += t.calls_pack;
        out->calls_restore += t.calls_restore;
        out->jobs += t.jobs;
        out->pages += t.pages;
        out->bytes_blob += t.bytes_blob;
        out->kernels_launched += t.kernels_launched;
        out->quartet_launches += t.quartet_launches;
        out->allocations += t.allocations;
        if (out->device_wait_expired == 0) out->device_wait_expired = t.device_wait_expired;
    }
    return GK_OK;
}

// ---------------------------------------------------------------------------
// gk_page_checksums_noalloc: page checksums without any allocation.
//
// Same kernels as gk_page_checksums (verify-mode streaming kernel, then the
// checksum-writing finalize kernel), but every byte of scratch -- job record,
// page map, per-page remainders, result words, the GF(2) tables -- lives in
// the file-scope device array below instead of a context's workspace.
// ---------------------------------------------------------------------------
}  // extern "C"

namespace {

constexpr uint32_t kNoallocMaxPages = GK_NOALLOC_MAX_PAGES;
constexpr uint32_t kNoallocMaxPageTokens = GK_NOALLOC_MAX_PAGE_TOKENS;

// Layout of the static scratch (all offsets multiples of 256 bytes).
struct NoallocLayout {
    static constexpr size_t job = 0;                                        // JobDev
    static constexpr size_t words = 256;                                    // bad_range, bad_dup, bad_crc, job_done, error
    static constexpr size_t thread_const = 512;                             // [GK_CRC_NT] u64
    static constexpr size_t init_term = thread_const + 8 * 256;             // [max page tokens + 1] u64
    static constexpr size_t page_job = init_term + 8 * (kNoallocMaxPageTokens + 1) + 248;  // [max pages] i32
    static constexpr size_t page_cnt = page_job + 4 * (size_t)kNoallocMaxPages;            // [max pages] u32
    static constexpr size_t page_acc = page_cnt + 4 * (size_t)kNoallocMaxPages;            // [max pages] u64
    static constexpr size_t total = page_acc + 8 * (size_t)kNoallocMaxPages;
};
static_assert(GK_CRC_NT + 2 * (GK_CRC_NT / 32) <= 256, "thread constant table");
static_assert(NoallocLayout::page_job % 256 == 0 && NoallocLayout::page_acc % 8 == 0, "scratch alignment");

// The scratch itself: about 133 KiB per GPU that loads the library, held until exit.
// In host code this name is only a stand-in for the symbol; the device address
// comes from cudaGetSymbolAddress (noalloc_setup below).
static __device__ __align__(256) unsigned char g_noalloc_scratch[NoallocLayout::total];

__device__ uint64_t dev_xpow(uint64_t n)
{
    uint64_t r = 1, base = 2;
    while (n) {
        if (n & 1ull) r = gf_mul(r, base);
        base = gf_mul(base, base);
        n >>= 1;
    }
    return r;
}

// One CTA.  Writes the job record and the tables into the scratch and resets
// every word that has to start from a known value; the array keeps whatever the
// previous call left behind.
__global__ void noalloc_setup_kernel(unsigned char *scratch, JobDev job, GeomDev g)
{
    JobDev *jd = reinterpret_cast<JobDev *>(scratch + NoallocLayout::job);
    int32_t *words = reinterpret_cast<int32_t *>(scratch + NoallocLayout::words);
    uint64_t *tc = reinterpret_cast<uint64_t *>(scratch + NoallocLayout::thread_const);
    uint64_t *it = reinterpret_cast<uint64_t *>(scratch + NoallocLayout::init_term);
    int32_t *page_job = reinterpret_cast<int32_t *>(scratch + NoallocLayout::page_job);
    uint32_t *page_cnt = reinterpret_cast<uint32_t *>(scratch + NoallocLayout::page_cnt);
    uint64_t *page_acc = reinterpret_cast<uint64_t *>(scratch + NoallocLayout::page_acc);
    if (threadIdx.x == 0) {
        *jd = job;
        words[0] = kNoPage;  // bad_range
        words[1] = kNoPage;  // bad_dup
        words[2] = kNoPage;  // bad_crc
        words[3] = 0;        // job_done
        words[4] = 0;        // error word
        words[5] = 0;        // work counters
        words[6] = 0;
        words[7] = 0;        // the error word as this call found it
        words[12] = 0;       // the bounds-checked build's record of a refused access
    }
    for (uint32_t t = threadIdx.x; t < (uint32_t)GK_CRC_NT; t += blockDim.x)
        tc[t] = dev_xpow(32ull * (GK_CRC_NT - 1 - t) + 64ull);
    for (uint32_t k = threadIdx.x; k < 2u * (GK_CRC_NT / 32); k += blockDim.x)  // the words above each warp
        tc[GK_CRC_NT + k] = dev_xpow(1024ull * (GK_CRC_NT / 32 - k / 2u) + 64ull + 32ull * (k & 1u));
    for (uint32_t t = threadIdx.x; t <= g.page_tokens; t += blockDim.x)
        it[t] = t ? gf_mul(~0ull, dev_xpow(8ull * (g.S + (uint64_t)t * g.tokB))) : 0ull;
    for (uint32_t p = threadIdx.x; p < job.n_pages; p += blockDim.x) {
        page_job[p] = 0;
        page_cnt[p] = 0u;
        page_acc[p] = 0ull;
    }
}

struct NoallocDevice {
    unsigned char *scratch = nullptr;
    int sm_count = 0;
    int occ = 0;
    bool ready = false;
};
NoallocDevice g_noalloc_dev[64];
std::mutex g_noalloc_mutex;

// Once per device, with that device current: resolve the scratch array's device
// address and prepare the kernel for its dynamic shared memory size.
int noalloc_setup(int device, NoallocDevice **out)
{
    if (device < 0 || device >= 64) return GK_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoallocDevice &d = g_noalloc_dev[device];
    if (!d.ready) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return GK_ERR_CUDA;
        }
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
            cudaGetLastError();
            return GK_ERR_CUDA;
        }
        if (major != 10) return GK_ERR_UNSUPPORTED;
        auto *kv = stream_kernel<kVerify, GK_CRC_NT, GK_CRC_STAGE, GK_CRC_STAGES, GK_VERIFY_MINB>;
        if (cudaFuncSetAttribute(kv, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)VerifyCfg::kSmemBytes) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&d.occ, kv, VerifyCfg::kThreads, VerifyCfg::kSmemBytes) != cudaSuccess ||
            d.occ < 1) {
            cudaGetLastError();
            return GK_ERR_CUDA;
        }
        d.scratch = static_cast<unsigned char *>(ptr);
        d.ready = true;
    }
    *out = &d;
    return GK_OK;
}

}  // namespace

extern "C" {

int gk_page_checksums_noalloc(const gk_geom *geom, const void *blob_dev, uint32_t n_tokens, uint64_t *checksums_dev,
                              int device, void *stream)
{
    GeomDev gd;
    int rc = check_geom(geom, &gd);
    if (rc != GK_OK) return rc;
    if (!blob_dev || !checksums_dev || n_tokens == 0) return GK_ERR_ARG;
    if (((uintptr_t)blob_dev & 15u) || ((uintptr_t)checksums_dev & 7u)) return GK_ERR_UNSUPPORTED;
    const uint64_t pages = ((uint64_t)n_tokens + gd.page_tokens - 1) / gd.page_tokens;
    if (pages > kNoallocMaxPages || gd.page_tokens > kNoallocMaxPageTokens) return GK_ERR_TOO_LARGE;

    DeviceGuard guard(device);
    NoallocDevice *nd = nullptr;
    if ((rc = noalloc_setup(device, &nd)) != GK_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char *sc = nd->scratch;

    // one segment per page: the scratch holds one remainder per page
    Tiling tl;
    tl.stage_bytes = GK_CRC_STAGE;
    tl.gran_bytes = VerifyCfg::kGran;
    const uint32_t gran_full = (uint32_t)((gd.R + tl.gran_bytes - 1) / tl.gran_bytes);
    tl.seg_tiles = gran_full * VerifyCfg::kTilesPerGran;
    tl.nseg_max = 1;

    JobDev job{};
    job.blob = (uint8_t *)const_cast<void *>(blob_dev);
    job.checksums = checksums_dev;
    job.page_table = nullptr;
    job.n_tokens = n_tokens;
    job.n_pages = (uint32_t)pages;
    job.page_base = 0;
    job.missing = 0;

    int32_t *words = reinterpret_cast<int32_t *>(sc + NoallocLayout::words);
    WorkDev w{};
    w.jobs = reinterpret_cast<const JobDev *>(sc + NoallocLayout::job);
    w.n_jobs = 1;
    w.page_begin = 0;
    w.total_pages = (uint32_t)pages;
    w.page_job = reinterpret_cast<int32_t *>(sc + NoallocLayout::page_job);
    w.page_acc = reinterpret_cast<uint64_t *>(sc + NoallocLayout::page_acc);
    w.bad_range = words + 0;
    w.bad_dup = words + 1;
    w.bad_crc = words + 2;
    w.page_cnt = reinterpret_cast<uint32_t *>(sc + NoallocLayout::page_cnt);
    w.job_done = reinterpret_cast<uint32_t *>(words + 3);
    w.claims = nullptr;
    w.error = reinterpret_cast<uint32_t *>(words + 4);
    w.work_ctr = reinterpret_cast<uint32_t *>(words + 5);
    w.init_term = reinterpret_cast<const uint64_t *>(sc + NoallocLayout::init_term);
    w.thread_const = reinterpret_cast<const uint64_t *>(sc + NoallocLayout::thread_const);
    w.wait_limit_ns = kWaitLimitNs;

    noalloc_setup_kernel<<<1, 256, 0, st>>>(sc, job, gd);
    if (cudaGetLastError() != cudaSuccess) return GK_ERR_CUDA;
    StreamParams P{};
    P.g = gd;
    P.w = w;
    P.tl = tl;
    P.n_items = (uint32_t)pages;
    uint32_t grid = (uint32_t)(nd->sm_count * nd->occ);
    if (grid > P.n_items) grid = P.n_items;
    stream_kernel<kVerify, GK_CRC_NT, GK_CRC_STAGE, GK_CRC_STAGES, GK_VERIFY_MINB>
        <<<grid, VerifyCfg::kThreads, VerifyCfg::kSmemBytes, st>>>(P);
    if (cudaGetLastError() != cudaSuccess) return GK_ERR_CUDA;
    finalize_kernel<<<(uint32_t)((pages + 127) / 128), 128, 0, st>>>(gd, w, tl, 1, nullptr);
    if (cudaGetLastError() != cudaSuccess) return GK_ERR_CUDA;
    return GK_OK;
}

}  // extern "C"
