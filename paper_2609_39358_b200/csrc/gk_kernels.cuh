// gk_kernels.cuh -- the kernels of libgk (sm_100a).
//
//   validate_kernel   page ids in range, missing records, page -> job map
//   claim_kernel      a destination page may be claimed once per call
//   prep_small_kernel both of the above plus the job table, in one launch (small calls)
//   stream_kernel<>   one warp-specialised streaming kernel in three modes:
//                       kVerify : blob -> smem -> CRC segment remainders
//                       kPack   : cache slabs -> smem -> CRC + blob
//                       kCommit : blob -> smem -> cache slabs (no CRC)
//                       kSingle : blob -> smem -> CRC + cache slabs (single-pass restore:
//                                 a block that fails only its checksum is reported, but
//                                 its own pages have received the unverified bytes)
//   restore_kernel<>  verify and commit pipelines side by side in one CTA; a job is
//                     committed only after all of its pages have verified
//   finalize_kernel   page accumulators -> page CRC-64/XZ; compare or write
//   report_kernel     result codes of a verify-only call
//
// Every role of a streaming CTA is one of: loader warp (draws work items from a
// global counter, fills ring stages with bulk async copies, tags them), consumer
// warps (CRC), storer warp (bulk async copies out).  All waits are bounded.
//
// The CRC is computed bit-sliced: a thread reads the words t, t+NT, t+2NT, ...
// of a segment, and each of the 32 bit positions of those words is treated as
// an independent bit stream (stride 32*NT bits, a power of two).  64 registers
// hold the 64 remainder coefficients of the 32 streams, so one step of the
// shift register costs a handful of 32-wide XORs.  Because squaring is linear
// over GF(2), a stream M(x^(2^e)) has remainder (M(x) mod P)^(2^e) mod P: the
// streams are reduced with the plain shift register and the 2^e-th power map,
// a fixed 64x64 bit matrix, is applied once per thread per segment.  The
// streams of a thread, the threads of a CTA and the segments of a page are then
// merged by multiplying each remainder by x^(distance to the end) mod P.
#pragma once

#include "gk_device.cuh"
#include "gk_gf2_generated.inc"

namespace gk {

// ---------------------------------------------------------------------------
// small kernels
// ---------------------------------------------------------------------------
// ids[i] = i: the page ids from which the streaming restore cuts its window page tables
__global__ void iota_kernel(int32_t *ids, uint32_t n)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) ids[i] = (int32_t)i;
}

// Layer-wise restore: folds the codes of one layer group into the block-level result.
// mask = largest code so far; first_bad = the page reported by the lowest failing group.
__global__ void merge_group_kernel(uint8_t *mask, int32_t *first_bad, const uint8_t *group_mask,
                                   const int32_t *group_first_bad, uint32_t n_jobs, int first_group)
{
    const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n_jobs) return;
    const uint8_t gm = group_mask[j];
    const uint8_t m = first_group ? (uint8_t)0 : mask[j];
    if (first_group) first_bad[j] = -1;
    if (m == 0 && gm != 0) first_bad[j] = group_first_bad[j];
    mask[j] = gm > m ? gm : m;
}

// Job table and segment powers of a call of at most kPrepMaxJobs jobs, as kernel arguments.
constexpr uint32_t kPrepMaxJobs = 64;
constexpr uint32_t kPrepMaxSeg = 64;
struct PrepSmallParams {
    JobDev jobs[kPrepMaxJobs];
    uint64_t seg_pow[2 * kPrepMaxSeg];
    uint32_t n_seg_pow;
    uint32_t do_claims;
    uint64_t num_pages;
    uint8_t *status_out;  // save calls: 0 or 2 per job; else null
};

// One CTA per job.  Initialises the job's result words, records the lowest
// out-of-range page id and fills page_job.  All CTAs together clear the claim
// words of the destination cache.
// ARGS: the job table (at most kPrepMaxJobs jobs) and the segment powers travel as kernel arguments -- no
// staging copy in front of the call; block 0 leaves them in the workspace for the kernels that follow.
template <bool ARGS>
__device__ __forceinline__ void validate_body(const PrepSmallParams *pp, const WorkDev &w, uint64_t num_pages,
                                              int clear_claims, uint8_t *status_out)
{
    allow_dependent_launch();  // the kernel directly behind this one may set itself up meanwhile
    const uint32_t j = blockIdx.x;
    if (ARGS && blockIdx.x == 0) {
        JobDev *jobs_out = const_cast<JobDev *>(w.jobs);
        uint64_t *pow_out = const_cast<uint64_t *>(w.seg_pow);
        for (uint32_t k = threadIdx.x; k < w.n_jobs; k += blockDim.x) jobs_out[k] = pp->jobs[k];
        for (uint32_t k = threadIdx.x; k < pp->n_seg_pow; k += blockDim.x) pow_out[k] = pp->seg_pow[k];
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        // every call draws its work items from zero (the host counts the draws of its launches)
        w.work_ctr[0] = 0u;
        w.work_ctr[1] = 0u;
        w.work_ctr[2] = *w.error;  // what earlier calls left: a set word refuses every commit of this call
    }
    if (clear_claims) {
        for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < num_pages;
             i += (uint64_t)gridDim.x * blockDim.x)
            w.claims[i] = 0ull;
    }
    if (j >= w.n_jobs) return;
    const JobDev jb = ARGS ? pp->jobs[j] : w.jobs[j];
    __shared__ int32_t s_bad;
    if (threadIdx.x == 0) s_bad = kNoPage;
    __syncthreads();
    int32_t bad = kNoPage;
#pragma unroll 4
    for (uint32_t p = threadIdx.x; p < jb.n_pages; p += blockDim.x) {
        w.page_job[jb.page_base + p] = (int32_t)j;
        w.page_cnt[jb.page_base + p] = 0u;
        w.page_acc[jb.page_base + p] = 0ull;
        if (jb.page_table) {
            const int32_t id = jb.page_table[p];
            if ((id < 0 || (uint64_t)id >= num_pages) && (int32_t)p < bad) bad = (int32_t)p;
        }
    }
    if (bad != kNoPage) atomicMin(&s_bad, bad);
    __syncthreads();
    if (threadIdx.x == 0) {
        w.bad_range[j] = s_bad;
        if (status_out) status_out[j] = s_bad != kNoPage ? 2u : 0u;  // save: the only thing that can fail
        w.bad_dup[j] = kNoPage;
        w.bad_crc[j] = kNoPage;
        w.job_done[j] = 0u;
        w.job_latch[j] = kUndecided;
    }
}

__global__ void validate_kernel(WorkDev w, uint64_t num_pages, int clear_claims, uint8_t *status_out)
{
    validate_body<false>(nullptr, w, num_pages, clear_claims, status_out);
}

__global__ void validate_args_kernel(const __grid_constant__ PrepSmallParams pp, WorkDev w, uint64_t num_pages,
                                     int clear_claims, uint8_t *status_out)
{
    validate_body<true>(&pp, w, num_pages, clear_claims, status_out);
}

// One thread per page of the call.  The first job to claim a destination page
// leaves (job+1, index) in its claim word; every later claimant marks itself
// and that first claimant.  Jobs that are missing or already failed the range
// check claim nothing.
__global__ void claim_kernel(WorkDev w)
{
    allow_dependent_launch();  // the streaming kernel behind this one may set up its rings meanwhile
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= w.total_pages) return;
    const uint32_t j = (uint32_t)w.page_job[g];
    const JobDev jb = w.jobs[j];
    if (jb.missing || w.bad_range[j] != kNoPage) return;
    const uint32_t p = g - jb.page_base;
    const int32_t id = jb.page_table[p];
    const unsigned long long mine = ((unsigned long long)(j + 1u) << 32) | p;
    const unsigned long long old = atomicCAS(&w.claims[id], 0ull, mine);
    if (old != 0ull) {
        atomicMin(&w.bad_dup[j], (int32_t)p);
        atomicMin(&w.bad_dup[(uint32_t)(old >> 32) - 1u], (int32_t)(old & 0xffffffffull));
    }
}

// Small calls: the whole preparation in ONE single-CTA launch, with the job table
// and the segment powers passed as kernel arguments instead of a host-to-device
// copy.  Writes the tables to the workspace, then does what validate_kernel and
// claim_kernel do, separated by a CTA barrier.  Only the claim words that this
// call can touch are cleared.
__global__ void __launch_bounds__(1024) prep_small_kernel(const __grid_constant__ PrepSmallParams pp, WorkDev w)
{
    allow_dependent_launch();  // the streaming kernel behind this one may set up its rings meanwhile
    JobDev *jobs_out = const_cast<JobDev *>(w.jobs);
    uint64_t *pow_out = const_cast<uint64_t *>(w.seg_pow);
    for (uint32_t j = threadIdx.x; j < w.n_jobs; j += blockDim.x) {
        jobs_out[j] = pp.jobs[j];
        w.bad_range[j] = kNoPage;
        w.bad_dup[j] = kNoPage;
        w.bad_crc[j] = kNoPage;
        w.job_done[j] = 0u;
        w.job_latch[j] = kUndecided;
    }
    for (uint32_t k = threadIdx.x; k < pp.n_seg_pow; k += blockDim.x) pow_out[k] = pp.seg_pow[k];
    if (threadIdx.x == 0) {
        w.work_ctr[0] = 0u;  // every call draws its work items from zero
        w.work_ctr[1] = 0u;
        w.work_ctr[2] = *w.error;  // what earlier calls left: a set word refuses every commit of this call
    }
    __syncthreads();
    // Both passes run over the pages of the whole call at once (a thread finds the job of its
    // page by bisection), so that the loads of all page tables are in flight together.
    const uint32_t total_pages = pp.jobs[w.n_jobs - 1u].page_base + pp.jobs[w.n_jobs - 1u].n_pages;
    auto job_of = [&](uint32_t gp) {
        uint32_t lo = 0, hi = w.n_jobs - 1u;
        while (lo < hi) {
            const uint32_t mid = (lo + hi + 1u) >> 1;
            if (pp.jobs[mid].page_base <= gp) lo = mid; else hi = mid - 1u;
        }
        return lo;
    };
    // pass 1: page -> job map, range check, clear the claim words that will be used
    for (uint32_t gp = threadIdx.x; gp < total_pages; gp += blockDim.x) {
        const uint32_t j = job_of(gp);
        const JobDev &jb = pp.jobs[j];
        const uint32_t p = gp - jb.page_base;
        w.page_job[gp] = (int32_t)j;
        w.page_cnt[gp] = 0u;
        w.page_acc[gp] = 0ull;
        if (jb.page_table) {
            const int32_t id = jb.page_table[p];
            if (id < 0 || (uint64_t)id >= pp.num_pages)
                atomicMin(&w.bad_range[j], (int32_t)p);
            else if (pp.do_claims)
                w.claims[id] = 0ull;
        }
    }
    if (pp.status_out) {
        __syncthreads();
        for (uint32_t j = threadIdx.x; j < w.n_jobs; j += blockDim.x)
            pp.status_out[j] = __ldcg(&w.bad_range[j]) != kNoPage ? 2u : 0u;
    }
    if (!pp.do_claims) return;
    __syncthreads();
    // pass 2: claims, as in claim_kernel
    for (uint32_t gp = threadIdx.x; gp < total_pages; gp += blockDim.x) {
        const uint32_t j = job_of(gp);
        const JobDev &jb = pp.jobs[j];
        if (jb.missing || __ldcg(&w.bad_range[j]) != kNoPage) continue;
        const uint32_t p = gp - jb.page_base;
        const int32_t id = jb.page_table[p];
        const unsigned long long mine = ((unsigned long long)(j + 1u) << 32) | p;
        const unsigned long long old = atomicCAS(&w.claims[id], 0ull, mine);
        if (old != 0ull) {
            atomicMin(&w.bad_dup[j], (int32_t)p);
            atomicMin(&w.bad_dup[(uint32_t)(old >> 32) - 1u], (int32_t)(old & 0xffffffffull));
        }
    }
}

// Result code of a job from the words the earlier kernels left.  Precedence:
// missing (3) > page table (2) > checksum (1) > a wait ran out (4) > ok (0).
// `verified` says that every page of the job is known to have been checked: in
// the fused kernel the caller has seen the job's page count in job_done (so a
// wait that ran out elsewhere in the same launch does not taint this job, only
// an error word that was already set when the call began does); in the kernels
// that run after a separate verify launch the live error word speaks for it.
__device__ __forceinline__ uint32_t job_code(const WorkDev &w, uint32_t j, int32_t *first_bad, bool fused,
                                             bool verified)
{
    *first_bad = -1;
    if (w.jobs[j].missing) return 3u;
    int32_t r = w.bad_range[j];
    if (r == kNoPage) r = w.bad_dup[j];
    if (r != kNoPage) {
        *first_bad = r;
        return 2u;
    }
    // written by other CTAs of the same launch in the fused kernel: read at L2
    r = __ldcg(&w.bad_crc[j]);
    if (r != kNoPage) {
        *first_bad = r;
        return 1u;
    }
    if (!verified) return 4u;
    if (__ldcg(fused ? &w.work_ctr[2] : w.error) != 0u) return 4u;
    if (w.ext_mask) return (uint32_t)w.ext_mask[j];  // verified elsewhere (another call, another rank)
    return 0u;
}

// One thread per job: result code and first failing page (gk_verify, which commits nothing).
__global__ void report_kernel(WorkDev w, uint8_t *mask_out, int32_t *first_bad_out)
{
    const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= w.n_jobs) return;
    int32_t fb;
    const uint32_t code = job_code(w, j, &fb, false, true);
    mask_out[j] = (uint8_t)code;
    first_bad_out[j] = fb;
}

// One thread per page.  The page's segment remainders have been XORed into
// page_acc by the CTAs that produced them (each already multiplied by
// x^(8 * bytes that follow the segment)); this adds the term of the all-ones
// initial register and the final xor, reflects, and either writes the checksum
// (write_mode) or compares it with the stored one.
__global__ void finalize_kernel(GeomDev g, WorkDev w, Tiling tl, int write_mode, uint8_t *status_out)
{
    const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= w.total_pages) return;
    const uint32_t gp = w.page_begin + idx;
    const uint32_t j = (uint32_t)w.page_job[gp];
    const JobDev jb = w.jobs[j];
    const uint32_t p = gp - jb.page_base;
    const bool bad_table = w.bad_range[j] != kNoPage;
    if (write_mode && p == 0u && status_out) status_out[j] = bad_table ? 2u : 0u;
    if (jb.missing || bad_table) return;
    if (!write_mode && w.bad_dup[j] != kNoPage) return;
    // after a wait that ran out some segments never arrived: write nothing that looks like a checksum
    if (*w.error != 0u) return;
    const PageShape sh = page_shape(g, jb, p, tl);
    const uint64_t crc = __brevll(w.page_acc[gp] ^ w.init_term[sh.t] ^ ~0ull);
    if (write_mode) {
        jb.checksums[p] = crc;
    } else if (crc != jb.checksums[p]) {
        atomicMin(&w.bad_crc[j], (int32_t)p);
    }
}

// ---------------------------------------------------------------------------
// the streaming kernels
// ---------------------------------------------------------------------------
// What the roles of a CTA need to know about a work item.  The loader works it
// out once and leaves it in shared memory; the other roles read it from there.
struct Item {
    uint8_t *rec;    // first byte of the page record in the job's blob
    uint64_t *sum;   // the record's checksum word
    uint32_t j, p, q;
    uint32_t gp;     // page index within the call
    uint32_t pad;
    uint32_t tile_begin, tile_count;
    uint32_t t;
    uint32_t nseg;
    int32_t phys;
};

// Page quartets: what the roles of a CTA need to know about an item of four
// pages, one per consumer warp, in the place of an Item.  Everything else about
// a page follows from (job, page) and the tables of the call.
struct QuadPages {
    uint32_t j[4];  // owning job of each page, or kNoJob: this warp's result is dropped
    uint32_t p[4];  // page index within the job
};
struct QuadItem {
    uint32_t tile_count;  // tiles of the quartet (those of its longest record)
    uint32_t reserved;
    QuadPages pages;
};
static_assert(sizeof(QuadItem) <= sizeof(Item), "a quartet must fit an item slot");
static_assert(sizeof(QuadPages) == 32, "the quartet's pages take the item copy's place in a hand-over slot");

template <int MODE, int NT, int STAGE_BYTES, int STAGES>
struct StreamCfg {
    static constexpr bool kCrc = (MODE != kCommit);
    static constexpr bool kStore = (MODE != kVerify);
    static constexpr int kConsWarps = kCrc ? NT / 32 : 0;
    static constexpr int kLoaderWarp = kConsWarps;
    static constexpr int kStorerWarp = kConsWarps + 1;
    static constexpr bool kOwnFinisher = kCrc && !kStore;   // else the storer warp finishes the segments
    static constexpr int kFinisherWarp = kConsWarps + 1;    // where it is a warp of its own
    static constexpr int kThreads = 32 * (kConsWarps + 1 + (kStore ? 1 : 0) + (kOwnFinisher ? 1 : 0));
    static constexpr int kGran = kCrc ? NT * 256 : STAGE_BYTES;  // 8 shift-register steps of 8 words per thread
    static constexpr int kSps = kCrc ? STAGE_BYTES / (NT * 32) : 1;  // 8-word steps per stage
    static constexpr int kTilesPerGran = kGran / STAGE_BYTES;
    // stages | full and empty barriers | tags | item slots | reduction slots [2][8] | abort flag | alignment slack
    static constexpr size_t kSmemBytes =
        (size_t)STAGES * STAGE_BYTES + 3 * STAGES * 8 + (STAGES + 1) * sizeof(Item) + 2 * 12 * 8 + 4 * 8 + 16 + 16;
    static_assert(!kCrc || (NT == 32 || NT == 64 || NT == 128 || NT == 256), "NT must be a power of two");
    static_assert(!kCrc || (STAGE_BYTES % (NT * 32) == 0 && (NT * 256) % STAGE_BYTES == 0), "stage/step mismatch");
    static_assert(STAGE_BYTES % 128 == 0, "stage alignment");
};

struct StreamParams {
    GeomDev g;
    CacheDev cache;   // kPack: source cache; kCommit / restore: destination cache; kVerify: unused
    WorkDev w;
    Tiling tl;        // tiling of the CRC modes (verify, pack)
    Tiling tlc;       // tiling of the commit mode
    uint32_t n_items;    // CRC work items: pages of the launch * tl.nseg_max (page quartets: a quarter of the pages)
    uint32_t n_items_c;  // commit work items: pages of the launch * tlc.nseg_max
    uint32_t fused;      // 1: verify and commit run in one launch; commit waits per job
    uint32_t inline_final;  // 1: the CTA that delivers a page's last segment finalizes the page itself
    uint32_t ctr_base_v, ctr_base_c;  // values of the work counters at the start of this launch
    uint32_t commit_reverse;  // 1: the commit side walks the pages of a job from the last to the first
    uint32_t l2_hints;        // bit 0: verify loads evict_last; bit 1: commit loads evict_first; bit 2: commit stores evict_first
    uint32_t test_drop_from;  // tests only: k > 0 makes the fused kernel verify nothing of jobs k-1, k, ...
    unsigned long long *trace;  // builds with GK_TRACE: time stamps of the first item of every role, else null
    uint8_t *mask_out;        // commit
    int32_t *first_bad_out;   // commit
};

// A shared-memory ring of STAGES tiles with a full and an empty barrier each.
// An item's description lives in one of STAGES + 1 slots: the loader is never
// more than STAGES items ahead of a role that still reads the slot of its item.
struct Ring {
    uint8_t *base;    // generic address of stage 0
    uint32_t stage0;  // shared-window address of stage 0
    uint32_t full0, empty0;
    uint2 *tag;   // per stage: (item slot, tile index within the item), or the end mark
    Item *items;  // [STAGES + 1]
    // CRC rings: hand-over of a reduced segment from the consumer warps to the finisher warp
    // (see finisher_role).  Two hand-over slots, used in turn.
    uint64_t *red;   // [2][kHandOverWords]
    uint32_t tail0;  // four barriers: slot 0 posted, slot 1 posted, slot 0 taken, slot 1 taken
};

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint64_t ld_acquire_u64(const uint64_t *p)
{
    uint64_t v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void red_xor_u64(uint64_t *p, uint64_t v)
{
    asm volatile("red.relaxed.gpu.global.xor.b64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Counts one arrival; everything this thread wrote before (the red.xor above it)
// is visible to whoever sees the count, and the returned count lets the last
// arriver see what the others wrote.
__device__ __forceinline__ uint32_t atom_add_acq_rel_u32(uint32_t *p, uint32_t v)
{
    uint32_t old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

// As above without the returned value: the thread does not wait for the memory system.
__device__ __forceinline__ void red_add_release_u32(uint32_t *p, uint32_t v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ void fence_sc_gpu()
{
    asm volatile("fence.sc.gpu;" ::: "memory");
}

// Fused restore: a job may be committed only after all of its pages have been
// verified.  The verify side counts finalized pages in job_done[j]; the commit
// side waits here, with a time limit.  The wait cannot deadlock as long as all
// CTAs of the launch are resident (the host sizes the grid so), because the
// verify warps never wait for the commit warps.
__device__ __forceinline__ bool wait_job_verified(const StreamParams &P, uint32_t j, uint32_t n_pages,
                                                  volatile uint32_t *abort_flag)
{
    const uint32_t *cnt = P.w.job_done + j;
    if (ld_acquire_u32(cnt) >= n_pages) return true;
    if (*abort_flag) return false;
    const unsigned long long t0 = global_timer_ns();
    uint32_t spins = 0;
    volatile uint32_t *beat = abort_flag + 1;  // tells the storer behind this loader that it is alive
    while (ld_acquire_u32(cnt) < n_pages) {
        __nanosleep(100);
        if ((++spins & 0x3fu) == 0u) {
            *beat = *beat + 1u;
            if (*abort_flag || global_timer_ns() - t0 > P.w.wait_limit_ns) {
                atomicCAS(P.w.error, 0u, 0x500u);
                return false;
            }
        }
    }
    return true;
}

// The commit decision of a job is taken ONCE, by whichever commit loader meets
// the job first: it waits (fused kernel) until the job has been verified, works
// out the result code, and publishes it in job_latch[j] with a compare-and-swap;
// the winner also writes the job's report (write_report, which it may put off
// until it has issued the copies of its own item).  Every other commit item of
// the job, in any CTA, reads the latched code, so a job is committed whole or
// not at all even if a wait runs out somewhere else in the meantime.  Lane 0
// decides, the warp gets the code.
struct Report {
    uint32_t pending = 0u;  // lane 0: this loader took the decision and still owes the report
    uint32_t j = 0u, code = 0u;
    int32_t first_bad = -1;
};

__device__ __forceinline__ void write_report(const StreamParams &P, Report &rep)
{
    if (!rep.pending) return;
    rep.pending = 0u;
    if (!P.mask_out) return;
    P.mask_out[rep.j] = (uint8_t)rep.code;
    P.first_bad_out[rep.j] = rep.first_bad;
    // a CTA that had to give up on one of this job's items may have changed the verdict meanwhile
    fence_sc_gpu();
    if (ld_acquire_u32(P.w.job_latch + rep.j) != rep.code) P.mask_out[rep.j] = 4u;
}

__device__ __forceinline__ uint32_t commit_decision(const StreamParams &P, uint32_t j, const JobDev &jb,
                                                    volatile uint32_t *abort_flag, int lane, Report &rep)
{
    uint32_t code = 0u;
    if (lane == 0) {
        code = ld_acquire_u32(P.w.job_latch + j);
        if (code == kUndecided) {
            bool verified = true;
            if (P.fused && !jb.missing && P.w.bad_range[j] == kNoPage && P.w.bad_dup[j] == kNoPage)
                verified = wait_job_verified(P, j, jb.n_pages, abort_flag);
            int32_t fb;
            code = job_code(P.w, j, &fb, P.fused != 0u, verified);
            const uint32_t old = atomicCAS(P.w.job_latch + j, kUndecided, code);
            if (old != kUndecided) {
                code = old;
            } else {
                write_report(P, rep);  // at most one report is owed at a time
                rep.pending = 1u;
                rep.j = j;
                rep.code = code;
                rep.first_bad = fb;
            }
        }
    }
    return __shfl_sync(0xffffffffu, code, 0);
}

// A CTA that has given up (one of its own bounded waits ran out) can no longer
// write the items it draws.  If such an item belongs to a job that was accepted,
// the job ends up partly written: its verdict becomes "a wait ran out" (4), for
// the report and for every commit item of the job that has not started yet.
__device__ __forceinline__ void revoke_job(const StreamParams &P, uint32_t j)
{
    atomicExch(P.w.job_latch + j, 4u);
    fence_sc_gpu();
    if (P.mask_out) P.mask_out[j] = 4u;
}

// Tiles of segment q of a page record with shape sh.  Returns false if the page
// has no such segment (a short last page has fewer).
__device__ __forceinline__ bool segment_tiles(const PageShape &sh, const Tiling &tl, uint32_t q, Item &it)
{
    it.nseg = sh.nseg;
    if (q >= sh.nseg) return false;
    it.q = q;
    it.pad = sh.pad;
    it.t = sh.t;
    it.tile_begin = q == 0u ? 0u : sh.ntiles0 + (q - 1u) * tl.seg_tiles;
    it.tile_count = q == 0u ? sh.ntiles0 : tl.seg_tiles;
    return true;
}

// Geometry of work item `item` of a launch from the tables of the call.  No decision is taken here.
template <int MODE>
__device__ __forceinline__ bool item_from_tables(const StreamParams &P, const Tiling &tl, uint32_t item,
                                                 const JobDev *&jbp, Item &it)
{
    const uint32_t local = item / tl.nseg_max;
    uint32_t q = item - local * tl.nseg_max;
    uint32_t gp = P.w.page_begin + local;
    it.j = P.w.n_jobs == 1u ? 0u : (uint32_t)P.w.page_job[gp];  // one dependent load less at the start of a lone block
    jbp = &P.w.jobs[it.j];
    const JobDev jb = *jbp;
    it.p = gp - jb.page_base;
    if (MODE == kCommit && P.commit_reverse) {
        // same items, walked from the end of the job: what was verified last is read back first
        it.p = jb.n_pages - 1u - it.p;
        gp = jb.page_base + it.p;
    }
    it.gp = gp;
    const PageShape sh = page_shape(P.g, jb, it.p, tl);
    if (MODE == kCommit && P.commit_reverse && q < sh.nseg) q = sh.nseg - 1u - q;
    it.rec = jb.blob + (uint64_t)it.p * P.g.R;
    it.sum = jb.checksums + it.p;
    it.phys = 0;
    return segment_tiles(sh, tl, q, it);
}

// The last job this commit loader asked about: consecutive items mostly belong to
// one job, whose latched decision need not be fetched again.
struct JobCache {
    uint32_t j = kUndecided, code = kUndecided;
};

// Loader only: geometry plus the decision whether the item is to be processed.
template <int MODE>
__device__ __forceinline__ bool admit_item(const StreamParams &P, const Tiling &tl, uint32_t item, Item &it,
                                           volatile uint32_t *abort_flag, int lane, Report &rep, JobCache &jc)
{
    const JobDev *jbp = nullptr;
    const bool exists = item_from_tables<MODE>(P, tl, item, jbp, it);
    const bool skip = jbp->missing || P.w.bad_range[it.j] != kNoPage ||
                      ((MODE == kVerify || MODE == kSingle) && P.w.bad_dup[it.j] != kNoPage);
    // the table entry does not depend on the decision: have it on its way while the decision is awaited
    if (MODE != kVerify && exists && !skip) it.phys = jbp->page_table[it.p];
    if (MODE == kCommit) {
        // every item asks, existing or not, so that every job of the launch gets its report
        uint32_t code;
        if (jc.j == it.j && jc.code != kUndecided) {
            code = jc.code;
        } else {
            code = commit_decision(P, it.j, *jbp, abort_flag, lane, rep);
            jc.j = it.j;
            jc.code = code;
        }
        bool take = code == 0u && exists;
        if (take && *abort_flag) {
            if (lane == 0) revoke_job(P, it.j);
            take = false;
        }
        if (!take) {
            if (lane == 0) write_report(P, rep);
            return false;
        }
    } else {
        if (!exists || skip) return false;
        if (MODE == kVerify && P.test_drop_from != 0u && it.j + 1u >= P.test_drop_from) return false;
    }
    return true;
}

// Byte range of a tile inside its record: `lead` zero bytes first (front
// padding), then `nreal` record bytes starting at record offset r0.
template <int STAGE_BYTES>
__device__ __forceinline__ void tile_range(uint32_t tile, uint32_t pad, uint32_t &lead, uint64_t &r0, uint32_t &nreal)
{
    const uint64_t v0 = (uint64_t)tile * STAGE_BYTES;
    lead = 0u;
    if (v0 < pad) lead = (pad - v0 >= (uint64_t)STAGE_BYTES) ? (uint32_t)STAGE_BYTES : (uint32_t)(pad - v0);
    r0 = v0 + lead - pad;
    nreal = (uint32_t)STAGE_BYTES - lead;
}

__device__ __forceinline__ uint8_t *slab_addr(const CacheDev &c, uint32_t slab, int32_t phys, uint64_t off)
{
    return c.data + (uint64_t)(slab >> 1) * c.layer_stride + (uint64_t)(slab & 1u) * c.kv_stride +
           (uint64_t)phys * c.page_stride + off;
}

// The data part of a record is a sequence of equal chunks, each contiguous in the
// cache.  Token-major slabs, and full pages in either layout: one chunk per slab
// (the first t rows).  A partial page of a head-major slab: one chunk per head
// (that head's first t tokens), kv_heads chunks per slab.
struct Chunks {
    uint32_t len;       // bytes of one chunk
    uint32_t per_slab;  // chunks per slab
    uint32_t stride;    // distance between the chunks of one slab in the cache
};

__device__ __forceinline__ Chunks chunks_of(const GeomDev &g, uint32_t t)
{
    Chunks c;
    if (g.head_major && t < g.page_tokens) {
        c.len = t * g.hrow;
        c.per_slab = g.kv_heads;
        c.stride = g.page_tokens * g.hrow;
    } else {
        c.len = t * g.row;
        c.per_slab = 1u;
        c.stride = 0u;
    }
    return c;
}

__device__ __forceinline__ uint8_t *chunk_addr(const CacheDev &c, const Chunks &ch, uint32_t chunk, int32_t phys,
                                               uint32_t off)
{
    if (ch.per_slab == 1u) return slab_addr(c, chunk, phys, off);  // the common case, without the division
    const uint32_t slab = chunk / ch.per_slab;
    const uint32_t sub = chunk - slab * ch.per_slab;
    return slab_addr(c, slab, phys, (uint64_t)sub * ch.stride + off);
}

__device__ __forceinline__ uint8_t *scale_addr(const GeomDev &g, const CacheDev &c, uint32_t idx, int32_t phys)
{
    // idx counts fp32 values of a scale section: [layer][kv < scale_kv][head]
    const uint32_t h = idx % g.kv_heads;
    const uint32_t lk = idx / g.kv_heads;
    const uint32_t kv = lk % g.scale_kv;
    const uint32_t l = lk / g.scale_kv;
    return c.scales + (uint64_t)l * c.s_layer_stride + (uint64_t)kv * c.s_kv_stride +
           (uint64_t)phys * c.s_page_stride + 4ull * h;
}

__device__ __forceinline__ uint32_t xor3(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ uint32_t xor2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("xor.b32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// All non-empty XOR combinations of four words; c[pat] = xor of t[i] for the bits i of pat.
__device__ __forceinline__ void combos4(uint32_t t0, uint32_t t1, uint32_t t2, uint32_t t3, uint32_t (&c)[16])
{
    c[0] = 0u;
    c[1] = t0;
    c[2] = t1;
    c[4] = t2;
    c[8] = t3;
    c[3] = xor2(t0, t1);
    c[5] = xor2(t0, t2);
    c[6] = xor2(t1, t2);
    c[9] = xor2(t0, t3);
    c[10] = xor2(t1, t3);
    c[12] = xor2(t2, t3);
    c[7] = xor3(t0, t1, t2);
    c[11] = xor3(t0, t1, t3);
    c[13] = xor3(t0, t2, t3);
    c[14] = xor3(t1, t2, t3);
    c[15] = xor3(c[3], t2, t3);
}

// One 8-bit step of the bit-sliced shift register: state <- state*x^8 + w(x) mod P
// for 32 streams at once.  U (0..7) is the number of steps taken since the
// registers were last in natural order; coefficient m lives in R[(m - 8U) & 63],
// so the shift itself costs nothing.  The eight top coefficients T[j] each add
// x^(64+j) mod P; their two groups of fifteen partial sums are shared by all
// outputs, so that every output costs one three-input XOR.  The XORs are spelled
// as lop3 so that the instruction count is exactly what is written here
// (64 + 22 per 8 words), whatever the compiler would make of a long ^ chain.
template <int U>
__device__ __forceinline__ void crc_step8(uint32_t (&R)[64], const uint32_t (&w)[8])
{
    constexpr uint64_t G[8] = GK_G8_INIT;
    uint32_t A[16], B[16];
    combos4(R[(56 - 8 * U) & 63], R[(57 - 8 * U) & 63], R[(58 - 8 * U) & 63], R[(59 - 8 * U) & 63], A);
    combos4(R[(60 - 8 * U) & 63], R[(61 - 8 * U) & 63], R[(62 - 8 * U) & 63], R[(63 - 8 * U) & 63], B);
#pragma unroll
    for (int m = 0; m < 64; ++m) {
        const int pa = (int)(((G[0] >> m) & 1ull) | (((G[1] >> m) & 1ull) << 1) | (((G[2] >> m) & 1ull) << 2) |
                             (((G[3] >> m) & 1ull) << 3));
        const int pb = (int)(((G[4] >> m) & 1ull) | (((G[5] >> m) & 1ull) << 1) | (((G[6] >> m) & 1ull) << 2) |
                             (((G[7] >> m) & 1ull) << 3));
        const int phys = (m - 8 - 8 * U) & 63;
        const uint32_t base = (m < 8) ? w[7 - m] : R[phys];
        if (pa != 0 && pb != 0)
            R[phys] = xor3(base, A[pa], B[pb]);
        else if (pa != 0)
            R[phys] = xor2(base, A[pa]);
        else if (pb != 0)
            R[phys] = xor2(base, B[pb]);
        else
            R[phys] = base;
    }
}

template <int NT>
struct FrobExp;
template <> struct FrobExp<32> { static constexpr int e = 10; };
template <> struct FrobExp<64> { static constexpr int e = 11; };
template <> struct FrobExp<128> { static constexpr int e = 12; };
template <> struct FrobExp<256> { static constexpr int e = 13; };

// The 32 streams of one thread as ONE unreduced polynomial,
//   sum_s x^(31-s) * (R_s)^(32*NT)   (degree < 95),
// in three 32-bit words: a0 = degrees 0..31, a1 = 32..63, a2 = 64..94.
template <int NT>
__device__ __forceinline__ void thread_poly(const uint32_t (&R)[64], uint32_t &a0, uint32_t &a1, uint32_t &a2)
{
    uint32_t Q[64];
    gk_frob<FrobExp<NT>::e>(R, Q);
    // bit s of Q[k] is the coefficient of x^(k+31-s)
    a0 = 0u;
    a1 = 0u;
    a2 = 0u;
#pragma unroll
    for (int k = 0; k < 64; ++k) {
        const uint32_t v = __brev(Q[k]);
        const int sh = k & 31;
        const uint32_t lo = v << sh;
        const uint32_t hi = sh ? (v >> (32 - sh)) : 0u;
        if (k < 32) {
            a0 ^= lo;
            a1 ^= hi;
        } else {
            a1 ^= lo;
            a2 ^= hi;
        }
    }
}

// w(x) * c(x) mod P for a 32-bit w: Horner over the bits of w, 32 steps of
// "times x, fold, add c if the bit is set" on a 64-bit value in two registers.
// The loop stays a loop (four steps per trip): the steps depend on one another
// anyway, and the instruction cache has better uses than 32 copies of them.
__device__ __forceinline__ uint64_t gf_mul32(uint32_t w, uint64_t c)
{
    const uint32_t cl = (uint32_t)c, ch = (uint32_t)(c >> 32);
    constexpr uint32_t pl = (uint32_t)kPoly, ph = (uint32_t)(kPoly >> 32);
    uint32_t rl = 0u, rh = 0u;
#pragma unroll 4
    for (int i = 0; i < 32; ++i) {
        const uint32_t m = (uint32_t)((int32_t)rh >> 31);
        rh = __funnelshift_l(rl, rh, 1);
        rl <<= 1;
        const uint32_t b = (uint32_t)((int32_t)w >> 31);
        w <<= 1;
        rl ^= (m & pl) ^ (b & cl);
        rh ^= (m & ph) ^ (b & ch);
    }
    return ((uint64_t)rh << 32) | rl;
}

// Threads -> CTA.  Thread t's polynomial sits 32 bits above thread t+1's, so the
// words of neighbouring threads overlap: inside a warp the three words that fall
// on one 32-bit slot are XORed across lanes, which leaves every lane ONE word to
// multiply by its constant kt = x^(32*(NT-1-t)+64) (32 steps instead of the 95 a
// whole polynomial would take), and two words that stick out above the warp's
// first lane (returned to lane 0 in over0, over1: slots 32 and 33 of the warp).
// Returns the XOR over the warp of the lanes' products (valid in every lane).
__device__ __forceinline__ uint64_t warp_remainder(uint32_t a0, uint32_t a1, uint32_t a2, uint64_t kt, int lane,
                                                   uint32_t &over0, uint32_t &over1)
{
    const uint32_t a1n = __shfl_down_sync(0xffffffffu, a1, 1);   // a1 of lane + 1
    const uint32_t a2n = __shfl_down_sync(0xffffffffu, a2, 1);   // a2 of lane + 1
    const uint32_t a2nn = __shfl_down_sync(0xffffffffu, a2, 2);  // a2 of lane + 2
    const uint32_t word = a0 ^ (lane < 31 ? a1n : 0u) ^ (lane < 30 ? a2nn : 0u);
    over0 = a1 ^ a2n;  // meaningful in lane 0 only
    over1 = a2;
    uint64_t v = gf_mul32(word, kt);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v ^= __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

// Ring position of a pipeline role: stage index and the parity of its use count.
struct RingPos {
    uint32_t stage = 0, phase = 0;
    template <int STAGES>
    __device__ __forceinline__ void advance()
    {
        if (++stage == (uint32_t)STAGES) {
            stage = 0;
            phase ^= 1u;
        }
    }
};

// The eight 8-word steps of one granule (after which the registers are back in
// natural order).  Every kSps steps a new stage is awaited and the finished one
// is handed back to the loader.  NT threads share TILE_BYTES of every stage (the
// whole stage, or with page quartets the warp's quarter of it: `smem` then points
// at that quarter of stage 0 and `tid` is the lane).
template <int U, int MODE, int NT, int STAGE_BYTES, int STAGES, int TILE_BYTES>
struct GranuleSteps {
    static constexpr int kSps = TILE_BYTES / (NT * 32);  // 8-word steps per stage
    static __device__ __forceinline__ void run(uint32_t (&R)[64], const uint8_t *smem, uint32_t full0, uint32_t empty0,
                                               RingPos &pos, volatile uint32_t *abort_flag, uint32_t *error,
                                               unsigned long long limit_ns, int tid, int lane)
    {
        if (U % kSps == 0) mbar_wait(full0 + 8u * pos.stage, pos.phase, abort_flag, error, 0x400u | MODE, limit_ns);
        const uint32_t *sw = reinterpret_cast<const uint32_t *>(smem + (size_t)pos.stage * STAGE_BYTES) + tid;
        uint32_t w[8];
#pragma unroll
        for (int jw = 0; jw < 8; ++jw) w[jw] = sw[((U % kSps) * 8 + jw) * NT];
        crc_step8<U>(R, w);
        if (U % kSps == kSps - 1) {
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8u * pos.stage);
            pos.template advance<STAGES>();
        }
        GranuleSteps<U + 1, MODE, NT, STAGE_BYTES, STAGES, TILE_BYTES>::run(R, smem, full0, empty0, pos, abort_flag, error,
                                                                            limit_ns, tid, lane);
    }
};
template <int MODE, int NT, int STAGE_BYTES, int STAGES, int TILE_BYTES>
struct GranuleSteps<8, MODE, NT, STAGE_BYTES, STAGES, TILE_BYTES> {
    static __device__ __forceinline__ void run(uint32_t (&)[64], const uint8_t *, uint32_t, uint32_t, RingPos &,
                                               volatile uint32_t *, uint32_t *, unsigned long long, int, int)
    {
    }
};

// Work is handed out dynamically: the loader warp of a CTA draws item numbers
// from a global counter (so the CTAs that are resident take all the work, in
// order, whatever their number), and tags every stage it fills with the item's
// slot and the tile index; the other roles of the CTA follow the tags.  A stage
// tagged kEndOfWork tells them to leave.  Where no CTA ever waits for another
// one's item (everything but the verify side of the fused kernel) a CTA takes
// the item with its own number first, without asking the counter.
constexpr uint32_t kEndOfWork = 0xffffffffu;
constexpr uint32_t kNoJob = 0xffffffffu;

// Developer aid, compiled in with -DGK_TRACE only: every role of every CTA leaves the
// %globaltimer value of its first pass through a few marked places in P.trace
// ([CTA][role 0..3][event 0..15]; roles: verify/pack loader, commit loader, consumer, storer).
#ifdef GK_TRACE
#define GK_TRACE_EVT(P, role, ev)                                                                     \
    do {                                                                                              \
        if ((P).trace && (threadIdx.x & 31) == 0) {                                                   \
            unsigned long long *slot_ = (P).trace + ((size_t)blockIdx.x * 4 + (role)) * 16 + (ev);     \
            if (*slot_ == 0ull) *slot_ = global_timer_ns();                                           \
        }                                                                                             \
    } while (0)
#else
#define GK_TRACE_EVT(P, role, ev) \
    do {                          \
    } while (0)
#endif

// Bounds-checked build (-DGK_DEBUG): before every access of a streaming kernel to caller
// memory -- the bulk copies from and to cache and blobs, the scale values, the checksum words --
// the address range is compared with the extent of the object it belongs to.  An access that
// falls outside is NOT made (a refused load still counts as arrived, so that nothing waits for
// it); the first one leaves what it was in the debug words behind the context's error word:
// [8] = role << 8 | kind, [9..10] = offset from the object's base, [11] = bytes.  Nothing traps.
enum DebugKind : uint32_t { kDbgCache = 1, kDbgBlob = 2, kDbgScales = 3, kDbgSums = 4, kDbgStage = 5 };
#ifdef GK_DEBUG
__device__ __noinline__ void debug_report(const StreamParams &P, uint32_t kind, uint32_t role, uint64_t addr,
                                          uint64_t bytes, uint64_t base)
{
    if (atomicCAS(P.w.error + 8, 0u, (role << 8) | kind) == 0u) {
        const uint64_t off = addr - base;
        P.w.error[9] = (uint32_t)off;
        P.w.error[10] = (uint32_t)(off >> 32);
        P.w.error[11] = (uint32_t)bytes;
    }
}
__device__ __forceinline__ bool debug_ok(const StreamParams &P, uint32_t kind, uint32_t role, const void *addr,
                                         uint64_t bytes, const void *base, uint64_t extent)
{
    if (range_inside((uint64_t)addr, bytes, (uint64_t)base, extent)) return true;
    debug_report(P, kind, role, (uint64_t)addr, bytes, (uint64_t)base);
    return false;
}
// extent of the blob of the job an item belongs to
__device__ __forceinline__ uint64_t debug_blob_bytes(const StreamParams &P, uint32_t j)
{
    const JobDev &jb = P.w.jobs[j];
    return (uint64_t)jb.n_pages * P.g.S + (uint64_t)jb.n_tokens * P.g.tokB;
}
#define GK_DEBUG_OK(P, kind, role, addr, bytes, base, extent) debug_ok(P, kind, role, addr, bytes, base, extent)
#else
#define GK_DEBUG_OK(P, kind, role, addr, bytes, base, extent) true
#endif

template <bool STATIC_FIRST>
__device__ __forceinline__ uint32_t next_item(uint32_t *ctr, uint32_t base, int lane)
{
    uint32_t v = 0;
    if (lane == 0) v = atomicAdd(ctr, 1u) - base + (STATIC_FIRST ? gridDim.x : 0u);
    return __shfl_sync(0xffffffffu, v, 0);
}

// Commit modes, after this CTA has given up: every job that may still have a tile
// of this CTA in flight loses its "accepted" verdict (see revoke_job).
template <int STAGES>
__device__ __forceinline__ void revoke_in_flight(const StreamParams &P, const Ring &ring)
{
    for (int k = 0; k <= STAGES; ++k) {
        const uint32_t j = ring.items[k].j;
        if (j != kNoJob) revoke_job(P, j);
    }
}

// ----------------------------- finisher role -----------------------------
// The kernels that verify have a warp for it; in the kernels that pack, whose
// consumers need the registers a further warp would take, consumer warp 0 does
// it after its own part of the segment.  Takes what the consumer warps
// hand over at the end of a segment and finishes it: adds the words that stick
// out above each warp (times their constants) to the warps' partial remainders,
// places the segment inside its page and XORs it into the page's accumulator.
// Where pages are finalized inline, the CTA that delivers the last segment of a
// page also finishes the page -- final xor, reflection, then write the checksum
// (pack) or compare it with the stored one and count the page in job_done, which
// the commit side of the fused kernel waits on.  Neither the consumers nor the
// loader are held up by any of this (the round trips to memory in particular).
//
// Hand-over slot (two of them, used in turn), 12 x 8 bytes: [0..3] the consumer
// warps' partial remainders, [4..7] as 32-bit words the two words above each
// warp, [8..11] a copy of what the finisher needs to know about the item.
struct HandOver {
    uint64_t *sum;
    uint32_t gp, j, p, q, nseg, t;
};
constexpr int kHandOverWords = 12;

struct Finisher {
    uint32_t done = 0;   // segments finished so far
    uint64_t kover = 0;  // lanes 0 .. 2*NT/32-1: constants of the words above the warps
};

// Where the constants of a record reduced by one warp (page quartets) start in thread_const.
template <int NT>
struct QuadConst {
    static constexpr int kLane0 = NT + 2 * (NT / 32);  // 32 lane constants
    static constexpr int kOver0 = kLane0 + 32;         // constants of the two words above the warp
};

template <int NT, bool QUAD = false>
__device__ __forceinline__ void finisher_init(const StreamParams &P, Finisher &fin, int lane)
{
    if (QUAD) {
        if (lane < 8) fin.kover = P.w.thread_const[QuadConst<NT>::kOver0 + (lane & 1)];
    } else if (NT > 0 && lane < 2 * (NT / 32)) {
        fin.kover = P.w.thread_const[NT + lane];
    }
}

// Has the next segment been handed over?  (Every lane may ask; use finisher_ready for a warp-wide answer.)
__device__ __forceinline__ bool finisher_posted(const Ring &ring, const Finisher &fin)
{
    return mbar_test_wait(ring.tail0 + 8u * (fin.done & 1u), (fin.done >> 1) & 1u);
}

__device__ __forceinline__ bool finisher_ready(const Ring &ring, const Finisher &fin)
{
    return __shfl_sync(0xffffffffu, finisher_posted(ring, fin) ? 1 : 0, 0) != 0;
}

// Finishes the segment in hand-over slot fin.done & 1 (the whole warp takes part).  `taken` is
// the barrier to arrive on once the slot has been read, or 0.
template <int MODE, int NT>
__device__ __forceinline__ void finish_segment(const StreamParams &P, const Ring &ring, Finisher &fin,
                                               const HandOver &it, uint32_t taken, volatile uint32_t *abort_flag,
                                               int lane)
{
    constexpr int kW = NT / 32;
    const uint32_t par = fin.done & 1u;
    const uint64_t *slot = ring.red + kHandOverWords * par;
    const uint32_t *oslot = reinterpret_cast<const uint32_t *>(slot + 4);
    const uint32_t nseg = it.nseg;
    // the factors that place the two halves of the remainder inside the page: loads first, arithmetic below
    uint64_t kplace = 0ull;
    if (nseg > 1u && lane < 2) kplace = P.w.seg_pow[2u * (nseg - 1u - it.q) + lane];
    uint64_t tot = 0;
    if (lane < 2 * kW) tot = gf_mul32(oslot[lane], fin.kover);
    if (lane < kW) tot ^= slot[lane];
    __syncwarp();
    if (taken != 0u && lane == 0) mbar_arrive(taken);  // the slot has been read: it may be used again
#pragma unroll
    for (int d = 4; d > 0; d >>= 1) tot ^= __shfl_xor_sync(0xffffffffu, tot, d);
    // place the segment: the short segment comes first and all others are full, so (nseg - 1 - q)
    // full segments follow this one
    if (nseg > 1u) {
        tot = __shfl_sync(0xffffffffu, tot, 0);
        uint64_t part = 0;
        if (lane < 2) part = gf_mul32(lane == 0 ? (uint32_t)tot : (uint32_t)(tot >> 32), kplace);
        tot = part ^ __shfl_xor_sync(0xffffffffu, part, 1);
    }
    if (lane == 0) {
        uint64_t *acc = P.w.page_acc + it.gp;
        if (!P.inline_final) {
            red_xor_u64(acc, tot);
        } else {
            uint64_t stored = 0;
#ifdef GK_DEBUG
            const bool sum_ok = debug_ok(P, kDbgSums, 2u, it.sum, 8u, P.w.jobs[it.j].checksums,
                                         8ull * P.w.jobs[it.j].n_pages);
#else
            constexpr bool sum_ok = true;
#endif
            if (MODE != kPack && sum_ok) stored = *it.sum;  // in flight together with the two atomics below
            uint64_t r = tot;
            bool last = true;
            if (nseg > 1u) {
                red_xor_u64(acc, tot);
                last = atom_add_acq_rel_u32(&P.w.page_cnt[it.gp], 1u) + 1u == nseg;
                if (last) r = ld_acquire_u64(acc);
            }
            if (last) {
                const uint64_t crc = __brevll(r ^ P.w.init_term[it.t] ^ ~0ull);
                if (MODE == kPack) {
                    if (sum_ok) *it.sum = crc;
                } else {
                    if (crc != stored || *abort_flag) atomicMin(&P.w.bad_crc[it.j], (int32_t)it.p);
                    red_add_release_u32(&P.w.job_done[it.j], 1u);  // nobody here waits for the count
                }
            }
        }
    }
    __syncwarp();
    ++fin.done;
    GK_TRACE_EVT(P, 2, 3);
}

__device__ __forceinline__ HandOver hand_over_of(const Item &it)
{
    HandOver h;
    h.sum = it.sum;
    h.gp = it.gp;
    h.j = it.j;
    h.p = it.p;
    h.q = it.q;
    h.nseg = it.nseg;
    h.t = it.t;
    return h;
}

// Page quartets: the four consumer warps hand over one whole record each (hand-over slot as
// above, with the quartet's pages in the place of the item copy).  Lanes 0..7 multiply the
// words above the warps by their constants, lanes 0..3 then finish one page each: final xor,
// reflection, and either the checksum is written (pack) or compared with the stored one and
// the page counted in job_done.
//
// `ahead` (pack, where a consumer warp does this between two records): what lanes 0..3 need
// from the tables of the call, fetched by them when the quartet began, so that no load from
// global memory stands between the end of the records and the next quartet.
struct QuadAhead {
    uint64_t *sum = nullptr;  // the page's checksum word, or null: no page in this lane
    uint64_t init = 0;        // the term of the all-ones initial register for the page's length
};

__device__ __forceinline__ QuadAhead quad_ahead(const StreamParams &P, const QuadPages &pg, int lane)
{
    QuadAhead a;
    if (lane < 4 && pg.j[lane] != kNoJob) {
        const JobDev jb = P.w.jobs[pg.j[lane]];
        a.sum = jb.checksums + pg.p[lane];
        a.init = P.w.init_term[page_fill(P.g, jb, pg.p[lane])];
    }
    return a;
}

template <int MODE>
__device__ __forceinline__ void finish_quad(const StreamParams &P, const Ring &ring, Finisher &fin,
                                            const QuadPages &pg, uint32_t taken, volatile uint32_t *abort_flag,
                                            int lane, const QuadAhead *ahead = nullptr)
{
    static_assert(MODE == kVerify || MODE == kPack, "page quartets: pack and verify only");
    const uint32_t par = fin.done & 1u;
    const uint64_t *slot = ring.red + kHandOverWords * par;
    const uint32_t *oslot = reinterpret_cast<const uint32_t *>(slot + 4);
    uint64_t tot = 0;
    if (lane < 8) tot = gf_mul32(oslot[lane], fin.kover);
    tot ^= __shfl_xor_sync(0xffffffffu, tot, 1);                                 // both words of a warp
    const uint64_t above = __shfl_sync(0xffffffffu, tot, (2 * lane) & 31);       // lane w: those of warp w
    uint32_t j = kNoJob, p = 0u;
    uint64_t r = 0;
    if (lane < 4) {
        j = pg.j[lane];
        p = pg.p[lane];
        r = slot[lane] ^ above;
    }
    __syncwarp();
    if (taken != 0u && lane == 0) mbar_arrive(taken);  // the slot has been read: it may be used again
#ifndef GK_DEBUG
    if (MODE == kPack && ahead != nullptr && P.inline_final) {
        if (ahead->sum) *ahead->sum = __brevll(r ^ ahead->init ^ ~0ull);
        __syncwarp();
        ++fin.done;
        return;
    }
#endif
    if (j != kNoJob) {
        const JobDev jb = P.w.jobs[j];
        if (!P.inline_final) {
            red_xor_u64(P.w.page_acc + jb.page_base + p, r);
        } else {
            uint64_t *sum = jb.checksums + p;
#ifdef GK_DEBUG
            const bool sum_ok = debug_ok(P, kDbgSums, 2u, sum, 8u, jb.checksums, 8ull * jb.n_pages);
#else
            constexpr bool sum_ok = true;
#endif
            const uint64_t crc = __brevll(r ^ P.w.init_term[page_fill(P.g, jb, p)] ^ ~0ull);
            if (MODE == kPack) {
                if (sum_ok) *sum = crc;
            } else {
                const uint64_t stored = sum_ok ? *sum : 0ull;
                if (crc != stored || *abort_flag) atomicMin(&P.w.bad_crc[j], (int32_t)p);
                red_add_release_u32(&P.w.job_done[j], 1u);  // nobody here waits for the count
            }
        }
    }
    __syncwarp();
    ++fin.done;
}

// Finishes segments until the loader's count of admitted items has been reached (the count is
// known once the loader has put the end mark into the ring).
template <int MODE, int NT, bool QUAD = false>
__device__ __forceinline__ void finisher_drain(const StreamParams &P, const Ring &ring, Finisher &fin,
                                               volatile uint32_t *abort_flag, int lane)
{
    volatile uint32_t *n_final = abort_flag + 2;
    for (;;) {
        bool posted = finisher_posted(ring, fin);
        if (!posted) {
            const unsigned long long t0 = global_timer_ns();
            uint32_t spins = 0;
            for (;;) {
                if (finisher_posted(ring, fin)) {
                    posted = true;
                    break;
                }
                if (*n_final == fin.done) break;
                __nanosleep(64);
                if ((++spins & 0xffu) == 0u) {
                    // the consumers' own waits are bounded; this one only has to outlast them
                    if (global_timer_ns() - t0 > 4ull * P.w.wait_limit_ns) {
                        *abort_flag = 1u;
                        atomicCAS(P.w.error, 0u, 0x700u | MODE);
                        break;
                    }
                }
            }
        }
        posted = __shfl_sync(0xffffffffu, posted ? 1 : 0, 0) != 0;  // one decision for the warp
        if (!posted) break;
        const uint32_t par = fin.done & 1u;
        if constexpr (QUAD) {
            const QuadPages pg = *reinterpret_cast<const QuadPages *>(ring.red + kHandOverWords * par + 8);
            finish_quad<MODE>(P, ring, fin, pg, ring.tail0 + 8u * (2u + par), abort_flag, lane);
        } else {
            const HandOver it = *reinterpret_cast<const HandOver *>(ring.red + kHandOverWords * par + 8);
            finish_segment<MODE, NT>(P, ring, fin, it, ring.tail0 + 8u * (2u + par), abort_flag, lane);
        }
    }
}

// The role as a warp of its own (kernels whose storer warp, if any, has no time for it).
template <int MODE, int NT, bool QUAD = false>
__device__ __forceinline__ void finisher_role(const StreamParams &P, const Ring &ring, volatile uint32_t *abort_flag,
                                              int lane)
{
    Finisher fin;
    finisher_init<NT, QUAD>(P, fin, lane);
    finisher_drain<MODE, NT, QUAD>(P, ring, fin, abort_flag, lane);
}

// ------------------------------ loader role ------------------------------
// One warp.  Draws work items, decides whether each is to be processed, walks it
// tile by tile, waits for a free stage and fills it: front padding zeroed by the
// lanes (CRC modes), scale values gathered by the lanes (pack), everything else
// by bulk async copies issued by lane 0 that complete on the stage's full barrier.
template <int MODE, int NT, int STAGE_BYTES, int STAGES, bool ZERO_PAD, bool STATIC_FIRST>
__device__ __forceinline__ void loader_role(const StreamParams &P, const Tiling &tl, uint32_t n_items, uint32_t *ctr,
                                            uint32_t ctr_base, const Ring &ring, volatile uint32_t *abort_flag,
                                            int lane)
{
    uint32_t n = 0;       // tiles issued
    uint32_t n_adm = 0;   // items admitted
    bool revoked = false;
    Report rep;
    JobCache jc;
    uint64_t policy = 0;
    const bool hint = (MODE == kVerify && (P.l2_hints & 1u)) || (MODE == kCommit && (P.l2_hints & 2u));
    if (hint) policy = (MODE == kVerify) ? policy_evict_last() : policy_evict_first();
    GK_TRACE_EVT(P, MODE == kCommit ? 1 : 0, 1);
    for (uint32_t item = STATIC_FIRST ? blockIdx.x : next_item<false>(ctr, ctr_base, lane); item < n_items;
         item = next_item<STATIC_FIRST>(ctr, ctr_base, lane)) {
        Item it;
        if (!admit_item<MODE>(P, tl, item, it, abort_flag, lane, rep, jc)) continue;
        GK_TRACE_EVT(P, MODE == kCommit ? 1 : 0, 2);
        const uint32_t slot = n_adm % (uint32_t)(STAGES + 1);
        ++n_adm;
#ifdef GK_TRACE
        if (n_adm == 16u) GK_TRACE_EVT(P, MODE == kCommit ? 1 : 0, 6);
        if (n_adm == 48u) GK_TRACE_EVT(P, MODE == kCommit ? 1 : 0, 7);
#endif
        const Chunks ch = chunks_of(P.g, it.t);
        for (uint32_t k = 0; k < it.tile_count; ++k, ++n) {
            const uint32_t s = n % STAGES;
            const uint32_t use = n / STAGES;
            if (use > 0u) mbar_wait(ring.empty0 + 8u * s, (use - 1u) & 1u, abort_flag, P.w.error, 0x100u | MODE,
                                    P.w.wait_limit_ns);
            if (k == 0u && lane == 0) ring.items[slot] = it;  // the stage's barrier publishes it with the tile
            uint32_t lead, nreal;
            uint64_t r0;
            tile_range<STAGE_BYTES>(it.tile_begin + k, it.pad, lead, r0, nreal);
            const uint32_t sbase = ring.stage0 + s * STAGE_BYTES;
            uint8_t *sgen = ring.base + (size_t)s * STAGE_BYTES;
            if (ZERO_PAD) {
                for (uint32_t o = lane * 16u; o < lead; o += 512u)
                    *reinterpret_cast<uint4 *>(sgen + o) = make_uint4(0u, 0u, 0u, 0u);
            }
            uint32_t scale_bytes = 0u;
            if (MODE == kPack && r0 < P.g.S && nreal > 0u) {
                // scale values of this tile: gathered with ordinary loads
                const uint64_t e1 = (r0 + nreal < P.g.S) ? r0 + nreal : P.g.S;
                scale_bytes = (uint32_t)(e1 - r0);
                // eight loads in flight per lane: the loader must not sit on one global latency per value
                const uint32_t i_end = (uint32_t)(e1 >> 2);
                for (uint32_t i0 = (uint32_t)(r0 >> 2) + lane; i0 < i_end; i0 += 32u * 8u) {
                    uint32_t v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const uint32_t i = i0 + 32u * u;
                        const uint8_t *sa = scale_addr(P.g, P.cache, i < i_end ? i : (uint32_t)(r0 >> 2), it.phys);
                        v[u] = (i < i_end && GK_DEBUG_OK(P, kDbgScales, 0u, sa, 4u, P.cache.scales, P.cache.scales_extent))
                                   ? *reinterpret_cast<const uint32_t *>(sa) : 0u;
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const uint32_t i = i0 + 32u * u;
                        if (i < i_end) *reinterpret_cast<uint32_t *>(sgen + lead + (4u * i - (uint32_t)r0)) = v[u];
                    }
                }
                fence_proxy_async_smem();
            }
            __syncwarp();
            if (lane == 0) {
                ring.tag[s] = make_uint2(slot, k);
                if (*abort_flag) {
                    if (MODE == kCommit && !revoked) {
                        revoke_in_flight<STAGES>(P, ring);
                        revoked = true;
                    }
                } else {
                    const uint32_t bar = ring.full0 + 8u * s;
                    if (MODE == kPack) {
                        const uint32_t data_bytes = nreal - scale_bytes;
                        if (data_bytes == 0u) {
                            mbar_arrive(bar);
                        } else {
                            mbar_arrive_expect_tx(bar, data_bytes);
                            uint64_t d0 = r0 + scale_bytes - P.g.S;  // offset in the record's data part
                            const uint64_t d1 = d0 + data_bytes;
                            uint32_t so = sbase + lead + scale_bytes;
                            uint32_t chunk = (uint32_t)(d0 / ch.len);
                            uint32_t off = (uint32_t)(d0 - (uint64_t)chunk * ch.len);
                            while (d0 < d1) {
                                uint32_t nb = ch.len - off;
                                if ((uint64_t)nb > d1 - d0) nb = (uint32_t)(d1 - d0);
                                if (nb == 0u) break;  // cannot happen with a valid geometry; never spin
                                const uint8_t *ca = chunk_addr(P.cache, ch, chunk, it.phys, off);
                                if (GK_DEBUG_OK(P, kDbgCache, 0u, ca, nb, P.cache.data, P.cache.data_extent) &&
                                    GK_DEBUG_OK(P, kDbgStage, 0u, (const void *)(uintptr_t)so, nb,
                                                (const void *)(uintptr_t)sbase, STAGE_BYTES))
                                    bulk_g2s(so, ca, nb, bar);
                                else
                                    mbar_complete_tx(bar, nb);
                                d0 += nb;
                                so += nb;
                                ++chunk;
                                off = 0u;
                            }
                        }
                    } else {
                        if (nreal == 0u) {
                            mbar_arrive(bar);
                        } else {
                            mbar_arrive_expect_tx(bar, nreal);
#ifdef GK_DEBUG
                            const bool in_blob = debug_ok(P, kDbgBlob, MODE == kCommit ? 1u : 0u, it.rec + r0, nreal,
                                                          P.w.jobs[it.j].blob, debug_blob_bytes(P, it.j)) &&
                                                 debug_ok(P, kDbgStage, 0u, (const void *)(uintptr_t)(lead + nreal), 0u,
                                                          nullptr, STAGE_BYTES);
#else
                            constexpr bool in_blob = true;
#endif
                            if (!in_blob) mbar_complete_tx(bar, nreal);
                            else if (hint) bulk_g2s_hint(sbase + lead, it.rec + r0, nreal, bar, policy);
                            else bulk_g2s(sbase + lead, it.rec + r0, nreal, bar);
                        }
                    }
                }
            }
            __syncwarp();
        }
        if (MODE == kCommit && lane == 0) write_report(P, rep);  // the item's copies are on their way
        GK_TRACE_EVT(P, MODE == kCommit ? 1 : 0, 3);
    }
    // tell the other roles of this CTA that there is no more work
    {
        const uint32_t s = n % STAGES;
        const uint32_t use = n / STAGES;
        if (use > 0u) mbar_wait(ring.empty0 + 8u * s, (use - 1u) & 1u, abort_flag, P.w.error, 0x100u | MODE,
                                P.w.wait_limit_ns);
        if (lane == 0) {
            ring.tag[s] = make_uint2(kEndOfWork, 0u);
            mbar_arrive(ring.full0 + 8u * s);
            if (NT > 0) abort_flag[2] = n_adm;  // tells the finisher warp how many segments there are
        }
        ++n;
    }
    GK_TRACE_EVT(P, MODE == kCommit ? 1 : 0, 4);
    // before leaving: every load this CTA issued must have landed
    if (lane == 0) {
        for (uint32_t back = 0; back < (uint32_t)STAGES && back < n; ++back) {
            const uint32_t m = n - 1u - back;
            mbar_drain(ring.full0 + 8u * (m % STAGES), (m / STAGES) & 1u, P.w.wait_limit_ns);
        }
    }
}

// ------------------------------ storer role ------------------------------
// One warp.  Waits for each tile to land, reads its tag and its item's slot, and
// writes it out with bulk async copies: one contiguous piece into the blob
// (pack), or one piece per slab into the destination cache plus the scale values
// by the lanes (commit).  A stage goes back to the loader once the copy of the
// following tile has been issued and the stage's own copy has finished reading
// shared memory.  The storer takes no decision of its own: a tile that the
// loader put into the ring is a tile to be written.
template <int MODE, int STAGE_BYTES, int STAGES>
__device__ __forceinline__ void storer_role(const StreamParams &P, const Ring &ring, volatile uint32_t *abort_flag,
                                            int lane)
{
    uint32_t n = 0;
    bool revoked = false;
    // commit: the written pages are not read again by this call -- let them leave L2 before the blob does
    const bool store_hint = MODE == kCommit && (P.l2_hints & 4u);
    uint64_t store_policy = 0;
    if (store_hint) store_policy = policy_evict_first();
    for (;; ++n) {
        const uint32_t s = n % STAGES;
        // the loader ahead of a commit storer may itself be waiting, job after job, for verification
        bool ok = mbar_wait(ring.full0 + 8u * s, (n / STAGES) & 1u, abort_flag, P.w.error, 0x300u | MODE,
                            P.w.wait_limit_ns, MODE == kCommit ? abort_flag + 1 : nullptr);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {  // the CTA has given up: nothing more is stored (decided by the whole warp)
            if (MODE == kCommit && lane == 0 && !revoked) revoke_in_flight<STAGES>(P, ring);
            break;
        }
        const uint2 tag = ring.tag[s];
        if (tag.x == kEndOfWork) break;
        GK_TRACE_EVT(P, 3, 0);
        const Item &it = ring.items[tag.x];
        const int32_t phys = it.phys;
        const Chunks ch = chunks_of(P.g, it.t);
        uint32_t lead, nreal;
        uint64_t r0;
        tile_range<STAGE_BYTES>(it.tile_begin + tag.y, it.pad, lead, r0, nreal);
        const uint32_t sbase = ring.stage0 + s * STAGE_BYTES;
        const uint8_t *sgen = ring.base + (size_t)s * STAGE_BYTES;
        const bool aborted = *abort_flag != 0u;
        if (aborted && MODE == kCommit && lane == 0 && !revoked) {
            revoke_in_flight<STAGES>(P, ring);
            revoked = true;
        }
        uint32_t scale_bytes = 0u;
        if ((MODE == kCommit || MODE == kSingle) && r0 < P.g.S && nreal > 0u) {
            const uint64_t e1 = (r0 + nreal < P.g.S) ? r0 + nreal : P.g.S;
            scale_bytes = (uint32_t)(e1 - r0);
            if (!aborted) {
                for (uint32_t i = (uint32_t)(r0 >> 2) + lane; i < (uint32_t)(e1 >> 2); i += 32u) {
                    const uint32_t v = *reinterpret_cast<const uint32_t *>(sgen + lead + (4u * i - (uint32_t)r0));
                    uint8_t *sa = scale_addr(P.g, P.cache, i, phys);
                    if (GK_DEBUG_OK(P, kDbgScales, 3u, sa, 4u, P.cache.scales, P.cache.scales_extent))
                        *reinterpret_cast<uint32_t *>(sa) = v;
                }
            }
        }
        __syncwarp();
        if (lane == 0) {
            if (!aborted && nreal > 0u) {
                if (MODE == kPack) {
#ifdef GK_DEBUG
                    if (debug_ok(P, kDbgBlob, 3u, it.rec + r0, nreal, P.w.jobs[it.j].blob, debug_blob_bytes(P, it.j)))
#endif
                        bulk_s2g(it.rec + r0, sbase + lead, nreal);
                } else {
                    const uint32_t data_bytes = nreal - scale_bytes;
                    uint64_t d0 = r0 + scale_bytes - P.g.S;
                    const uint64_t d1 = d0 + data_bytes;
                    uint32_t so = sbase + lead + scale_bytes;
                    uint32_t chunk = (uint32_t)(d0 / ch.len);
                    uint32_t off = (uint32_t)(d0 - (uint64_t)chunk * ch.len);
                    while (d0 < d1) {
                        uint32_t nb = ch.len - off;
                        if ((uint64_t)nb > d1 - d0) nb = (uint32_t)(d1 - d0);
                        if (nb == 0u) break;  // cannot happen with a valid geometry; never spin
                        uint8_t *ca = chunk_addr(P.cache, ch, chunk, phys, off);
                        if (GK_DEBUG_OK(P, kDbgCache, 3u, ca, nb, P.cache.data, P.cache.data_extent)) {
                            if (store_hint) bulk_s2g_hint(ca, so, nb, store_policy);
                            else bulk_s2g(ca, so, nb);
                        }
                        d0 += nb;
                        so += nb;
                        ++chunk;
                        off = 0u;
                    }
                }
            }
            bulk_commit();
            GK_TRACE_EVT(P, 3, 1);
            if (n > 0u) {
                bulk_wait_read<1>();
                mbar_arrive(ring.empty0 + 8u * ((n - 1u) % STAGES));
            }
        }
        __syncwarp();
    }
    if (lane == 0) {
        bulk_wait_all();
        if (n > 0u) mbar_arrive(ring.empty0 + 8u * ((n - 1u) % STAGES));
    }
    GK_TRACE_EVT(P, 3, 2);
}

// ------------------------- page quartets: loader, storer -------------------------
// Small records (tens of KiB) pay the per-thread epilogue of the checksum once per record
// and NT threads, which costs as much as the record's main loop when the record is short.
// With page quartets a work item is four consecutive pages of the launch and every
// consumer warp reduces one WHOLE record on its own (32 threads per record: a quarter of
// the epilogues per byte): a shared-memory stage holds one tile of STAGE_BYTES / 4 bytes
// of each of the four records.  Lanes 0..3 of the loader (and of the storer) serve one page
// each and issue its copies themselves.  Records of a quartet that are shorter than its
// longest one (the last page of a job) get whole tiles of zeros in front; a page that is
// not to be processed (missing job, bad table, past the end of the launch) has job kNoJob:
// nothing is copied for it, its warp reduces whatever the stage holds and the result is
// dropped.
template <int MODE, int STAGE_BYTES, int STAGES, bool STATIC_FIRST>
__device__ __forceinline__ void loader_role_quad(const StreamParams &P, uint32_t *ctr, uint32_t ctr_base,
                                                 const Ring &ring, volatile uint32_t *abort_flag, int lane)
{
    static_assert(MODE == kVerify || MODE == kPack, "page quartets: pack and verify only");
    constexpr uint32_t QB = STAGE_BYTES / 4;
    uint32_t n = 0;      // tiles (stages) issued
    uint32_t n_adm = 0;  // items admitted
    uint64_t policy = 0;
    const bool hint = MODE == kVerify && (P.l2_hints & 1u);
    if (hint) policy = policy_evict_last();
    GK_TRACE_EVT(P, 0, 1);
    for (uint32_t item = STATIC_FIRST ? blockIdx.x : next_item<false>(ctr, ctr_base, lane); item < P.n_items;
         item = next_item<STATIC_FIRST>(ctr, ctr_base, lane)) {
        // lanes 0..3: one page each
        uint32_t j = kNoJob, p = 0u, t = 0u, ntiles = 0u, pad = 0u;
        int32_t phys = 0;
        uint8_t *rec = nullptr;
        const uint32_t local = item * 4u + (uint32_t)lane;
        if (lane < 4 && local < P.w.total_pages) {
            const uint32_t gp = P.w.page_begin + local;
            const uint32_t jj = (uint32_t)P.w.page_job[gp];
            const JobDev jb = P.w.jobs[jj];
            bool skip = jb.missing || P.w.bad_range[jj] != kNoPage;
            if (MODE == kVerify)
                skip = skip || P.w.bad_dup[jj] != kNoPage || (P.test_drop_from != 0u && jj + 1u >= P.test_drop_from);
            if (!skip) {
                j = jj;
                p = gp - jb.page_base;
                const PageShape sh = page_shape(P.g, jb, p, P.tl);
                t = sh.t;
                ntiles = sh.ntiles;
                pad = sh.pad;
                rec = jb.blob + (uint64_t)p * P.g.R;
                if (MODE == kPack) phys = jb.page_table[p];
            }
        }
        uint32_t nmax = ntiles;  // 0 in the lanes without a page
        nmax = max(nmax, __shfl_xor_sync(0xffffffffu, nmax, 1));
        nmax = max(nmax, __shfl_xor_sync(0xffffffffu, nmax, 2));
        nmax = __shfl_sync(0xffffffffu, nmax, 0);
        if (nmax == 0u) continue;
        pad += (nmax - ntiles) * QB;  // a shorter record starts later: whole tiles of zeros in front
        GK_TRACE_EVT(P, 0, 2);
        const uint32_t slot = n_adm % (uint32_t)(STAGES + 1);
        ++n_adm;
        const Chunks ch = chunks_of(P.g, t);
        for (uint32_t k = 0; k < nmax; ++k, ++n) {
            const uint32_t s = n % STAGES;
            const uint32_t use = n / STAGES;
            if (use > 0u) mbar_wait(ring.empty0 + 8u * s, (use - 1u) & 1u, abort_flag, P.w.error, 0x100u | MODE,
                                    P.w.wait_limit_ns);
            if (k == 0u && lane < 4) {  // the stage's barrier publishes it with the tile
                QuadItem *q = reinterpret_cast<QuadItem *>(ring.items + slot);
                q->pages.j[lane] = j;
                q->pages.p[lane] = p;
                if (lane == 0) q->tile_count = nmax;
            }
            uint32_t lead = 0u, nreal = 0u;
            uint64_t r0 = 0;
            if (j != kNoJob) tile_range<(int)QB>(k, pad, lead, r0, nreal);
            const uint32_t sbase = ring.stage0 + s * STAGE_BYTES;
            uint8_t *sgen = ring.base + (size_t)s * STAGE_BYTES;
#pragma unroll
            for (int wq = 0; wq < 4; ++wq) {  // front padding, zeroed by all lanes
                const uint32_t lw = __shfl_sync(0xffffffffu, lead, wq);
                for (uint32_t o = lane * 16u; o < lw; o += 512u)
                    *reinterpret_cast<uint4 *>(sgen + wq * QB + o) = make_uint4(0u, 0u, 0u, 0u);
            }
            uint32_t total = nreal;  // bytes the copies of this stage will deliver
            total += __shfl_xor_sync(0xffffffffu, total, 1);
            total += __shfl_xor_sync(0xffffffffu, total, 2);
            __syncwarp();
            uint32_t aborted = 0u;
            const uint32_t bar = ring.full0 + 8u * s;
            if (lane == 0) {
                ring.tag[s] = make_uint2(slot, k);
                aborted = *abort_flag;
                if (!aborted) {
                    if (total == 0u) mbar_arrive(bar);
                    else mbar_arrive_expect_tx(bar, total);
                }
            }
            aborted = __shfl_sync(0xffffffffu, aborted, 0);
            if (!aborted && nreal > 0u) {  // lanes 0..3 that have a page
                const uint32_t so0 = sbase + (uint32_t)lane * QB + lead;
                if (MODE == kPack) {
                    // no scale sections in this mode: the record is its data part
                    uint64_t d0 = r0;
                    const uint64_t d1 = d0 + nreal;
                    uint32_t so = so0;
                    uint32_t chunk = (uint32_t)(d0 / ch.len);
                    uint32_t off = (uint32_t)(d0 - (uint64_t)chunk * ch.len);
                    while (d0 < d1) {
                        uint32_t nb = ch.len - off;
                        if ((uint64_t)nb > d1 - d0) nb = (uint32_t)(d1 - d0);
                        if (nb == 0u) break;  // cannot happen with a valid geometry; never spin
                        const uint8_t *ca = chunk_addr(P.cache, ch, chunk, phys, off);
                        if (GK_DEBUG_OK(P, kDbgCache, 0u, ca, nb, P.cache.data, P.cache.data_extent) &&
                            GK_DEBUG_OK(P, kDbgStage, 0u, (const void *)(uintptr_t)so, nb,
                                        (const void *)(uintptr_t)sbase, STAGE_BYTES))
                            bulk_g2s(so, ca, nb, bar);
                        else
                            mbar_complete_tx(bar, nb);
                        d0 += nb;
                        so += nb;
                        ++chunk;
                        off = 0u;
                    }
                } else {
#ifdef GK_DEBUG
                    const bool in_blob = debug_ok(P, kDbgBlob, 0u, rec + r0, nreal, P.w.jobs[j].blob,
                                                  debug_blob_bytes(P, j)) &&
                                         debug_ok(P, kDbgStage, 0u, (const void *)(uintptr_t)(lead + nreal), 0u, nullptr,
                                                  QB);
#else
                    constexpr bool in_blob = true;
#endif
                    if (!in_blob) mbar_complete_tx(bar, nreal);
                    else if (hint) bulk_g2s_hint(so0, rec + r0, nreal, bar, policy);
                    else bulk_g2s(so0, rec + r0, nreal, bar);
                }
            }
            __syncwarp();
        }
        GK_TRACE_EVT(P, 0, 3);
    }
    // tell the other roles of this CTA that there is no more work
    {
        const uint32_t s = n % STAGES;
        const uint32_t use = n / STAGES;
        if (use > 0u) mbar_wait(ring.empty0 + 8u * s, (use - 1u) & 1u, abort_flag, P.w.error, 0x100u | MODE,
                                P.w.wait_limit_ns);
        if (lane == 0) {
            ring.tag[s] = make_uint2(kEndOfWork, 0u);
            mbar_arrive(ring.full0 + 8u * s);
            abort_flag[2] = n_adm;  // tells the finisher warp how many items there are
        }
        ++n;
    }
    GK_TRACE_EVT(P, 0, 4);
    // before leaving: every load this CTA issued must have landed
    if (lane == 0) {
        for (uint32_t back = 0; back < (uint32_t)STAGES && back < n; ++back) {
            const uint32_t m = n - 1u - back;
            mbar_drain(ring.full0 + 8u * (m % STAGES), (m / STAGES) & 1u, P.w.wait_limit_ns);
        }
    }
}

// Pack with page quartets: lanes 0..3 write the tile of one record each into its blob.  Bulk
// copy groups belong to the thread that issued them, so each of the four lanes commits and
// awaits its own; lane 0 hands the stage back once all four have read it.
template <int STAGE_BYTES, int STAGES>
__device__ __forceinline__ void storer_role_quad(const StreamParams &P, const Ring &ring, volatile uint32_t *abort_flag,
                                                 int lane)
{
    constexpr uint32_t QB = STAGE_BYTES / 4;
    uint32_t n = 0;
    bool live = false;  // this lane has a page of the current item
    uint8_t *rec = nullptr;
    uint32_t pad = 0u;
#ifdef GK_DEBUG
    uint32_t cur_j = 0u;
#endif
    for (;; ++n) {
        const uint32_t s = n % STAGES;
        bool ok = mbar_wait(ring.full0 + 8u * s, (n / STAGES) & 1u, abort_flag, P.w.error, 0x300u | kPack,
                            P.w.wait_limit_ns);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;  // the CTA has given up: nothing more is stored (decided by the whole warp)
        const uint2 tag = ring.tag[s];
        if (tag.x == kEndOfWork) break;
        GK_TRACE_EVT(P, 3, 0);
        if (tag.y == 0u) {  // first tile of an item: where this lane's record lies
            const QuadItem &q = *reinterpret_cast<const QuadItem *>(ring.items + tag.x);
            live = false;
            if (lane < 4 && q.pages.j[lane] != kNoJob) {
                const JobDev jb = P.w.jobs[q.pages.j[lane]];
                const uint32_t p = q.pages.p[lane];
                const PageShape sh = page_shape(P.g, jb, p, P.tl);
                pad = sh.pad + (q.tile_count - sh.ntiles) * QB;
                rec = jb.blob + (uint64_t)p * P.g.R;
                live = true;
#ifdef GK_DEBUG
                cur_j = q.pages.j[lane];
#endif
            }
        }
        if (live && *abort_flag == 0u) {
            uint32_t lead, nreal;
            uint64_t r0;
            tile_range<(int)QB>(tag.y, pad, lead, r0, nreal);
            if (nreal > 0u) {
#ifdef GK_DEBUG
                if (debug_ok(P, kDbgBlob, 3u, rec + r0, nreal, P.w.jobs[cur_j].blob, debug_blob_bytes(P, cur_j)))
#endif
                    bulk_s2g(rec + r0, ring.stage0 + s * STAGE_BYTES + (uint32_t)lane * QB + lead, nreal);
            }
        }
        if (lane < 4) {
            bulk_commit();
            if (n > 0u) bulk_wait_read<1>();
        }
        __syncwarp();
        if (lane == 0 && n > 0u) mbar_arrive(ring.empty0 + 8u * ((n - 1u) % STAGES));
    }
    if (lane < 4) bulk_wait_all();
    __syncwarp();
    if (lane == 0 && n > 0u) mbar_arrive(ring.empty0 + 8u * ((n - 1u) % STAGES));
    GK_TRACE_EVT(P, 3, 2);
}

// ----------------------------- consumer role -----------------------------
// NT threads.  Reduce each segment to one partial remainder per warp (see the
// top of this file) and hand these over to the loader warp of the ring, which
// finishes the segment (finish_segment) while the consumers start on the next.
//
// QUAD (page quartets): every warp reduces a record of its own -- 32 threads per
// record, the warp's quarter of every stage -- and hands over that record's
// remainder; nothing is merged across warps.
template <int MODE, int NT, int STAGE_BYTES, int STAGES, bool OWN_FINISHER, bool QUAD = false>
__device__ __forceinline__ void consumer_role(const StreamParams &P, const Ring &ring,
                                              volatile uint32_t *abort_flag, int tid, int warp, int lane)
{
    static_assert(!QUAD || NT == 128, "page quartets: four consumer warps");
    constexpr int kRecThreads = QUAD ? 32 : NT;                         // threads that share a record
    constexpr int kTileBytes = QUAD ? STAGE_BYTES / 4 : STAGE_BYTES;    // bytes of a stage they share
    const uint64_t kt = P.w.thread_const[QUAD ? QuadConst<NT>::kLane0 + lane : tid];
    const uint8_t *my_base = QUAD ? ring.base + (size_t)warp * kTileBytes : ring.base;
    const int my_tid = QUAD ? lane : tid;
    Finisher fin;  // kernels without a finisher warp: consumer warp 0 finishes the segments itself
    if (!OWN_FINISHER && warp == 0) finisher_init<NT, QUAD>(P, fin, lane);
    RingPos pos;
    uint32_t parity_red = 0;
    uint32_t n_done = 0;  // segments handed over so far
#ifdef GK_TRACE
    uint32_t trace_items = 0;
    unsigned long long tr_sum[4] = {0, 0, 0, 0}, tr_t0 = 0, tr_t1 = 0, tr_t2 = 0, tr_t3 = 0;
#endif
    constexpr int kTilesPerGran = (kRecThreads * 256) / kTileBytes;
    for (;;) {
#ifdef GK_TRACE
        tr_t0 = global_timer_ns();
#endif
        // the first tile of the next item (or the end mark) says what comes next
        const bool ok = mbar_wait(ring.full0 + 8u * pos.stage, pos.phase, abort_flag, P.w.error, 0x400u | MODE,
                                  P.w.wait_limit_ns);
        // leaving must be a decision of all NT consumer threads, or the barrier below would hang
        uint32_t any_failed;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.u32 q, %1, 0;\n\t"
            "barrier.red.or.pred p, 2, %2, q;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(any_failed)
            : "r"(ok ? 0u : 1u), "n"(NT)
            : "memory");
        if (any_failed) break;
        const uint32_t slot = ring.tag[pos.stage].x;
        if (slot == kEndOfWork) break;
        GK_TRACE_EVT(P, 2, 0);
#ifdef GK_TRACE
        tr_t1 = global_timer_ns();
#endif
        const uint32_t ngran = (QUAD ? reinterpret_cast<const QuadItem *>(ring.items + slot)->tile_count
                                     : ring.items[slot].tile_count) / kTilesPerGran;
        QuadAhead ahead;
        if (QUAD && !OWN_FINISHER && warp == 0)
            ahead = quad_ahead(P, reinterpret_cast<const QuadItem *>(ring.items + slot)->pages, lane);
        uint32_t R[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) R[i] = 0u;
        for (uint32_t gi = 0; gi < ngran; ++gi)
            GranuleSteps<0, MODE, kRecThreads, STAGE_BYTES, STAGES, kTileBytes>::run(
                R, my_base, ring.full0, ring.empty0, pos, abort_flag, P.w.error, P.w.wait_limit_ns, my_tid, lane);
        GK_TRACE_EVT(P, 2, 1);
#ifdef GK_TRACE
        tr_t2 = global_timer_ns();
#endif
        // merge streams -> thread -> warp -> CTA
        uint32_t a0, a1, a2, over0, over1;
        thread_poly<kRecThreads>(R, a0, a1, a2);
        const uint64_t v = warp_remainder(a0, a1, a2, kt, lane, over0, over1);
        uint64_t *rslot = ring.red + kHandOverWords * parity_red;
        uint32_t *oslot = reinterpret_cast<uint32_t *>(rslot + 4);  // [2 * NT / 32] words sticking out above the warps
        if (OWN_FINISHER) {
            // hand the segment over to the finisher warp and go on with the next one
            if (n_done >= 2u)  // the slot's previous segment must have been taken
                mbar_wait(ring.tail0 + 8u * (2u + parity_red), ((n_done >> 1) - 1u) & 1u, abort_flag, P.w.error,
                          0x600u | MODE, P.w.wait_limit_ns);
            if (lane == 0) {
                rslot[warp] = v;
                oslot[2 * warp] = over0;
                oslot[2 * warp + 1] = over1;
                // what the finisher needs to know about the item (its slot in the ring may be gone by then)
                if (warp == 0) {
                    if (QUAD)
                        *reinterpret_cast<QuadPages *>(rslot + 8) =
                            reinterpret_cast<const QuadItem *>(ring.items + slot)->pages;
                    else
                        *reinterpret_cast<HandOver *>(rslot + 8) = hand_over_of(ring.items[slot]);
                }
                mbar_arrive(ring.tail0 + 8u * parity_red);
            }
            GK_TRACE_EVT(P, 2, 2);
        } else {
            // no finisher warp in this kernel: warp 0 finishes the segment once all warps have left their
            // parts; the others go on (the two slots alternate, and the barrier of the next segment keeps
            // them from getting two segments ahead of warp 0)
            if (lane == 0) {
                rslot[warp] = v;
                oslot[2 * warp] = over0;
                oslot[2 * warp + 1] = over1;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory");
            GK_TRACE_EVT(P, 2, 2);
            if (warp == 0) {
                if constexpr (QUAD)
                    finish_quad<MODE>(P, ring, fin, reinterpret_cast<const QuadItem *>(ring.items + slot)->pages, 0u,
                                      abort_flag, lane, &ahead);
                else
                    finish_segment<MODE, NT>(P, ring, fin, hand_over_of(ring.items[slot]), 0u, abort_flag, lane);
            }
        }
#ifdef GK_TRACE
        tr_t3 = global_timer_ns();
#endif
#ifdef GK_TRACE
        {
            // steady state: when this CTA's 16th and 48th item were finished, and where the time between went
            if (++trace_items == 16u) GK_TRACE_EVT(P, 2, 5);
            if (trace_items > 16u && trace_items <= 48u) {
                const unsigned long long now = global_timer_ns();
                tr_sum[0] += tr_t1 - tr_t0;  // waiting for the item's first tile
                tr_sum[1] += tr_t2 - tr_t1;  // main loop
                tr_sum[2] += tr_t3 - tr_t2;  // epilogue up to the hand-over
                tr_sum[3] += now - tr_t3;
            }
            if (trace_items == 48u) {
                GK_TRACE_EVT(P, 2, 6);
                if (P.trace && threadIdx.x == 0)
                    for (int k = 0; k < 4; ++k) P.trace[((size_t)blockIdx.x * 4 + 2) * 16 + 8 + k] = tr_sum[k] + 1ull;
            }
        }
#endif
        ++n_done;
        parity_red ^= 1u;
    }
}

__device__ __forceinline__ void ring_init(Ring &ring, uint8_t *base, uint64_t *bars, uint2 *tags, Item *items,
                                          int stages, uint32_t empty_count, uint64_t *red = nullptr,
                                          uint64_t *tail_bars = nullptr, uint32_t consumer_warps = 0)
{
    ring.base = base;
    ring.tag = tags;
    ring.items = items;
    ring.red = red;
    ring.tail0 = tail_bars ? smem_u32(tail_bars) : 0u;
    if (threadIdx.x == 0 && tail_bars) {
        for (int k = 0; k < 2; ++k) {
            mbar_init(ring.tail0 + 8u * k, consumer_warps);  // posted: one arrival per consumer warp
            mbar_init(ring.tail0 + 8u * (2 + k), 1u);        // taken: the loader warp
        }
    }
    ring.stage0 = smem_u32(base);
    ring.full0 = smem_u32(bars);
    ring.empty0 = smem_u32(bars + stages);
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(ring.full0 + 8u * s, 1u);
            mbar_init(ring.empty0 + 8u * s, empty_count);
        }
        for (int s = 0; s <= stages; ++s) items[s].j = kNoJob;
    }
}

// pack, verify-only and commit-only launches
template <int MODE, int NT, int STAGE_BYTES, int STAGES, int MINB, bool QUAD = false>
__global__ void __launch_bounds__(StreamCfg<MODE, NT, STAGE_BYTES, STAGES>::kThreads, MINB)
    stream_kernel(const __grid_constant__ StreamParams P)
{
    static_assert(!QUAD || MODE == kPack || MODE == kVerify, "page quartets: packing, verifying, and the fused restore");
    using Cfg = StreamCfg<MODE, NT, STAGE_BYTES, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 15) & ~(uintptr_t)15);  // bulk copies need 16 bytes
    uint64_t *bars = (uint64_t *)(smem + (size_t)STAGES * STAGE_BYTES);
    uint64_t *red = bars + 2 * STAGES;                 // [2][kHandOverWords]
    uint64_t *tail_bars = red + 2 * kHandOverWords;    // [4]
    volatile uint32_t *abort_flag = (volatile uint32_t *)(tail_bars + 4);
    uint2 *tags = (uint2 *)(tail_bars + 6);
    Item *items = (Item *)(tags + STAGES);
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    Ring ring;
    ring_init(ring, smem, bars, tags, items, STAGES, (uint32_t)(Cfg::kConsWarps + (Cfg::kStore ? 1 : 0)), red,
              Cfg::kOwnFinisher ? tail_bars : nullptr, (uint32_t)Cfg::kConsWarps);
    if (threadIdx.x == 0) {
        abort_flag[0] = 0u;
        abort_flag[1] = 0u;           // the commit loader's sign of life while it waits for a job
        abort_flag[2] = 0xffffffffu;  // segments of this CTA: not known yet (finisher warp)
        fence_mbar_init();
    }
    GK_TRACE_EVT(P, 0, 0);
    grid_dependency_wait();  // everything above is CTA-local; the tables of the call are read below
    GK_TRACE_EVT(P, 0, 5);
    __syncthreads();

    if (warp == Cfg::kLoaderWarp) {
        if (MODE == kCommit)
            loader_role<MODE, 0, STAGE_BYTES, STAGES, false, true>(P, P.tlc, P.n_items_c, P.w.work_ctr + 1, P.ctr_base_c,
                                                                   ring, abort_flag, lane);
        else if constexpr (QUAD)
            loader_role_quad<MODE, STAGE_BYTES, STAGES, true>(P, P.w.work_ctr, P.ctr_base_v, ring, abort_flag, lane);
        else
            loader_role<MODE, NT, STAGE_BYTES, STAGES, true, true>(P, P.tl, P.n_items, P.w.work_ctr, P.ctr_base_v, ring,
                                                                   abort_flag, lane);
    } else if (Cfg::kStore && warp == Cfg::kStorerWarp) {
        if constexpr (QUAD)
            storer_role_quad<STAGE_BYTES, STAGES>(P, ring, abort_flag, lane);
        else
            storer_role<MODE, STAGE_BYTES, STAGES>(P, ring, abort_flag, lane);
    } else if constexpr (Cfg::kCrc) {
        if (Cfg::kOwnFinisher && warp == Cfg::kFinisherWarp)
            finisher_role<MODE, NT, QUAD>(P, ring, abort_flag, lane);
        else
            consumer_role<MODE, NT, STAGE_BYTES, STAGES, Cfg::kOwnFinisher, QUAD>(P, ring, abort_flag, threadIdx.x, warp,
                                                                                  lane);
    }
    __syncthreads();
}

// Fused restore: the verify pipeline (loader warp + NT consumer threads) and the
// commit pipeline (loader warp + storer warp) of one CTA run side by side on
// two rings.  Verify is bound by the integer pipes, commit by DRAM, so the two
// overlap; fail-closed order is kept per job by commit_decision().
template <int NT, int VSB, int VST, int CSB, int CST>
struct RestoreCfg {
    static constexpr int kConsWarps = NT / 32;
    static constexpr int kThreads = NT + 128;
    static constexpr size_t kSmemBytes = (size_t)VST * VSB + (size_t)CST * CSB + 3 * (VST + CST) * 8 +
                                         (VST + CST + 2) * sizeof(Item) + 2 * 12 * 8 + 4 * 8 + 16 + 16;
};

template <int NT, int VSB, int VST, int CSB, int CST, int MINB, bool QUAD = false>
__global__ void __launch_bounds__(NT + 128, MINB) restore_kernel(const __grid_constant__ StreamParams P)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 15) & ~(uintptr_t)15);  // bulk copies need 16 bytes
    uint8_t *vbase = smem;
    uint8_t *cbase = smem + (size_t)VST * VSB;
    uint64_t *vbars = (uint64_t *)(cbase + (size_t)CST * CSB);
    uint64_t *cbars = vbars + 2 * VST;
    uint64_t *red = cbars + 2 * CST;                   // [2][kHandOverWords]
    uint64_t *tail_bars = red + 2 * kHandOverWords;    // [4]
    volatile uint32_t *abort_flag = (volatile uint32_t *)(tail_bars + 4);
    uint2 *vtags = (uint2 *)(tail_bars + 6);
    uint2 *ctags = vtags + VST;
    Item *vitems = (Item *)(ctags + CST);
    Item *citems = vitems + (VST + 1);
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    Ring vring, cring;
    ring_init(vring, vbase, vbars, vtags, vitems, VST, (uint32_t)(NT / 32), red, tail_bars, (uint32_t)(NT / 32));
    ring_init(cring, cbase, cbars, ctags, citems, CST, 1u);
    if (threadIdx.x == 0) {
        abort_flag[0] = 0u;
        abort_flag[1] = 0u;           // the commit loader's sign of life while it waits for a job
        abort_flag[2] = 0xffffffffu;  // segments of this CTA: not known yet (finisher warp)
        fence_mbar_init();
    }
    GK_TRACE_EVT(P, 0, 0);
#ifdef GK_TRACE
    if (P.trace && threadIdx.x == 0) {
        uint32_t smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        P.trace[((size_t)blockIdx.x * 4 + 0) * 16 + 15] = smid + 1u;
    }
#endif
    grid_dependency_wait();  // everything above is CTA-local; the tables of the call are read below
    GK_TRACE_EVT(P, 0, 5);
    __syncthreads();

    constexpr int kCons = NT / 32;
    if (warp < kCons) {
        consumer_role<kVerify, NT, VSB, VST, true, QUAD>(P, vring, abort_flag, threadIdx.x, warp, lane);
    } else if (warp == kCons) {
        if constexpr (QUAD)
            loader_role_quad<kVerify, VSB, VST, false>(P, P.w.work_ctr, P.ctr_base_v, vring, abort_flag, lane);
        else
            loader_role<kVerify, NT, VSB, VST, true, false>(P, P.tl, P.n_items, P.w.work_ctr, P.ctr_base_v, vring,
                                                            abort_flag, lane);
    } else if (warp == kCons + 1) {
        loader_role<kCommit, 0, CSB, CST, false, true>(P, P.tlc, P.n_items_c, P.w.work_ctr + 1, P.ctr_base_c, cring,
                                                       abort_flag, lane);
    } else if (warp == kCons + 2) {
        storer_role<kCommit, CSB, CST>(P, cring, abort_flag, lane);
    } else {
        finisher_role<kVerify, NT, QUAD>(P, vring, abort_flag, lane);
    }
    __syncthreads();
}

}  // namespace gk
