// gk_device.cuh -- device-side structures and primitives shared by the kernels
// of libgk (sm_100a only).  Not part of the public interface.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace gk {

// CRC-64/XZ generator polynomial without its x^64 term (bit k = coefficient of x^k).
constexpr uint64_t kPoly = 0x42F0E1EBA9EA3693ull;
constexpr int32_t kNoPage = 0x7fffffff;
constexpr uint32_t kUndecided = 0xffffffffu;  // job_latch: the job's commit decision has not been taken yet

// bounded device waits: by default give up after this many nanoseconds of %globaltimer
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

enum Mode : int { kVerify = 0, kPack = 1, kCommit = 2, kSingle = 3 };

struct GeomDev {
    uint32_t layers, kv_heads, page_tokens, scale_kv;
    uint32_t row;   // bytes of one token row of one slab: kv_heads*head_dim*elem
    uint32_t S;     // scale section bytes of a record: layers*scale_kv*kv_heads*4
    uint32_t h4;    // kv_heads*4
    uint32_t flags;
    uint32_t hrow;  // bytes of one token of one head: head_dim*elem
    uint32_t head_major;  // 1: slabs are [head][token][dim]
    uint64_t tokB;  // bytes per token in a record: 2*layers*row
    uint64_t R;     // bytes of a full page record: S + page_tokens*tokB
};

struct CacheDev {
    uint8_t *data;
    uint64_t num_pages, layer_stride, kv_stride, page_stride;
    uint8_t *scales;
    uint64_t s_layer_stride, s_kv_stride, s_page_stride;
    uint64_t data_extent, scales_extent;  // bytes from the base pointers to the end of the last slab / scale row
};

// Is [addr, addr + bytes) inside [base, base + extent)?  (The bounds-checked build asks this before
// every access to caller memory; a host test asks it, too.)
__host__ __device__ inline bool range_inside(uint64_t addr, uint64_t bytes, uint64_t base, uint64_t extent)
{
    if (addr < base) return false;
    const uint64_t off = addr - base;
    return off <= extent && bytes <= extent - off;
}

struct JobDev {
    uint8_t *blob;
    uint64_t *checksums;
    const int32_t *page_table;
    uint32_t n_tokens;
    uint32_t n_pages;
    uint32_t page_base;  // index of this job's page 0 among all pages of the call
    uint32_t missing;    // 1: blob or checksums null
};

// Workspace views for one call.  All arrays live in the context's device workspace.
struct WorkDev {
    const JobDev *jobs;
    uint32_t n_jobs;
    uint32_t page_begin;          // first page (of the call) this launch covers
    uint32_t total_pages;         // pages this launch covers
    int32_t *page_job;            // [total_pages] owning job of each page of the call
    uint64_t *page_acc;           // [total_pages] XOR of the placed segment remainders of each page
    int32_t *bad_range;           // [n_jobs] lowest out-of-range table index, or kNoPage
    int32_t *bad_dup;             // [n_jobs] lowest index of a page claimed twice, or kNoPage
    int32_t *bad_crc;             // [n_jobs] lowest page whose checksum differs, or kNoPage
    uint32_t *page_cnt;           // [total_pages] segments delivered per page (fused restore)
    uint32_t *job_done;           // [n_jobs] pages finalized per job (fused restore)
    uint32_t *job_latch;          // [n_jobs] commit decision of the job, taken once: kUndecided or a result code
    unsigned long long *claims;   // [num_pages] first claimant of each destination page
    const uint8_t *ext_mask;      // [n_jobs] or null: codes decided outside this call (gk_commit)
    uint32_t *work_ctr;           // [2] running work-item counters: CRC modes, commit mode; [2] = the
                                  // error word as the call's first kernel found it
    uint32_t *error;              // sticky: non-zero once a bounded wait has run out
    const uint64_t *init_term;    // [page_tokens+1] ones * x^(8*len(t)) mod P
    const uint64_t *thread_const; // [NT] x^(32*(NT-1-t)+64) mod P, then for each warp w of NT/32 the constants
                                  // of the two words above it: x^(1024*(NT/32-w)+64) and that times x^32;
                                  // then the same for a record that ONE warp reduces (page quartets): 32
                                  // lane constants x^(32*(31-lane)+64) and x^(1024+64), x^(1024+96)
    const uint64_t *seg_pow;      // [nseg_max][2] (x^(8*segment bytes))^k mod P and that times x^32: place
                                  // the two halves of a segment remainder
    unsigned long long wait_limit_ns;  // time limit of every device-side wait
};

// How a page record is cut into tiles and segments.  A record of `len` bytes is
// zero-padded AT THE FRONT to a multiple of gran_bytes (leading zeros do not
// change a remainder), cut into tiles of stage_bytes and grouped into segments
// of seg_tiles tiles; the short segment, if any, is the first one.
//
// Page quartets (quad = 1; small records in large calls): a work item is FOUR
// consecutive pages of the launch, one per consumer warp, every record whole
// (one segment); stage_bytes is then the quarter of a shared-memory stage that
// one record's tile takes, and a launch of n pages has (n + 3) / 4 items.
struct Tiling {
    uint32_t stage_bytes;  // a power of two
    uint32_t gran_bytes;   // a power of two, a multiple of stage_bytes
    uint32_t seg_tiles;
    uint32_t nseg_max;   // segments of a full page
    uint32_t quad = 0;
};

struct PageShape {
    uint32_t t;        // tokens in the page
    uint64_t len;      // record bytes
    uint32_t pad;      // leading zero bytes
    uint32_t ntiles;
    uint32_t nseg;
    uint32_t ntiles0;  // tiles in segment 0
};

__device__ __forceinline__ uint32_t page_fill(const GeomDev &g, const JobDev &jb, uint32_t p)
{
    return (p + 1u < jb.n_pages) ? g.page_tokens : jb.n_tokens - (jb.n_pages - 1u) * g.page_tokens;
}

// Shape of the record of a page that holds t tokens.
__device__ __forceinline__ PageShape page_shape_t(const GeomDev &g, uint32_t t, const Tiling &tl)
{
    PageShape s;
    s.t = t;
    s.len = (uint64_t)g.S + (uint64_t)s.t * g.tokB;
    // gran_bytes and stage_bytes are powers of two: masks and shifts, no 64-bit division
    const uint64_t v = (s.len + tl.gran_bytes - 1) & ~(uint64_t)(tl.gran_bytes - 1u);
    s.pad = (uint32_t)(v - s.len);
    s.ntiles = (uint32_t)(v >> (31 - __clz((int)tl.stage_bytes)));
    s.nseg = (s.ntiles + tl.seg_tiles - 1u) / tl.seg_tiles;
    s.ntiles0 = s.ntiles - (s.nseg - 1u) * tl.seg_tiles;
    return s;
}

__device__ __forceinline__ PageShape page_shape(const GeomDev &g, const JobDev &jb, uint32_t p,
                                                const Tiling &tl)
{
    return page_shape_t(g, page_fill(g, jb, p), tl);
}

// ---- GF(2)[x] mod P on 64-bit values (bit k = coefficient of x^k) ----
__host__ __device__ __forceinline__ uint64_t gf_mulx(uint64_t a)
{
    return (a << 1) ^ ((a >> 63) ? kPoly : 0ull);
}

__host__ __device__ inline uint64_t gf_mul(uint64_t a, uint64_t b)
{
    uint64_t r = 0;
    for (int i = 63; i >= 0; --i) {
        r = gf_mulx(r);
        if ((b >> i) & 1ull) r ^= a;
    }
    return r;
}

// ---- PTX wrappers: mbarrier, bulk async copies (every copy has one destination CTA) ----
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Non-blocking form: try_wait may suspend the thread for a while before it answers "not yet",
// which a loop that watches two barriers cannot afford.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Waits for a barrier phase, but never for ever: after limit_ns (or at once,
// when another thread of the CTA has already given up) it records the failure in
// *abort_flag (shared) and *error (global) and returns false.  Callers carry on
// without blocking and without issuing further async copies; the host and the
// commit kernel treat a set error word as "commit nothing".  `beat` (may be
// null) is a shared counter that the role this wait depends on bumps while it is
// itself inside a bounded wait of its own: as long as it moves, the clock here
// starts afresh, so that only a partner that has gone silent counts as a failure.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          uint32_t *error, uint32_t where, unsigned long long limit_ns,
                                          const volatile uint32_t *beat = nullptr)
{
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    unsigned long long t0 = global_timer_ns();
    uint32_t last_beat = beat ? *beat : 0u;
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3ffu) == 0u) {
            const unsigned long long now = global_timer_ns();
            if (beat) {
                const uint32_t b = *beat;
                if (b != last_beat) {
                    last_beat = b;
                    t0 = now;
                }
            }
            if (*abort_flag || now - t0 > limit_ns) {
                *abort_flag = 1u;
                atomicCAS(error, 0u, where);
                return false;
            }
        }
    }
    return true;
}

// Last wait of a loader before its CTA exits: lets copies that are still in
// flight land, for a bounded time, whether or not the CTA has given up.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity, unsigned long long limit_ns)
{
    if (mbar_try_wait(bar, parity)) return;
    const unsigned long long t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3ffu) == 0u && global_timer_ns() - t0 > limit_ns / 4) return;
    }
}

// global -> shared bulk copy completing on an mbarrier.  16-byte aligned
// addresses, size a multiple of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar,
                                              uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            dst_smem),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}

// shared -> global bulk copy in the current bulk group.
__device__ __forceinline__ void bulk_s2g(void *dst, uint32_t src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem),
                 "r"(bytes)
                 : "memory");
}

// The same with an L2 eviction policy for the lines written.
__device__ __forceinline__ void bulk_s2g_hint(void *dst, uint32_t src_smem, uint32_t bytes, uint64_t policy)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(dst),
                 "r"(src_smem), "r"(bytes), "l"(policy)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void bulk_wait_all()
{
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// Counts `bytes` as arrived on a barrier without a copy (the bounds-checked build: a refused
// copy must still let the waiters go on).
__device__ __forceinline__ void mbar_complete_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.complete_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// Programmatic dependent launch.  A kernel launched with the programmatic stream
// serialization attribute may start while the kernel before it in the stream is
// still running; grid_dependency_wait() then blocks until that kernel has finished
// and its writes are visible (without the attribute it returns at once).  The
// earlier kernel calls allow_dependent_launch() to let the next one start early.
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ void allow_dependent_launch()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

__device__ __forceinline__ uint64_t policy_evict_last()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}

}  // namespace gk
