// gk_sha256.cuh -- SHA-256 kernels: block fingerprints and the digest of a blob.
//
// SHA-256 has no parallelism inside one message, so all parallelism here is across
// messages: one thread hashes one message from start to end, with the eight state
// words, a rolling 16-word message schedule and the round constants (immediates of
// the fully unrolled rounds) all in registers.  The digest of a blob is therefore a
// tree: leaves of 4096 record bytes (hundreds of thousands of independent messages
// per call, which is what fills the GPU), one node per page over its leaves, one
// root per blob over its pages.  The work is integer ALU work -- about 1,400
// instructions per 64 input bytes -- not memory work.
//
// Message formats (|| is concatenation, integers little-endian):
//   leaf   = SHA-256( chunk || "GKL0" )
//   page_p = SHA-256( leaf_0 || ... || leaf_{m-1} || u64(record bytes) || "GKP0" )
//   digest = SHA-256( page_0 || ... || page_{P-1} || key[32] || u32(n_tokens) || u32(P) || "GKB0" )
//   inner_i = SHA-256( bytes_i || model[32] || tenant[32] || u64(len_i) || "GKF1" )
//   key_i   = SHA-256( parent_key || inner_i || "GKF2" )
#pragma once

#include <cstdint>

#include "gk_device.cuh"

namespace gk {

constexpr uint32_t kDigestChunk = 4096u;

// FIPS 180-4, section 4.2.2
__device__ constexpr uint32_t kShaK[64] = {
    0x428a2f98u, 0x71374491u, 0xb5c0fbcfu, 0xe9b5dba5u, 0x3956c25bu, 0x59f111f1u, 0x923f82a4u, 0xab1c5ed5u,
    0xd807aa98u, 0x12835b01u, 0x243185beu, 0x550c7dc3u, 0x72be5d74u, 0x80deb1feu, 0x9bdc06a7u, 0xc19bf174u,
    0xe49b69c1u, 0xefbe4786u, 0x0fc19dc6u, 0x240ca1ccu, 0x2de92c6fu, 0x4a7484aau, 0x5cb0a9dcu, 0x76f988dau,
    0x983e5152u, 0xa831c66du, 0xb00327c8u, 0xbf597fc7u, 0xc6e00bf3u, 0xd5a79147u, 0x06ca6351u, 0x14292967u,
    0x27b70a85u, 0x2e1b2138u, 0x4d2c6dfcu, 0x53380d13u, 0x650a7354u, 0x766a0abbu, 0x81c2c92eu, 0x92722c85u,
    0xa2bfe8a1u, 0xa81a664bu, 0xc24b8b70u, 0xc76c51a3u, 0xd192e819u, 0xd6990624u, 0xf40e3585u, 0x106aa070u,
    0x19a4c116u, 0x1e376c08u, 0x2748774cu, 0x34b0bcb5u, 0x391c0cb3u, 0x4ed8aa4au, 0x5b9cca4fu, 0x682e6ff3u,
    0x748f82eeu, 0x78a5636fu, 0x84c87814u, 0x8cc70208u, 0x90befffau, 0xa4506cebu, 0xbef9a3f7u, 0xc67178f2u};

// FIPS 180-4, section 5.3.3
__device__ __forceinline__ void sha_init(uint32_t h[8])
{
    h[0] = 0x6a09e667u; h[1] = 0xbb67ae85u; h[2] = 0x3c6ef372u; h[3] = 0xa54ff53au;
    h[4] = 0x510e527fu; h[5] = 0x9b05688cu; h[6] = 0x1f83d9abu; h[7] = 0x5be0cd19u;
}

__device__ __forceinline__ uint32_t rotr32(uint32_t x, int n) { return __funnelshift_r(x, x, n); }
__device__ __forceinline__ uint32_t bswap32(uint32_t x) { return __byte_perm(x, 0u, 0x0123u); }

__device__ __forceinline__ uint32_t sha_xor3(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t sha_ch(uint32_t x, uint32_t y, uint32_t z)
{
    uint32_t d;  // (x & y) ^ (~x & z)
    asm("lop3.b32 %0, %1, %2, %3, 0xCA;" : "=r"(d) : "r"(x), "r"(y), "r"(z));
    return d;
}
__device__ __forceinline__ uint32_t sha_maj(uint32_t x, uint32_t y, uint32_t z)
{
    uint32_t d;  // majority
    asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(d) : "r"(x), "r"(y), "r"(z));
    return d;
}

// One 512-bit block (FIPS 180-4, section 6.2.2).  w holds the block as 16
// big-endian words and is used up as the rolling message schedule.
__device__ __forceinline__ void sha_compress(uint32_t h[8], uint32_t w[16])
{
    uint32_t a = h[0], b = h[1], c = h[2], d = h[3], e = h[4], f = h[5], g = h[6], hh = h[7];
#pragma unroll
    for (int t = 0; t < 64; ++t) {
        if (t >= 16) {
            const uint32_t w15 = w[(t - 15) & 15], w2 = w[(t - 2) & 15];
            const uint32_t s0 = sha_xor3(rotr32(w15, 7), rotr32(w15, 18), w15 >> 3);
            const uint32_t s1 = sha_xor3(rotr32(w2, 17), rotr32(w2, 19), w2 >> 10);
            w[t & 15] = w[t & 15] + s0 + w[(t - 7) & 15] + s1;
        }
        const uint32_t S1 = sha_xor3(rotr32(e, 6), rotr32(e, 11), rotr32(e, 25));
        const uint32_t T1 = hh + S1 + sha_ch(e, f, g) + kShaK[t] + w[t & 15];
        const uint32_t S0 = sha_xor3(rotr32(a, 2), rotr32(a, 13), rotr32(a, 22));
        const uint32_t T2 = S0 + sha_maj(a, b, c);
        hh = g; g = f; f = e; e = d + T1;
        d = c; c = b; b = a; a = T1 + T2;
    }
    h[0] += a; h[1] += b; h[2] += c; h[3] += d;
    h[4] += e; h[5] += f; h[6] += g; h[7] += hh;
}

// Stores a state as the 32 digest bytes (big-endian words) at a 16-byte aligned address.
__device__ __forceinline__ void sha_store(uint8_t *out, const uint32_t h[8])
{
    uint4 *o = reinterpret_cast<uint4 *>(out);
    o[0] = make_uint4(bswap32(h[0]), bswap32(h[1]), bswap32(h[2]), bswap32(h[3]));
    o[1] = make_uint4(bswap32(h[4]), bswap32(h[5]), bswap32(h[6]), bswap32(h[7]));
}

// p: any address space (the message may be a thread's own array), 16-byte aligned
__device__ __forceinline__ void sha_load_block16(const uint8_t *p, uint32_t w[16])
{
    const uint4 *q = reinterpret_cast<const uint4 *>(p);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 v = q[i];
        w[4 * i] = bswap32(v.x);
        w[4 * i + 1] = bswap32(v.y);
        w[4 * i + 2] = bswap32(v.z);
        w[4 * i + 3] = bswap32(v.w);
    }
}

// Byte `pos` of the tail of a message: the last `r` data bytes that did not fill a
// block, then the suffix, then the padding of FIPS 180-4 section 5.1.1 (0x80,
// zeros, the bit length as 8 big-endian bytes at the end of the last block).
__device__ __forceinline__ uint32_t sha_tail_byte(const uint8_t *rest, uint32_t r, const uint8_t *suffix,
                                                  uint32_t suffix_len, uint32_t tail_bytes, uint64_t bit_len,
                                                  uint32_t pos)
{
    if (pos < r) return rest[pos];
    if (pos < r + suffix_len) return suffix[pos - r];
    if (pos == r + suffix_len) return 0x80u;
    if (pos >= tail_bytes - 8u) return (uint32_t)(bit_len >> (8u * (tail_bytes - 1u - pos))) & 0xffu;
    return 0u;
}

// SHA-256( data[0..len) || suffix[0..suffix_len) ).  data needs no alignment (16-byte
// aligned data takes vector loads); suffix is the calling thread's own array.
__device__ __noinline__ void sha256_message(const uint8_t *data, uint64_t len, const uint8_t *suffix,
                                            uint32_t suffix_len, uint32_t h[8])
{
    sha_init(h);
    uint32_t w[16];
    const uint64_t full = len / 64u;
    if ((reinterpret_cast<uintptr_t>(data) & 15u) == 0u) {
        for (uint64_t b = 0; b < full; ++b) {
            sha_load_block16(data + 64u * b, w);
            sha_compress(h, w);
        }
    } else {
        for (uint64_t b = 0; b < full; ++b) {
            const uint8_t *p = data + 64u * b;
#pragma unroll
            for (int i = 0; i < 16; ++i)
                w[i] = ((uint32_t)p[4 * i] << 24) | ((uint32_t)p[4 * i + 1] << 16) | ((uint32_t)p[4 * i + 2] << 8) |
                       (uint32_t)p[4 * i + 3];
            sha_compress(h, w);
        }
    }
    const uint32_t r = (uint32_t)(len - 64u * full);
    const uint8_t *rest = data + 64u * full;
    const uint32_t tail_bytes = (r + suffix_len + 9u + 63u) / 64u * 64u;
    const uint64_t bit_len = 8u * (len + suffix_len);
    for (uint32_t base = 0; base < tail_bytes; base += 64u) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            uint32_t v = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                v = (v << 8) | sha_tail_byte(rest, r, suffix, suffix_len, tail_bytes, bit_len, base + 4u * i + k);
            w[i] = v;
        }
        sha_compress(h, w);
    }
}

__device__ __forceinline__ void put_tag(uint8_t *p, char a, char b, char c, char d)
{
    p[0] = (uint8_t)a; p[1] = (uint8_t)b; p[2] = (uint8_t)c; p[3] = (uint8_t)d;
}

__device__ __forceinline__ void put_le(uint8_t *p, uint64_t v, int bytes)
{
    for (int i = 0; i < bytes; ++i) p[i] = (uint8_t)(v >> (8 * i));
}

struct DigestParams {
    GeomDev g;
    const JobDev *jobs;
    uint32_t n_jobs;
    uint32_t total_pages;
    uint32_t m_max;          // leaves of a full page record
    uint8_t *leaves;         // [total_pages][m_max][32]
    uint8_t *page_digests;   // [total_pages][32]
    const uint8_t *keys;     // [n_jobs][32]
    uint8_t *digests;        // [n_jobs][32]
};

// the job that owns page gp of the call (jobs are in page order)
__device__ __forceinline__ uint32_t job_of_page(const JobDev *jobs, uint32_t n_jobs, uint32_t gp)
{
    uint32_t lo = 0, hi = n_jobs - 1u;
    while (lo < hi) {
        const uint32_t mid = (lo + hi + 1u) / 2u;
        if (jobs[mid].page_base <= gp) lo = mid; else hi = mid - 1u;
    }
    return lo;
}

__device__ __forceinline__ uint64_t record_len(const GeomDev &g, const JobDev &jb, uint32_t p)
{
    const uint32_t t = (p + 1u < jb.n_pages) ? g.page_tokens : jb.n_tokens - (jb.n_pages - 1u) * g.page_tokens;
    return (uint64_t)g.S + (uint64_t)t * g.tokB;
}

// One thread per leaf.  A full leaf is 64 data blocks and one constant last block
// (tag, padding, length); the next block's data is requested before the current
// block is compressed.
__global__ void __launch_bounds__(128) sha_leaf_kernel(const DigestParams P)
{
    const uint64_t tid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t gp = (uint32_t)(tid / P.m_max);
    const uint32_t c = (uint32_t)(tid - (uint64_t)gp * P.m_max);
    if (gp >= P.total_pages) return;
    const uint32_t j = job_of_page(P.jobs, P.n_jobs, gp);
    const JobDev jb = P.jobs[j];
    const uint32_t p = gp - jb.page_base;
    const uint64_t len = record_len(P.g, jb, p);
    const uint64_t lo = (uint64_t)c * kDigestChunk;
    if (lo >= len) return;
    const uint8_t *chunk = jb.blob + (uint64_t)p * P.g.R + lo;
    const uint32_t n = (len - lo < kDigestChunk) ? (uint32_t)(len - lo) : kDigestChunk;
    uint32_t h[8];
    if (n == kDigestChunk) {
        sha_init(h);
        uint32_t w[16];
        uint4 nx[4];
        const uint4 *q = reinterpret_cast<const uint4 *>(chunk);
#pragma unroll
        for (int i = 0; i < 4; ++i) nx[i] = __ldg(q + i);
        for (uint32_t b = 0; b < kDigestChunk / 64u; ++b) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                w[4 * i] = bswap32(nx[i].x);
                w[4 * i + 1] = bswap32(nx[i].y);
                w[4 * i + 2] = bswap32(nx[i].z);
                w[4 * i + 3] = bswap32(nx[i].w);
            }
            if (b + 1u < kDigestChunk / 64u) {
#pragma unroll
                for (int i = 0; i < 4; ++i) nx[i] = __ldg(q + 4u * (b + 1u) + i);
            }
            sha_compress(h, w);
        }
        // last block: "GKL0", 0x80, zeros, bit length of 4100 bytes
        w[0] = 0x474b4c30u;
        w[1] = 0x80000000u;
#pragma unroll
        for (int i = 2; i < 15; ++i) w[i] = 0u;
        w[15] = 8u * (kDigestChunk + 4u);
        sha_compress(h, w);
    } else {
        uint8_t tag[4];
        put_tag(tag, 'G', 'K', 'L', '0');
        sha256_message(chunk, n, tag, 4u, h);
    }
    sha_store(P.leaves + ((uint64_t)gp * P.m_max + c) * 32u, h);
}

// One thread per page: the node over the page's leaves.
__global__ void __launch_bounds__(64) sha_page_kernel(const DigestParams P)
{
    const uint32_t gp = blockIdx.x * blockDim.x + threadIdx.x;
    if (gp >= P.total_pages) return;
    const uint32_t j = job_of_page(P.jobs, P.n_jobs, gp);
    const JobDev jb = P.jobs[j];
    const uint64_t len = record_len(P.g, jb, gp - jb.page_base);
    const uint32_t m = (uint32_t)((len + kDigestChunk - 1u) / kDigestChunk);
    uint8_t suffix[12];
    put_le(suffix, len, 8);
    put_tag(suffix + 8, 'G', 'K', 'P', '0');
    uint32_t h[8];
    sha256_message(P.leaves + (uint64_t)gp * P.m_max * 32u, (uint64_t)m * 32u, suffix, 12u, h);
    sha_store(P.page_digests + (uint64_t)gp * 32u, h);
}

// One thread per blob: the root over its page nodes, bound to the key it is filed under.
__global__ void __launch_bounds__(64) sha_blob_kernel(const DigestParams P)
{
    const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= P.n_jobs) return;
    const JobDev jb = P.jobs[j];
    uint8_t suffix[44];
    for (int i = 0; i < 32; ++i) suffix[i] = P.keys[(uint64_t)j * 32u + i];
    put_le(suffix + 32, jb.n_tokens, 4);
    put_le(suffix + 36, jb.n_pages, 4);
    put_tag(suffix + 40, 'G', 'K', 'B', '0');
    uint32_t h[8];
    sha256_message(P.page_digests + (uint64_t)jb.page_base * 32u, (uint64_t)jb.n_pages * 32u, suffix, 44u, h);
    sha_store(P.digests + (uint64_t)j * 32u, h);
}

struct FingerprintParams {
    const uint8_t *data;
    const uint64_t *offsets;   // [n + 1]
    const int32_t *parent;     // [n] or null
    const uint32_t *depth;     // [n] length of the chain above each message (0 = no parent); null with parent
    uint32_t n;
    uint32_t max_depth;
    uint8_t model[32];
    uint8_t tenant[32];
    uint8_t *inner;            // [n][32] scratch
    uint8_t *keys;             // [n][32]
};

// One thread per message: everything of a key that does not depend on the parent.
__global__ void __launch_bounds__(64) fingerprint_inner_kernel(const __grid_constant__ FingerprintParams P)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= P.n) return;
    const uint64_t lo = P.offsets[i], len = P.offsets[i + 1] - lo;
    uint8_t suffix[76];
    for (int k = 0; k < 32; ++k) {
        suffix[k] = P.model[k];
        suffix[32 + k] = P.tenant[k];
    }
    put_le(suffix + 64, len, 8);
    put_tag(suffix + 72, 'G', 'K', 'F', '1');
    uint32_t h[8];
    sha256_message(P.data + lo, len, suffix, 76u, h);
    sha_store(P.inner + (uint64_t)i * 32u, h);
}

// One CTA.  Chains are walked level by level: in round d every message whose chain
// above it has length d takes its parent's key (finished in an earlier round) and
// hashes two blocks.  max_depth + 1 rounds, a barrier between them.
__global__ void __launch_bounds__(1024) fingerprint_chain_kernel(const __grid_constant__ FingerprintParams P)
{
    for (uint32_t d = 0; d <= P.max_depth; ++d) {
        for (uint32_t i = threadIdx.x; i < P.n; i += blockDim.x) {
            const uint32_t di = P.depth ? P.depth[i] : 0u;
            if (di != d) continue;
            uint8_t msg[64];
            const int32_t par = P.parent ? P.parent[i] : -1;
            for (int k = 0; k < 32; ++k) {
                msg[k] = par >= 0 ? P.keys[(uint64_t)par * 32u + k] : (uint8_t)0;
                msg[32 + k] = P.inner[(uint64_t)i * 32u + k];
            }
            uint8_t tag[4];
            put_tag(tag, 'G', 'K', 'F', '2');
            uint32_t h[8];
            sha256_message(msg, 64u, tag, 4u, h);
            sha_store(P.keys + (uint64_t)i * 32u, h);
        }
        __threadfence_block();
        __syncthreads();
    }
}

}  // namespace gk
