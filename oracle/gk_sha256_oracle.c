/*
 * gk_sha256_oracle.c -- CPU oracle (test infrastructure only; see the header).
 *
 * SHA-256 written from FIPS 180-4, one loop per clause of the standard; the
 * fingerprint and digest messages are assembled in a buffer and hashed whole.
 */
#include "gk_sha256_oracle.h"

#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------
 * Constants (FIPS 180-4, 4.2.2 and 5.3.3): the first 32 bits of the fractional
 * parts of the cube roots (K) and square roots (H0) of the first primes.
 * floor(root(p) * 2^32) is the integer root of p * 2^96 (cube) or p * 2^64
 * (square); its low 32 bits are the fractional bits wanted.
 * ---------------------------------------------------------------------- */
typedef unsigned __int128 u128;

static uint32_t g_k[64], g_h0[8];
static int g_ready = 0;

static uint64_t int_root(u128 v, int degree)
{
    uint64_t lo = 0, hi = (degree == 3) ? ((uint64_t)1 << 36) : ((uint64_t)1 << 38);
    while (lo < hi) { /* largest x with x^degree <= v */
        uint64_t mid = lo + (hi - lo + 1) / 2;
        u128 pw = (u128)mid * mid;
        if (degree == 3)
            pw *= mid;
        if (pw <= v)
            lo = mid;
        else
            hi = mid - 1;
    }
    return lo;
}

static void constants_init(void)
{
    uint32_t primes[64];
    uint32_t count = 0;
    for (uint32_t c = 2; count < 64; ++c) {
        int is_prime = 1;
        for (uint32_t d = 2; d * d <= c; ++d)
            if (c % d == 0)
                is_prime = 0;
        if (is_prime)
            primes[count++] = c;
    }
    for (int i = 0; i < 64; ++i)
        g_k[i] = (uint32_t)int_root((u128)primes[i] << 96, 3);
    for (int i = 0; i < 8; ++i)
        g_h0[i] = (uint32_t)int_root((u128)primes[i] << 64, 2);
    g_ready = 1;
}

void ok_sha256_constants(uint32_t k[64], uint32_t h0[8])
{
    if (!g_ready)
        constants_init();
    memcpy(k, g_k, sizeof g_k);
    memcpy(h0, g_h0, sizeof g_h0);
}

/* ------------------------------------------------------------------------
 * Functions of 4.1.2.
 * ---------------------------------------------------------------------- */
static uint32_t rotr(uint32_t x, unsigned n) { return (x >> n) | (x << (32u - n)); }
static uint32_t ch(uint32_t x, uint32_t y, uint32_t z) { return (x & y) ^ (~x & z); }
static uint32_t maj(uint32_t x, uint32_t y, uint32_t z) { return (x & y) ^ (x & z) ^ (y & z); }
static uint32_t big_sigma0(uint32_t x) { return rotr(x, 2) ^ rotr(x, 13) ^ rotr(x, 22); }
static uint32_t big_sigma1(uint32_t x) { return rotr(x, 6) ^ rotr(x, 11) ^ rotr(x, 25); }
static uint32_t small_sigma0(uint32_t x) { return rotr(x, 7) ^ rotr(x, 18) ^ (x >> 3); }
static uint32_t small_sigma1(uint32_t x) { return rotr(x, 17) ^ rotr(x, 19) ^ (x >> 10); }

/* 6.2.2: one 512-bit block */
static void compress(uint32_t H[8], const uint8_t block[64])
{
    uint32_t W[64];
    for (int t = 0; t < 16; ++t)
        W[t] = ((uint32_t)block[4 * t] << 24) | ((uint32_t)block[4 * t + 1] << 16) |
               ((uint32_t)block[4 * t + 2] << 8) | (uint32_t)block[4 * t + 3];
    for (int t = 16; t < 64; ++t)
        W[t] = small_sigma1(W[t - 2]) + W[t - 7] + small_sigma0(W[t - 15]) + W[t - 16];
    uint32_t a = H[0], b = H[1], c = H[2], d = H[3], e = H[4], f = H[5], g = H[6], h = H[7];
    for (int t = 0; t < 64; ++t) {
        uint32_t T1 = h + big_sigma1(e) + ch(e, f, g) + g_k[t] + W[t];
        uint32_t T2 = big_sigma0(a) + maj(a, b, c);
        h = g;
        g = f;
        f = e;
        e = d + T1;
        d = c;
        c = b;
        b = a;
        a = T1 + T2;
    }
    H[0] += a; H[1] += b; H[2] += c; H[3] += d;
    H[4] += e; H[5] += f; H[6] += g; H[7] += h;
}

void ok_sha256(const uint8_t *data, size_t len, uint8_t out[32])
{
    if (!g_ready)
        constants_init();
    /* 5.1.1: message || 0x80 || zeros || 64-bit big-endian bit length, a multiple of 64 bytes */
    size_t padded = ((len + 9 + 63) / 64) * 64;
    uint8_t *m = (uint8_t *)calloc(padded, 1);
    if (len)
        memcpy(m, data, len);
    m[len] = 0x80;
    uint64_t bits = (uint64_t)len * 8u;
    for (int i = 0; i < 8; ++i)
        m[padded - 1 - i] = (uint8_t)(bits >> (8 * i));
    uint32_t H[8];
    memcpy(H, g_h0, sizeof H);
    for (size_t off = 0; off < padded; off += 64)
        compress(H, m + off);
    for (int i = 0; i < 8; ++i) {
        out[4 * i] = (uint8_t)(H[i] >> 24);
        out[4 * i + 1] = (uint8_t)(H[i] >> 16);
        out[4 * i + 2] = (uint8_t)(H[i] >> 8);
        out[4 * i + 3] = (uint8_t)H[i];
    }
    free(m);
}

/* ------------------------------------------------------------------------
 * Message assembly helpers.
 * ---------------------------------------------------------------------- */
static uint8_t *put(uint8_t *w, const void *src, size_t n)
{
    if (n)
        memcpy(w, src, n);
    return w + n;
}

static uint8_t *put_le(uint8_t *w, uint64_t v, int bytes)
{
    for (int i = 0; i < bytes; ++i)
        *w++ = (uint8_t)(v >> (8 * i));
    return w;
}

/* ------------------------------------------------------------------------
 * Fingerprints.
 * ---------------------------------------------------------------------- */
int ok_fingerprints(uint32_t n, const uint8_t *data, const uint64_t *offsets, const int32_t *parent,
                    const uint8_t model[32], const uint8_t tenant[32], uint8_t *keys)
{
    if (parent)
        for (uint32_t i = 0; i < n; ++i)
            if (parent[i] >= 0 && (uint32_t)parent[i] >= i)
                return -1;
    for (uint32_t i = 0; i < n; ++i) {
        uint64_t len = offsets[i + 1] - offsets[i];
        uint8_t *msg = (uint8_t *)malloc((size_t)len + 76);
        uint8_t *w = put(msg, data + offsets[i], (size_t)len);
        w = put(w, model, 32);
        w = put(w, tenant, 32);
        w = put_le(w, len, 8);
        w = put(w, "GKF1", 4);
        uint8_t inner[32];
        ok_sha256(msg, (size_t)(w - msg), inner);
        free(msg);

        uint8_t chain[68];
        uint8_t zero[32] = {0};
        const uint8_t *pk = (parent && parent[i] >= 0) ? keys + 32u * (uint32_t)parent[i] : zero;
        w = put(chain, pk, 32);
        w = put(w, inner, 32);
        w = put(w, "GKF2", 4);
        ok_sha256(chain, 68, keys + 32u * i);
    }
    return 0;
}

/* ------------------------------------------------------------------------
 * Blob digest: leaves of 4096 record bytes, one node per page, one root.
 * ---------------------------------------------------------------------- */
void ok_blob_digest(const ok_geom *g, const uint8_t *blob, uint32_t n_tokens, const uint8_t key[32],
                    uint8_t *page_digests, uint8_t out[32])
{
    uint32_t P = 0;
    ok_blob_size(g, n_tokens, NULL, &P);
    uint8_t *root_msg = (uint8_t *)malloc((size_t)P * 32 + 44);
    uint8_t *rw = root_msg;
    for (uint32_t p = 0; p < P; ++p) {
        const uint8_t *rec = blob + ok_record_offset(g, p);
        uint64_t len = ok_record_bytes(g, n_tokens, p);
        uint64_t m = (len + OK_DIGEST_CHUNK - 1) / OK_DIGEST_CHUNK;
        uint8_t *page_msg = (uint8_t *)malloc((size_t)m * 32 + 12);
        uint8_t *pw = page_msg;
        for (uint64_t c = 0; c < m; ++c) {
            uint64_t lo = c * OK_DIGEST_CHUNK;
            uint64_t n = (len - lo < OK_DIGEST_CHUNK) ? len - lo : OK_DIGEST_CHUNK;
            uint8_t leaf_msg[OK_DIGEST_CHUNK + 4];
            uint8_t *lw = put(leaf_msg, rec + lo, (size_t)n);
            lw = put(lw, "GKL0", 4);
            ok_sha256(leaf_msg, (size_t)(lw - leaf_msg), pw);
            pw += 32;
        }
        pw = put_le(pw, len, 8);
        pw = put(pw, "GKP0", 4);
        ok_sha256(page_msg, (size_t)(pw - page_msg), rw);
        if (page_digests)
            memcpy(page_digests + 32u * p, rw, 32);
        rw += 32;
        free(page_msg);
    }
    rw = put(rw, key, 32);
    rw = put_le(rw, n_tokens, 4);
    rw = put_le(rw, P, 4);
    rw = put(rw, "GKB0", 4);
    ok_sha256(root_msg, (size_t)(rw - root_msg), out);
    free(root_msg);
}
