/*
 * gk_sha256_oracle.h -- CPU oracle for the block fingerprint and the blob digest.
 *
 * TEST INFRASTRUCTURE ONLY, like gk_oracle.h: the plain definition that the CUDA
 * library is compared against; no code, table or constant is shared with it.
 *
 * What it follows.  In the paper the lookup key of a block's stored KV state is
 * derived from three things: the block's input, byte for byte, the identity of
 * the model, and the identity of the tenant (Section 2.2); the library will not
 * run without the latter two, which keeps one model's or tenant's records out of
 * another's reach (Section 2.1); a block is reused only at identical token
 * positions (Section 2.2, Section 5); and the paper
 * lists a confirmation hash among its safety mechanisms (Section 3, sabotage
 * testing); Section 7 names hashes, besides comparing bytes, as the judge of
 * whether loaded state is right.  The paper gives no formats, so the messages below are
 * this build's own; the hash is SHA-256 as FIPS 180-4 defines it.
 *
 * Definitions (|| is concatenation, integers little-endian)
 *   inner_i = SHA-256( bytes_i || model[32] || tenant[32] || u64(len_i) || "GKF1" )
 *   key_i   = SHA-256( parent_key || inner_i || "GKF2" )
 *             parent_key = key_{parent[i]}, or 32 zero bytes when parent[i] < 0;
 *             parent[i] < i.  The chain makes a key depend on everything before
 *             the block in its prompt, i.e. on the block's token positions.
 *   leaf    = SHA-256( chunk || "GKL0" )            chunk = 4096 record bytes (the last may be shorter)
 *   page_p  = SHA-256( leaf_0 || ... || leaf_{m-1} || u64(record bytes) || "GKP0" )
 *   digest  = SHA-256( page_0 || ... || page_{P-1} || key[32] || u32(n_tokens) || u32(P) || "GKB0" )
 *             the confirmation hash of a stored block: it covers every record
 *             byte and the key the block is filed under.
 *
 * Pins: tests/test_oracle_sha256_pins.py.
 */
#ifndef GK_SHA256_ORACLE_H
#define GK_SHA256_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#include "gk_oracle.h"

#ifdef __cplusplus
extern "C" {
#endif

#define OK_DIGEST_CHUNK 4096u

/* SHA-256 (FIPS 180-4, sections 4.1.2, 4.2.2, 5.1.1, 5.3.3, 6.2).  The round
 * constants and the initial hash value are derived from the primes as 4.2.2 and
 * 5.3.3 define them, not typed in. */
void ok_sha256(const uint8_t *data, size_t len, uint8_t out[32]);
/* The constants themselves, for the pins: k[64], h0[8]. */
void ok_sha256_constants(uint32_t k[64], uint32_t h0[8]);

/* Keys of n messages; message i is data[offsets[i] .. offsets[i+1]).  parent
 * may be NULL (no chains).  Returns -1 (nothing written) unless parent[i] < i. */
int ok_fingerprints(uint32_t n, const uint8_t *data, const uint64_t *offsets, const int32_t *parent,
                    const uint8_t model[32], const uint8_t tenant[32], uint8_t *keys /* n*32 */);

/* Digest of a blob of n_tokens filed under key; page_digests (P*32 bytes) may be NULL. */
void ok_blob_digest(const ok_geom *g, const uint8_t *blob, uint32_t n_tokens, const uint8_t key[32],
                    uint8_t *page_digests, uint8_t out[32]);

#ifdef __cplusplus
}
#endif
#endif
