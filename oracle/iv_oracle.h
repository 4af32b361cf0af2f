/*
 * iv_oracle.h -- plain CPU oracle for the integrity-verification hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a slow, obviously-correct restatement of
 * what the path computes, written from the definitions:
 *   - SHA-256: FIPS 180-4 sections 4.1.2, 4.2.2, 5.1.1, 5.3.3, 6.2
 *     (the paper names SHA-256 as its digest and cites FIPS 180-4);
 *   - chunk digests: Algorithm 1 of the paper ("Streaming Model Verification"),
 *     chunk_count = ceil(|M| / C), H_i = HASH(M_i);
 *   - Merkle root: binary tree over the leaf digests in index order, a node is
 *     SHA-256(left || right) of exactly 64 bytes, an unpaired last node moves
 *     up unchanged, one leaf is its own root, zero leaves give SHA-256("");
 *   - verification: Algorithm 1's last two steps, "compare root hash with
 *     expected value", extended to the per-chunk digests of the manifest.
 *
 * Nothing here is shared with the CUDA library: no common header, table,
 * helper or constant generator.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.  All four results are exact, so
 * there is no tolerance anywhere.  Every function is pinned by the tests under
 * tests/ that are not marked gpu (FIPS vectors, hashlib, Merkle closed forms,
 * exhaustive single-bit tamper detection); nothing is "parity unpinned".
 */
#ifndef IV_ORACLE_H
#define IV_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* FIPS 180-4 section 4.2.2 / 5.3.3: the 64 round constants and the 8 initial
 * hash words, derived from the cube / square roots of the first primes by
 * integer root extraction (not a typed table).  Copies 64 resp. 8 words. */
void ivo_constants(uint32_t k_out[64], uint32_t h0_out[8]);

/* FIPS 180-4 section 6.2: SHA-256 of msg[0..len).  out = H0..H7 big-endian. */
void ivo_sha256(const uint8_t *msg, uint64_t len, uint8_t out[32]);

/* Algorithm 1, chunk loop: n = ceil(nbytes / chunk_bytes) digests, the last
 * chunk hashed at its true (shorter) length.  Returns n.  nthreads >= 1
 * splits the chunks over that many host threads (one chunk per task). */
uint64_t ivo_hash_chunks(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                         uint8_t *digests_out, int nthreads);

/* Merkle root, level by level, odd last node promoted.  leaves = n * 32 bytes. */
void ivo_merkle_root(const uint8_t *leaves, uint64_t n, uint8_t root_out[32]);

/* Same root by the recursive definition: split at the largest power of two
 * strictly below n.  Exists so the tests can check the two against each other. */
void ivo_merkle_root_recursive(const uint8_t *leaves, uint64_t n, uint8_t root_out[32]);

/* Algorithm 1 end to end plus the per-chunk comparison.  Recomputes chunk
 * digests and root from data, compares with the manifest.
 *   mismatch_idx_out : ascending indices i with digest_i != manifest digest_i,
 *                      at most idx_cap of them are written
 *   returns          : exact number of mismatching chunks (may exceed idx_cap)
 *   *root_ok_out     : 1 iff the recomputed root equals manifest_root
 *   root_out         : the recomputed root (32 bytes), may be NULL */
uint64_t ivo_verify(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                    const uint8_t *manifest_digests, const uint8_t manifest_root[32],
                    uint64_t *mismatch_idx_out, uint64_t idx_cap,
                    int *root_ok_out, uint8_t *root_out, int nthreads);

/* Per-tensor digests: digest k = SHA-256(base[offsets[k] .. offsets[k]+lengths[k])). */
void ivo_hash_ragged(const uint8_t *base, const uint64_t *offsets, const uint64_t *lengths,
                     uint64_t n, uint8_t *digests_out, int nthreads);

/* ---------------------------------------------------------------------------
 * SHA-384 variant (the digest of the paper's own listings).  FIPS 180-4 section
 * 6.5 (SHA-384 = SHA-512 with the initial value of 5.3.4, truncated to 384
 * bits), sections 4.1.3, 4.2.3, 5.1.2.  Digests are 48 bytes.  The tree rule is
 * the same with SHA-384 as the node hash: parent = SHA-384(left || right) over
 * exactly 96 bytes, odd last node promoted, zero leaves give SHA-384("").
 * ------------------------------------------------------------------------- */
void ivo_constants512(uint64_t k_out[80], uint64_t h0_384_out[8]);
void ivo_sha384(const uint8_t *msg, uint64_t len, uint8_t out[48]);
uint64_t ivo_hash_chunks_sha384(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                                uint8_t *digests_out, int nthreads);
void ivo_merkle_root_sha384(const uint8_t *leaves, uint64_t n, uint8_t root_out[48]);

/* ---------------------------------------------------------------------------
 * SHA-512 variant: FIPS 180-4 section 6.4 with the initial value of section
 * 5.3.5, no truncation; digests are 64 bytes.  Tree rule as above with
 * parent = SHA-512(left || right) over exactly 128 bytes.
 * ------------------------------------------------------------------------- */
void ivo_h0_sha512(uint64_t h0_out[8]);
void ivo_sha512(const uint8_t *msg, uint64_t len, uint8_t out[64]);
uint64_t ivo_hash_chunks_sha512(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                                uint8_t *digests_out, int nthreads);
void ivo_merkle_root_sha512(const uint8_t *leaves, uint64_t n, uint8_t root_out[64]);

/* ---------------------------------------------------------------------------
 * RFC 6962 section 2.1 mode (the paper cites RFC 6962 for its tree): the Merkle
 * Tree Hash with domain separation over SHA-256, the entries being the chunks.
 * leaf = SHA-256(0x00 || chunk), node = SHA-256(0x01 || left || right), split
 * at the largest power of two below n, empty list = SHA-256("").
 * ------------------------------------------------------------------------- */
uint64_t ivo_hash_chunks_rfc6962(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                                 uint8_t *leaf_hashes_out, int nthreads);
void ivo_merkle_root_rfc6962(const uint8_t *leaf_hashes, uint64_t n, uint8_t root_out[32]);

#ifdef __cplusplus
}
#endif
#endif
