/*
 * iv_oracle.c -- plain CPU oracle (test infrastructure, see iv_oracle.h).
 *
 * Written for reading, not for speed: the message schedule is a full 64-word
 * array, the round loop is a loop, constants come from integer roots of the
 * primes.  No intrinsics, no unrolling, no code shared with the CUDA library.
 */
#include "iv_oracle.h"

#include <pthread.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

/* ------------------------------------------------------------------------- */
/* FIPS 180-4 section 4.2.2 and 5.3.3: constants from the first 64 primes.    */
/* ------------------------------------------------------------------------- */

static uint32_t g_k[64];
static uint32_t g_h0[8];
static pthread_once_t g_once = PTHREAD_ONCE_INIT;

/* floor of the square root of v, by bisection on the answer. */
static uint64_t isqrt128(u128 v)
{
    uint64_t lo = 0, hi = ((uint64_t)1 << 40);
    while (lo < hi) {
        uint64_t mid = lo + (hi - lo + 1) / 2;
        if ((u128)mid * mid <= v) lo = mid; else hi = mid - 1;
    }
    return lo;
}

/* floor of the cube root of v, by bisection on the answer. */
static uint64_t icbrt128(u128 v)
{
    uint64_t lo = 0, hi = ((uint64_t)1 << 36);
    while (lo < hi) {
        uint64_t mid = lo + (hi - lo + 1) / 2;
        if ((u128)mid * mid * mid <= v) lo = mid; else hi = mid - 1;
    }
    return lo;
}

static void derive_constants(void)
{
    int found = 0;
    for (unsigned p = 2; found < 64; ++p) {
        int prime = 1;
        for (unsigned q = 2; q * q <= p; ++q)
            if (p % q == 0) { prime = 0; break; }
        if (!prime) continue;
        /* first 32 bits of the fractional part of the root:
         * floor(root(p) * 2^32) mod 2^32 = floor(root(p * 2^(32*degree))) mod 2^32 */
        if (found < 8)
            g_h0[found] = (uint32_t)isqrt128((u128)p << 64);
        g_k[found] = (uint32_t)icbrt128((u128)p << 96);
        ++found;
    }
}

void ivo_constants(uint32_t k_out[64], uint32_t h0_out[8])
{
    pthread_once(&g_once, derive_constants);
    memcpy(k_out, g_k, sizeof g_k);
    memcpy(h0_out, g_h0, sizeof g_h0);
}

/* ------------------------------------------------------------------------- */
/* FIPS 180-4 section 4.1.2: the six logical functions.                       */
/* ------------------------------------------------------------------------- */

static uint32_t rotr(uint32_t x, unsigned n) { return (x >> n) | (x << (32u - n)); }
static uint32_t shr(uint32_t x, unsigned n) { return x >> n; }

static uint32_t ch(uint32_t x, uint32_t y, uint32_t z) { return (x & y) ^ (~x & z); }
static uint32_t maj(uint32_t x, uint32_t y, uint32_t z) { return (x & y) ^ (x & z) ^ (y & z); }
static uint32_t big_sigma0(uint32_t x) { return rotr(x, 2) ^ rotr(x, 13) ^ rotr(x, 22); }
static uint32_t big_sigma1(uint32_t x) { return rotr(x, 6) ^ rotr(x, 11) ^ rotr(x, 25); }
static uint32_t small_sigma0(uint32_t x) { return rotr(x, 7) ^ rotr(x, 18) ^ shr(x, 3); }
static uint32_t small_sigma1(uint32_t x) { return rotr(x, 17) ^ rotr(x, 19) ^ shr(x, 10); }

/* FIPS 180-4 section 6.2.2: one 512-bit block into the hash state. */
static void process_block(uint32_t hash[8], const uint8_t block[64])
{
    uint32_t w[64];
    for (int t = 0; t < 16; ++t)
        w[t] = ((uint32_t)block[4 * t] << 24) | ((uint32_t)block[4 * t + 1] << 16) |
               ((uint32_t)block[4 * t + 2] << 8) | (uint32_t)block[4 * t + 3];
    for (int t = 16; t < 64; ++t)
        w[t] = small_sigma1(w[t - 2]) + w[t - 7] + small_sigma0(w[t - 15]) + w[t - 16];

    uint32_t a = hash[0], b = hash[1], c = hash[2], d = hash[3];
    uint32_t e = hash[4], f = hash[5], g = hash[6], h = hash[7];
    for (int t = 0; t < 64; ++t) {
        uint32_t t1 = h + big_sigma1(e) + ch(e, f, g) + g_k[t] + w[t];
        uint32_t t2 = big_sigma0(a) + maj(a, b, c);
        h = g; g = f; f = e; e = d + t1;
        d = c; c = b; b = a; a = t1 + t2;
    }
    hash[0] += a; hash[1] += b; hash[2] += c; hash[3] += d;
    hash[4] += e; hash[5] += f; hash[6] += g; hash[7] += h;
}

/* FIPS 180-4 section 5.1.1 (padding) + 6.2 (digest). */
void ivo_sha256(const uint8_t *msg, uint64_t len, uint8_t out[32])
{
    pthread_once(&g_once, derive_constants);
    uint32_t hash[8];
    memcpy(hash, g_h0, sizeof hash);

    uint64_t full = len / 64;
    for (uint64_t i = 0; i < full; ++i)
        process_block(hash, msg + 64 * i);

    /* the remaining bytes, then 0x80, zeros up to 56 mod 64, then the length
     * in bits as a 64-bit big-endian integer: one or two more blocks */
    uint8_t tail[128];
    uint64_t rem = len - 64 * full;
    memset(tail, 0, sizeof tail);
    if (rem) memcpy(tail, msg + 64 * full, rem);
    tail[rem] = 0x80;
    uint64_t tail_len = (rem + 1 + 8 <= 64) ? 64 : 128;
    uint64_t bits = len * 8u;
    for (int i = 0; i < 8; ++i)
        tail[tail_len - 1 - i] = (uint8_t)(bits >> (8 * i));
    for (uint64_t off = 0; off < tail_len; off += 64)
        process_block(hash, tail + off);

    for (int i = 0; i < 8; ++i) {
        out[4 * i] = (uint8_t)(hash[i] >> 24);
        out[4 * i + 1] = (uint8_t)(hash[i] >> 16);
        out[4 * i + 2] = (uint8_t)(hash[i] >> 8);
        out[4 * i + 3] = (uint8_t)hash[i];
    }
}

/* ------------------------------------------------------------------------- */
/* A tiny "one task per index" thread pool (for the timed CPU baseline only). */
/* ------------------------------------------------------------------------- */

typedef void (*task_fn)(void *arg, uint64_t index);

typedef struct {
    task_fn fn;
    void *arg;
    uint64_t n;
    uint64_t next;
    pthread_mutex_t lock;
} task_pool;

static void *pool_worker(void *p)
{
    task_pool *pool = (task_pool *)p;
    for (;;) {
        pthread_mutex_lock(&pool->lock);
        uint64_t i = pool->next;
        if (i < pool->n) pool->next = i + 1;
        pthread_mutex_unlock(&pool->lock);
        if (i >= pool->n) return NULL;
        pool->fn(pool->arg, i);
    }
}

static void run_tasks(task_fn fn, void *arg, uint64_t n, int nthreads)
{
    if (nthreads < 1) nthreads = 1;
    if (nthreads == 1 || n <= 1) {
        for (uint64_t i = 0; i < n; ++i) fn(arg, i);
        return;
    }
    task_pool pool;
    pool.fn = fn; pool.arg = arg; pool.n = n; pool.next = 0;
    pthread_mutex_init(&pool.lock, NULL);
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    int started = 0;
    for (int t = 0; t < nthreads; ++t)
        if (pthread_create(&th[started], NULL, pool_worker, &pool) == 0) ++started;
    if (started == 0) pool_worker(&pool);
    for (int t = 0; t < started; ++t) pthread_join(th[t], NULL);
    free(th);
    pthread_mutex_destroy(&pool.lock);
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1: chunk digests.                                                */
/* ------------------------------------------------------------------------- */

typedef struct {
    const uint8_t *data;
    uint64_t nbytes, chunk_bytes;
    uint8_t *out;
} chunk_job;

static void chunk_task(void *arg, uint64_t i)
{
    chunk_job *job = (chunk_job *)arg;
    uint64_t begin = i * job->chunk_bytes;
    uint64_t end = begin + job->chunk_bytes;
    if (end > job->nbytes || end < begin) end = job->nbytes;
    ivo_sha256(job->data + begin, end - begin, job->out + 32 * i);
}

uint64_t ivo_hash_chunks(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                         uint8_t *digests_out, int nthreads)
{
    if (chunk_bytes == 0 || nbytes == 0) return 0;
    uint64_t n = nbytes / chunk_bytes + (nbytes % chunk_bytes ? 1 : 0);
    chunk_job job = { data, nbytes, chunk_bytes, digests_out };
    run_tasks(chunk_task, &job, n, nthreads);
    return n;
}

/* ------------------------------------------------------------------------- */
/* Merkle root.                                                               */
/* ------------------------------------------------------------------------- */

static void hash_pair(const uint8_t left[32], const uint8_t right[32], uint8_t out[32])
{
    uint8_t both[64];
    memcpy(both, left, 32);
    memcpy(both + 32, right, 32);
    ivo_sha256(both, 64, out);
}

void ivo_merkle_root(const uint8_t *leaves, uint64_t n, uint8_t root_out[32])
{
    if (n == 0) { ivo_sha256((const uint8_t *)"", 0, root_out); return; }
    uint8_t *level = (uint8_t *)malloc((size_t)n * 32);
    memcpy(level, leaves, (size_t)n * 32);
    while (n > 1) {
        uint64_t parents = n / 2;
        for (uint64_t j = 0; j < parents; ++j) {
            uint8_t node[32];
            hash_pair(level + 64 * j, level + 64 * j + 32, node);
            memcpy(level + 32 * j, node, 32);
        }
        if (n % 2) {                    /* unpaired last node moves up unchanged */
            memmove(level + 32 * parents, level + 32 * (n - 1), 32);
            ++parents;
        }
        n = parents;
    }
    memcpy(root_out, level, 32);
    free(level);
}

void ivo_merkle_root_recursive(const uint8_t *leaves, uint64_t n, uint8_t root_out[32])
{
    if (n == 0) { ivo_sha256((const uint8_t *)"", 0, root_out); return; }
    if (n == 1) { memcpy(root_out, leaves, 32); return; }
    uint64_t split = 1;
    while (split * 2 < n) split *= 2;   /* largest power of two strictly below n */
    uint8_t left[32], right[32];
    ivo_merkle_root_recursive(leaves, split, left);
    ivo_merkle_root_recursive(leaves + 32 * split, n - split, right);
    hash_pair(left, right, root_out);
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1 end to end: recompute, then compare with the manifest.          */
/* ------------------------------------------------------------------------- */

uint64_t ivo_verify(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                    const uint8_t *manifest_digests, const uint8_t manifest_root[32],
                    uint64_t *mismatch_idx_out, uint64_t idx_cap,
                    int *root_ok_out, uint8_t *root_out, int nthreads)
{
    uint64_t n = (chunk_bytes == 0 || nbytes == 0)
                     ? 0 : nbytes / chunk_bytes + (nbytes % chunk_bytes ? 1 : 0);
    uint8_t *digests = (uint8_t *)malloc((size_t)(n ? n : 1) * 32);
    ivo_hash_chunks(data, nbytes, chunk_bytes, digests, nthreads);

    uint64_t bad = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (memcmp(digests + 32 * i, manifest_digests + 32 * i, 32) != 0) {
            if (bad < idx_cap && mismatch_idx_out) mismatch_idx_out[bad] = i;
            ++bad;
        }
    }
    uint8_t root[32];
    ivo_merkle_root(digests, n, root);
    if (root_ok_out) *root_ok_out = memcmp(root, manifest_root, 32) == 0;
    if (root_out) memcpy(root_out, root, 32);
    free(digests);
    return bad;
}

/* ------------------------------------------------------------------------- */
/* Ragged set: one digest per (offset, length).                               */
/* ------------------------------------------------------------------------- */

typedef struct {
    const uint8_t *base;
    const uint64_t *offsets, *lengths;
    uint8_t *out;
} ragged_job;

static void ragged_task(void *arg, uint64_t k)
{
    ragged_job *job = (ragged_job *)arg;
    ivo_sha256(job->base + job->offsets[k], job->lengths[k], job->out + 32 * k);
}

void ivo_hash_ragged(const uint8_t *base, const uint64_t *offsets, const uint64_t *lengths,
                     uint64_t n, uint8_t *digests_out, int nthreads)
{
    ragged_job job = { base, offsets, lengths, digests_out };
    run_tasks(ragged_task, &job, n, nthreads);
}

/* ------------------------------------------------------------------------- */
/* SHA-384 (FIPS 180-4 sections 4.1.3, 4.2.3, 5.1.2, 5.3.4, 6.4.2, 6.5).       */
/* ------------------------------------------------------------------------- */

static uint64_t g_k512[80];
static uint64_t g_h0_384[8];
static uint64_t g_h0_512[8];
static pthread_once_t g_once512 = PTHREAD_ONCE_INIT;

/* 256-bit unsigned integers as four 64-bit limbs, least significant first: just
 * enough arithmetic to test r^2 and r^3 against p * 2^128 and p * 2^192. */
typedef struct { uint64_t w[4]; } u256;

static u256 u256_from_u128(u128 v)
{
    u256 r = { { (uint64_t)v, (uint64_t)(v >> 64), 0, 0 } };
    return r;
}

/* a * b for a below 2^192 and b below 2^128 (the product must fit 256 bits) */
static u256 u256_mul(u256 a, u128 b)
{
    const uint64_t bl[2] = { (uint64_t)b, (uint64_t)(b >> 64) };
    u256 r = { { 0, 0, 0, 0 } };
    for (int i = 0; i < 4; ++i) {
        u128 carry = 0;
        for (int j = 0; j < 2 && i + j < 4; ++j) {
            u128 cur = (u128)a.w[i] * bl[j] + r.w[i + j] + carry;
            r.w[i + j] = (uint64_t)cur;
            carry = cur >> 64;
        }
        for (int k = i + 2; k < 4 && carry; ++k) {
            u128 cur = (u128)r.w[k] + carry;
            r.w[k] = (uint64_t)cur;
            carry = cur >> 64;
        }
    }
    return r;
}

static int u256_le(u256 a, u256 b)
{
    for (int i = 3; i >= 0; --i) {
        if (a.w[i] != b.w[i]) return a.w[i] < b.w[i];
    }
    return 1;
}

/* p * 2^shift for shift = 128 or 192 */
static u256 u256_prime_shifted(unsigned p, int shift)
{
    u256 r = { { 0, 0, 0, 0 } };
    r.w[shift / 64] = p;
    return r;
}

/* floor(root_degree(p) * 2^64), degree 2 or 3, bit by bit from the top */
static u128 scaled_root(unsigned p, int degree)
{
    const u256 target = u256_prime_shifted(p, 64 * degree);
    u128 r = 0;
    for (int bit = 68; bit >= 0; --bit) {
        const u128 cand = r | ((u128)1 << bit);
        u256 pw = u256_mul(u256_from_u128(cand), cand);
        if (degree == 3) pw = u256_mul(pw, cand);
        /* cand < 2^69 keeps every product below 2^207 */
        if (u256_le(pw, target)) r = cand;
    }
    return r;
}

static void derive_constants512(void)
{
    int found = 0;
    for (unsigned p = 2; found < 80; ++p) {
        int prime = 1;
        for (unsigned q = 2; q * q <= p; ++q)
            if (p % q == 0) { prime = 0; break; }
        if (!prime) continue;
        g_k512[found] = (uint64_t)scaled_root(p, 3);            /* first 64 fraction bits of the cube root */
        if (found >= 8 && found < 16)                           /* SHA-384: the 9th to 16th primes */
            g_h0_384[found - 8] = (uint64_t)scaled_root(p, 2);  /* first 64 fraction bits of the square root */
        if (found < 8)                                          /* SHA-512 (section 5.3.5): the first eight primes */
            g_h0_512[found] = (uint64_t)scaled_root(p, 2);
        ++found;
    }
}

void ivo_constants512(uint64_t k_out[80], uint64_t h0_384_out[8])
{
    pthread_once(&g_once512, derive_constants512);
    memcpy(k_out, g_k512, sizeof g_k512);
    memcpy(h0_384_out, g_h0_384, sizeof g_h0_384);
}

static uint64_t rotr64(uint64_t x, unsigned n) { return (x >> n) | (x << (64u - n)); }
static uint64_t ch64(uint64_t x, uint64_t y, uint64_t z) { return (x & y) ^ (~x & z); }
static uint64_t maj64(uint64_t x, uint64_t y, uint64_t z) { return (x & y) ^ (x & z) ^ (y & z); }
static uint64_t big_sigma0_512(uint64_t x) { return rotr64(x, 28) ^ rotr64(x, 34) ^ rotr64(x, 39); }
static uint64_t big_sigma1_512(uint64_t x) { return rotr64(x, 14) ^ rotr64(x, 18) ^ rotr64(x, 41); }
static uint64_t small_sigma0_512(uint64_t x) { return rotr64(x, 1) ^ rotr64(x, 8) ^ (x >> 7); }
static uint64_t small_sigma1_512(uint64_t x) { return rotr64(x, 19) ^ rotr64(x, 61) ^ (x >> 6); }

/* FIPS 180-4 section 6.4.2: one 1024-bit block into the hash state. */
static void process_block512(uint64_t hash[8], const uint8_t block[128])
{
    uint64_t w[80];
    for (int t = 0; t < 16; ++t) {
        uint64_t v = 0;
        for (int b = 0; b < 8; ++b) v = (v << 8) | block[8 * t + b];
        w[t] = v;
    }
    for (int t = 16; t < 80; ++t)
        w[t] = small_sigma1_512(w[t - 2]) + w[t - 7] + small_sigma0_512(w[t - 15]) + w[t - 16];

    uint64_t a = hash[0], b = hash[1], c = hash[2], d = hash[3];
    uint64_t e = hash[4], f = hash[5], g = hash[6], h = hash[7];
    for (int t = 0; t < 80; ++t) {
        uint64_t t1 = h + big_sigma1_512(e) + ch64(e, f, g) + g_k512[t] + w[t];
        uint64_t t2 = big_sigma0_512(a) + maj64(a, b, c);
        h = g; g = f; f = e; e = d + t1;
        d = c; c = b; b = a; a = t1 + t2;
    }
    hash[0] += a; hash[1] += b; hash[2] += c; hash[3] += d;
    hash[4] += e; hash[5] += f; hash[6] += g; hash[7] += h;
}

/* FIPS 180-4 section 5.1.2 (padding to 1024-bit blocks, 128-bit length) + 6.5 (truncation). */
void ivo_sha384(const uint8_t *msg, uint64_t len, uint8_t out[48])
{
    pthread_once(&g_once512, derive_constants512);
    uint64_t hash[8];
    memcpy(hash, g_h0_384, sizeof hash);

    uint64_t full = len / 128;
    for (uint64_t i = 0; i < full; ++i)
        process_block512(hash, msg + 128 * i);

    uint8_t tail[256];
    uint64_t rem = len - 128 * full;
    memset(tail, 0, sizeof tail);
    if (rem) memcpy(tail, msg + 128 * full, rem);
    tail[rem] = 0x80;
    uint64_t tail_len = (rem + 1 + 16 <= 128) ? 128 : 256;
    /* the length in bits as a 128-bit big-endian integer; len < 2^64 bytes, so bits < 2^67 */
    u128 bits = (u128)len * 8u;
    for (int i = 0; i < 16; ++i)
        tail[tail_len - 1 - i] = (uint8_t)(bits >> (8 * i));
    for (uint64_t off = 0; off < tail_len; off += 128)
        process_block512(hash, tail + off);

    for (int i = 0; i < 6; ++i)                     /* the leftmost 384 bits */
        for (int b = 0; b < 8; ++b)
            out[8 * i + b] = (uint8_t)(hash[i] >> (56 - 8 * b));
}

typedef struct {
    const uint8_t *data;
    uint64_t nbytes, chunk_bytes;
    uint8_t *out;
} chunk384_job;

static void chunk384_task(void *arg, uint64_t i)
{
    chunk384_job *job = (chunk384_job *)arg;
    uint64_t begin = i * job->chunk_bytes;
    uint64_t end = begin + job->chunk_bytes;
    if (end > job->nbytes || end < begin) end = job->nbytes;
    ivo_sha384(job->data + begin, end - begin, job->out + 48 * i);
}

uint64_t ivo_hash_chunks_sha384(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                                uint8_t *digests_out, int nthreads)
{
    if (chunk_bytes == 0 || nbytes == 0) return 0;
    uint64_t n = nbytes / chunk_bytes + (nbytes % chunk_bytes ? 1 : 0);
    chunk384_job job = { data, nbytes, chunk_bytes, digests_out };
    run_tasks(chunk384_task, &job, n, nthreads);
    return n;
}

void ivo_merkle_root_sha384(const uint8_t *leaves, uint64_t n, uint8_t root_out[48])
{
    if (n == 0) { ivo_sha384((const uint8_t *)"", 0, root_out); return; }
    uint8_t *level = (uint8_t *)malloc((size_t)n * 48);
    memcpy(level, leaves, (size_t)n * 48);
    while (n > 1) {
        uint64_t parents = n / 2;
        for (uint64_t j = 0; j < parents; ++j) {
            uint8_t node[48];
            ivo_sha384(level + 96 * j, 96, node);      /* left || right are adjacent records */
            memcpy(level + 48 * j, node, 48);
        }
        if (n % 2) {
            memmove(level + 48 * parents, level + 48 * (n - 1), 48);
            ++parents;
        }
        n = parents;
    }
    memcpy(root_out, level, 48);
    free(level);
}

/* ------------------------------------------------------------------------- */
/* SHA-512 (FIPS 180-4 sections 5.1.2, 5.3.5, 6.4): the same compression      */
/* function, the initial value from the first eight primes, all 512 bits out. */
/* ------------------------------------------------------------------------- */

void ivo_h0_sha512(uint64_t h0_out[8])
{
    pthread_once(&g_once512, derive_constants512);
    memcpy(h0_out, g_h0_512, sizeof g_h0_512);
}

void ivo_sha512(const uint8_t *msg, uint64_t len, uint8_t out[64])
{
    pthread_once(&g_once512, derive_constants512);
    uint64_t hash[8];
    memcpy(hash, g_h0_512, sizeof hash);

    uint64_t full = len / 128;
    for (uint64_t i = 0; i < full; ++i)
        process_block512(hash, msg + 128 * i);

    /* section 5.1.2: 0x80, zeros up to 112 mod 128, then the bit length as a 128-bit big-endian integer */
    uint8_t tail[256];
    uint64_t rem = len - 128 * full;
    memset(tail, 0, sizeof tail);
    if (rem) memcpy(tail, msg + 128 * full, rem);
    tail[rem] = 0x80;
    uint64_t tail_len = (rem + 1 + 16 <= 128) ? 128 : 256;
    u128 bits = (u128)len * 8u;
    for (int i = 0; i < 16; ++i)
        tail[tail_len - 1 - i] = (uint8_t)(bits >> (8 * i));
    for (uint64_t off = 0; off < tail_len; off += 128)
        process_block512(hash, tail + off);

    for (int i = 0; i < 8; ++i)
        for (int b = 0; b < 8; ++b)
            out[8 * i + b] = (uint8_t)(hash[i] >> (56 - 8 * b));
}

typedef struct {
    const uint8_t *data;
    uint64_t nbytes, chunk_bytes;
    uint8_t *out;
} chunk512_job;

static void chunk512_task(void *arg, uint64_t i)
{
    chunk512_job *job = (chunk512_job *)arg;
    uint64_t begin = i * job->chunk_bytes;
    uint64_t end = begin + job->chunk_bytes;
    if (end > job->nbytes || end < begin) end = job->nbytes;
    ivo_sha512(job->data + begin, end - begin, job->out + 64 * i);
}

uint64_t ivo_hash_chunks_sha512(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                                uint8_t *digests_out, int nthreads)
{
    if (chunk_bytes == 0 || nbytes == 0) return 0;
    uint64_t n = nbytes / chunk_bytes + (nbytes % chunk_bytes ? 1 : 0);
    chunk512_job job = { data, nbytes, chunk_bytes, digests_out };
    run_tasks(chunk512_task, &job, n, nthreads);
    return n;
}

/* The tree rule of the default path with SHA-512 as the node hash: parent = SHA-512(left || right) over
 * exactly 128 bytes, an unpaired last node moves up unchanged, one leaf is the root, no leaf gives SHA-512(""). */
void ivo_merkle_root_sha512(const uint8_t *leaves, uint64_t n, uint8_t root_out[64])
{
    if (n == 0) { ivo_sha512((const uint8_t *)"", 0, root_out); return; }
    uint8_t *level = (uint8_t *)malloc((size_t)n * 64);
    memcpy(level, leaves, (size_t)n * 64);
    while (n > 1) {
        uint64_t parents = n / 2;
        for (uint64_t j = 0; j < parents; ++j) {
            uint8_t node[64];
            ivo_sha512(level + 128 * j, 128, node);
            memcpy(level + 64 * j, node, 64);
        }
        if (n % 2) {
            memmove(level + 64 * parents, level + 64 * (n - 1), 64);
            ++parents;
        }
        n = parents;
    }
    memcpy(root_out, level, 64);
    free(level);
}

/* ------------------------------------------------------------------------- */
/* RFC 6962 section 2.1: domain-separated Merkle Tree Hash over SHA-256.      */
/*   leaf hash  = SHA-256(0x00 || entry),  node = SHA-256(0x01 || left || right) */
/*   MTH({})    = SHA-256(""),             MTH({d0}) = leaf hash of d0           */
/*   MTH(D[n])  = node(MTH(D[0:k]), MTH(D[k:n])), k the largest power of two < n */
/* Written as that recursion over the entries (here: the chunks of a blob).   */
/* ------------------------------------------------------------------------- */

static void rfc6962_leaf(const uint8_t *entry, uint64_t len, uint8_t out[32])
{
    uint8_t *msg = (uint8_t *)malloc((size_t)len + 1);
    msg[0] = 0x00;
    if (len) memcpy(msg + 1, entry, (size_t)len);
    ivo_sha256(msg, len + 1, out);
    free(msg);
}

static void rfc6962_node(const uint8_t left[32], const uint8_t right[32], uint8_t out[32])
{
    uint8_t msg[65];
    msg[0] = 0x01;
    memcpy(msg + 1, left, 32);
    memcpy(msg + 33, right, 32);
    ivo_sha256(msg, 65, out);
}

static void chunk6962_task(void *arg, uint64_t i)
{
    chunk_job *job = (chunk_job *)arg;
    uint64_t begin = i * job->chunk_bytes;
    uint64_t end = begin + job->chunk_bytes;
    if (end > job->nbytes || end < begin) end = job->nbytes;
    rfc6962_leaf(job->data + begin, end - begin, job->out + 32 * i);
}

uint64_t ivo_hash_chunks_rfc6962(const uint8_t *data, uint64_t nbytes, uint64_t chunk_bytes,
                                 uint8_t *leaf_hashes_out, int nthreads)
{
    if (chunk_bytes == 0 || nbytes == 0) return 0;
    uint64_t n = nbytes / chunk_bytes + (nbytes % chunk_bytes ? 1 : 0);
    chunk_job job = { data, nbytes, chunk_bytes, leaf_hashes_out };
    run_tasks(chunk6962_task, &job, n, nthreads);
    return n;
}

void ivo_merkle_root_rfc6962(const uint8_t *leaf_hashes, uint64_t n, uint8_t root_out[32])
{
    if (n == 0) { ivo_sha256((const uint8_t *)"", 0, root_out); return; }
    if (n == 1) { memcpy(root_out, leaf_hashes, 32); return; }
    uint64_t k = 1;
    while (k * 2 < n) k *= 2;
    uint8_t left[32], right[32];
    ivo_merkle_root_rfc6962(leaf_hashes, k, left);
    ivo_merkle_root_rfc6962(leaf_hashes + 32 * k, n - k, right);
    rfc6962_node(left, right, root_out);
}
