// SHA-256 (FIPS 180-4 section 6.2.2) for one compression chain per thread.
//
// The 64 rounds are written out by macro with the round constants as literals,
// the 16-word message window stays in registers, rotates are funnel shifts
// (SHF), the three-input boolean functions are single LOP3s.
#pragma once
#include <cstdint>

namespace ivk {

// FIPS 180-4 section 5.3.3.
#define IV_H0_0 0x6a09e667u
#define IV_H0_1 0xbb67ae85u
#define IV_H0_2 0x3c6ef372u
#define IV_H0_3 0xa54ff53au
#define IV_H0_4 0x510e527fu
#define IV_H0_5 0x9b05688cu
#define IV_H0_6 0x1f83d9abu
#define IV_H0_7 0x5be0cd19u

__device__ __forceinline__ uint32_t rotr(uint32_t x, uint32_t n) { return __funnelshift_r(x, x, n); }

template <int LUT>
__device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(r) : "r"(a), "r"(b), "r"(c), "n"(LUT));
    return r;
}
__device__ __forceinline__ uint32_t xor3(uint32_t a, uint32_t b, uint32_t c) { return lop3<0x96>(a, b, c); }
// FIPS 180-4 section 4.1.2, equations 4.2 - 4.7.
__device__ __forceinline__ uint32_t f_ch(uint32_t x, uint32_t y, uint32_t z) { return lop3<0xCA>(x, y, z); }
__device__ __forceinline__ uint32_t f_maj(uint32_t x, uint32_t y, uint32_t z) { return lop3<0xE8>(x, y, z); }
__device__ __forceinline__ uint32_t big_s0(uint32_t x) { return xor3(rotr(x, 2), rotr(x, 13), rotr(x, 22)); }
__device__ __forceinline__ uint32_t big_s1(uint32_t x) { return xor3(rotr(x, 6), rotr(x, 11), rotr(x, 25)); }
__device__ __forceinline__ uint32_t small_s0(uint32_t x) { return xor3(rotr(x, 7), rotr(x, 18), x >> 3); }
__device__ __forceinline__ uint32_t small_s1(uint32_t x) { return xor3(rotr(x, 17), rotr(x, 19), x >> 10); }

// Big-endian word from four bytes in memory order held little-endian in x.
__device__ __forceinline__ uint32_t bswap32(uint32_t x) { return __byte_perm(x, 0, 0x0123); }

__device__ __forceinline__ void sha256_init(uint32_t (&st)[8]) {
    st[0] = IV_H0_0; st[1] = IV_H0_1; st[2] = IV_H0_2; st[3] = IV_H0_3;
    st[4] = IV_H0_4; st[5] = IV_H0_5; st[6] = IV_H0_6; st[7] = IV_H0_7;
}

// Two-input add on a chosen pipe.  The INT32 ALU pipe (SHF, LOP3, PRMT, IADD3) is what bounds
// SHA-256; an integer multiply-add runs on the FMA pipe, which is otherwise idle here, so
// "a * one + b" with a multiplier the compiler cannot see (a kernel argument equal to 1)
// moves the add off the ALU pipe.  FMA = false gives the plain add.
template <bool FMA>
__device__ __forceinline__ uint32_t padd(uint32_t a, uint32_t b, uint32_t one) {
    if (FMA) {
        uint32_t r;
        asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(one), "r"(b));
        return r;
    }
    return a + b;
}

// Where the additions of a compression go (template parameter ADD):
//   0  left to the compiler (mostly three-input adds on the ALU pipe)
//   2  the message schedule's additions and the feed-forward on the FMA pipe, the rounds' left to the
//      compiler; pays only with three warps per SM scheduler, which hide the longer dependency chains

// One round (FIPS 180-4 section 6.2.2 step 3):
//   T1 = h + S1(e) + Ch(e,f,g) + K + W;  d += T1;  h = T1 + S0(a) + Maj(a,b,c).
// The caller rotates the variable names instead of moving values.
__device__ __forceinline__ void sha_round(uint32_t a, uint32_t b, uint32_t c, uint32_t &d, uint32_t e, uint32_t f,
                                          uint32_t g, uint32_t &h, uint32_t k, uint32_t w) {
    const uint32_t t1 = h + big_s1(e) + f_ch(e, f, g) + (k + w);
    d += t1;
    h = t1 + big_s0(a) + f_maj(a, b, c);
}

// Message-schedule step in the rolling 16-word window (i = t mod 16):
// W[t] = s1(W[t-2]) + W[t-7] + s0(W[t-15]) + W[t-16].
template <int ADD>
__device__ __forceinline__ void sha_sched(uint32_t (&w)[16], int i, uint32_t one) {
    constexpr bool F = ADD == 2;
    const uint32_t s = padd<F>(small_s1(w[(i + 14) & 15]), w[(i + 9) & 15], one);
    const uint32_t t = padd<F>(small_s0(w[(i + 1) & 15]), w[i & 15], one);
    w[i & 15] = padd<F>(s, t, one);
}

#define IV_ROUND(a, b, c, d, e, f, g, h, k, wv) ivk::sha_round(a, b, c, d, e, f, g, h, k, wv)

// Eight rounds starting at a round index that is a multiple of 8 (so the
// variable rotation returns to a..h), constants k0..k7 from FIPS 180-4 4.2.2.
#define IV_ROUNDS8(v, w, i, k0, k1, k2, k3, k4, k5, k6, k7)                           \
    IV_ROUND(v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7], k0, (w)[((i) + 0) & 15]); \
    IV_ROUND(v[7], v[0], v[1], v[2], v[3], v[4], v[5], v[6], k1, (w)[((i) + 1) & 15]); \
    IV_ROUND(v[6], v[7], v[0], v[1], v[2], v[3], v[4], v[5], k2, (w)[((i) + 2) & 15]); \
    IV_ROUND(v[5], v[6], v[7], v[0], v[1], v[2], v[3], v[4], k3, (w)[((i) + 3) & 15]); \
    IV_ROUND(v[4], v[5], v[6], v[7], v[0], v[1], v[2], v[3], k4, (w)[((i) + 4) & 15]); \
    IV_ROUND(v[3], v[4], v[5], v[6], v[7], v[0], v[1], v[2], k5, (w)[((i) + 5) & 15]); \
    IV_ROUND(v[2], v[3], v[4], v[5], v[6], v[7], v[0], v[1], k6, (w)[((i) + 6) & 15]); \
    IV_ROUND(v[1], v[2], v[3], v[4], v[5], v[6], v[7], v[0], k7, (w)[((i) + 7) & 15])

#define IV_SCHED8(w, i)                                                                      \
    ivk::sha_sched<ADD>(w, (i) + 0, one); ivk::sha_sched<ADD>(w, (i) + 1, one);               \
    ivk::sha_sched<ADD>(w, (i) + 2, one); ivk::sha_sched<ADD>(w, (i) + 3, one);               \
    ivk::sha_sched<ADD>(w, (i) + 4, one); ivk::sha_sched<ADD>(w, (i) + 5, one);               \
    ivk::sha_sched<ADD>(w, (i) + 6, one); ivk::sha_sched<ADD>(w, (i) + 7, one)

// st <- compress(st, block) where w[0..15] holds the block as big-endian words.
// w is destroyed (it is the rolling schedule window).  ADD places the additions (0 or 2, see above);
// for ADD != 0 `one` must hold the value 1 in a way the compiler cannot see through.
template <int ADD = 0>
__device__ __forceinline__ void sha256_compress(uint32_t (&st)[8], uint32_t (&w)[16], uint32_t one = 1u) {
    static_assert(ADD == 0 || ADD == 2, "addition placements 0 and 2 exist");
    uint32_t v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = st[i];

    IV_ROUNDS8(v, w, 0, 0x428a2f98u, 0x71374491u, 0xb5c0fbcfu, 0xe9b5dba5u, 0x3956c25bu, 0x59f111f1u, 0x923f82a4u, 0xab1c5ed5u);
    IV_ROUNDS8(v, w, 8, 0xd807aa98u, 0x12835b01u, 0x243185beu, 0x550c7dc3u, 0x72be5d74u, 0x80deb1feu, 0x9bdc06a7u, 0xc19bf174u);
    IV_SCHED8(w, 0);
    IV_ROUNDS8(v, w, 0, 0xe49b69c1u, 0xefbe4786u, 0x0fc19dc6u, 0x240ca1ccu, 0x2de92c6fu, 0x4a7484aau, 0x5cb0a9dcu, 0x76f988dau);
    IV_SCHED8(w, 8);
    IV_ROUNDS8(v, w, 8, 0x983e5152u, 0xa831c66du, 0xb00327c8u, 0xbf597fc7u, 0xc6e00bf3u, 0xd5a79147u, 0x06ca6351u, 0x14292967u);
    IV_SCHED8(w, 0);
    IV_ROUNDS8(v, w, 0, 0x27b70a85u, 0x2e1b2138u, 0x4d2c6dfcu, 0x53380d13u, 0x650a7354u, 0x766a0abbu, 0x81c2c92eu, 0x92722c85u);
    IV_SCHED8(w, 8);
    IV_ROUNDS8(v, w, 8, 0xa2bfe8a1u, 0xa81a664bu, 0xc24b8b70u, 0xc76c51a3u, 0xd192e819u, 0xd6990624u, 0xf40e3585u, 0x106aa070u);
    IV_SCHED8(w, 0);
    IV_ROUNDS8(v, w, 0, 0x19a4c116u, 0x1e376c08u, 0x2748774cu, 0x34b0bcb5u, 0x391c0cb3u, 0x4ed8aa4au, 0x5b9cca4fu, 0x682e6ff3u);
    IV_SCHED8(w, 8);
    IV_ROUNDS8(v, w, 8, 0x748f82eeu, 0x78a5636fu, 0x84c87814u, 0x8cc70208u, 0x90befffau, 0xa4506cebu, 0xbef9a3f7u, 0xc67178f2u);

#pragma unroll
    for (int i = 0; i < 8; ++i) st[i] = padd<ADD != 0>(st[i], v[i], one);
}

// The last block of a message whose length is a multiple of 64 bytes holds no
// data: 0x80, zeros, and the bit length (FIPS 180-4 section 5.1.1).
__device__ __forceinline__ void sha256_pad_only_block(uint32_t (&w)[16], uint64_t msg_bytes) {
    const uint64_t bits = msg_bytes << 3;
    w[0] = 0x80000000u;
#pragma unroll
    for (int i = 1; i < 14; ++i) w[i] = 0u;
    w[14] = (uint32_t)(bits >> 32);
    w[15] = (uint32_t)bits;
}

// Digest record: H0..H7 big-endian, written as two 16-byte stores (dst 16-byte aligned).
__device__ __forceinline__ void store_digest_aligned(uint8_t *dst, const uint32_t (&st)[8]) {
    uint4 lo = make_uint4(bswap32(st[0]), bswap32(st[1]), bswap32(st[2]), bswap32(st[3]));
    uint4 hi = make_uint4(bswap32(st[4]), bswap32(st[5]), bswap32(st[6]), bswap32(st[7]));
    reinterpret_cast<uint4 *>(dst)[0] = lo;
    reinterpret_cast<uint4 *>(dst)[1] = hi;
}

// Digest record at any alignment.
__device__ __forceinline__ void store_digest(uint8_t *dst, const uint32_t (&st)[8]) {
    if ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
        store_digest_aligned(dst, st);
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            dst[4 * i + 0] = (uint8_t)(st[i] >> 24);
            dst[4 * i + 1] = (uint8_t)(st[i] >> 16);
            dst[4 * i + 2] = (uint8_t)(st[i] >> 8);
            dst[4 * i + 3] = (uint8_t)(st[i]);
        }
    }
}

// Message tail: the last (len mod 64) bytes of a message, then the padding.
// Reads the bytes one by one (any alignment) into tw[0..31] as big-endian words
// and returns the number of 64-byte blocks the tail occupies (1 or 2).
static __device__ __noinline__ int sha256_build_tail(const uint8_t *tail_bytes, uint32_t rem, uint64_t msg_bytes,
                                              uint32_t *tw /* [32] */) {
    for (int i = 0; i < 32; ++i) tw[i] = 0u;
    for (uint32_t k = 0; k < rem; ++k)
        tw[k >> 2] |= (uint32_t)tail_bytes[k] << (24 - 8 * (k & 3));
    tw[rem >> 2] |= 0x80u << (24 - 8 * (rem & 3));
    const int nblk = (rem + 1 + 8 <= 64) ? 1 : 2;
    const uint64_t bits = msg_bytes << 3;
    tw[16 * nblk - 2] = (uint32_t)(bits >> 32);
    tw[16 * nblk - 1] = (uint32_t)bits;
    return nblk;
}

}  // namespace ivk
