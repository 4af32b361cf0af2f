// SHA-384 and SHA-512 (FIPS 180-4 sections 4.1.3, 4.2.3, 5.3.4, 5.3.5, 6.4.2, 6.5) for one compression chain
// per thread: one compression function on 64-bit words; SHA-384 starts from its own initial value and keeps
// the first six words, SHA-512 keeps all eight.  64-bit rotates compile to pairs of funnel shifts, the boolean
// functions to pairs of LOP3.
#pragma once
#include <cstdint>

namespace ivk {

// Round constants, FIPS 180-4 section 4.2.3.
static __constant__ uint64_t kSha512K[80] = {
    0x428a2f98d728ae22ull, 0x7137449123ef65cdull, 0xb5c0fbcfec4d3b2full, 0xe9b5dba58189dbbcull,
    0x3956c25bf348b538ull, 0x59f111f1b605d019ull, 0x923f82a4af194f9bull, 0xab1c5ed5da6d8118ull,
    0xd807aa98a3030242ull, 0x12835b0145706fbeull, 0x243185be4ee4b28cull, 0x550c7dc3d5ffb4e2ull,
    0x72be5d74f27b896full, 0x80deb1fe3b1696b1ull, 0x9bdc06a725c71235ull, 0xc19bf174cf692694ull,
    0xe49b69c19ef14ad2ull, 0xefbe4786384f25e3ull, 0x0fc19dc68b8cd5b5ull, 0x240ca1cc77ac9c65ull,
    0x2de92c6f592b0275ull, 0x4a7484aa6ea6e483ull, 0x5cb0a9dcbd41fbd4ull, 0x76f988da831153b5ull,
    0x983e5152ee66dfabull, 0xa831c66d2db43210ull, 0xb00327c898fb213full, 0xbf597fc7beef0ee4ull,
    0xc6e00bf33da88fc2ull, 0xd5a79147930aa725ull, 0x06ca6351e003826full, 0x142929670a0e6e70ull,
    0x27b70a8546d22ffcull, 0x2e1b21385c26c926ull, 0x4d2c6dfc5ac42aedull, 0x53380d139d95b3dfull,
    0x650a73548baf63deull, 0x766a0abb3c77b2a8ull, 0x81c2c92e47edaee6ull, 0x92722c851482353bull,
    0xa2bfe8a14cf10364ull, 0xa81a664bbc423001ull, 0xc24b8b70d0f89791ull, 0xc76c51a30654be30ull,
    0xd192e819d6ef5218ull, 0xd69906245565a910ull, 0xf40e35855771202aull, 0x106aa07032bbd1b8ull,
    0x19a4c116b8d2d0c8ull, 0x1e376c085141ab53ull, 0x2748774cdf8eeb99ull, 0x34b0bcb5e19b48a8ull,
    0x391c0cb3c5c95a63ull, 0x4ed8aa4ae3418acbull, 0x5b9cca4f7763e373ull, 0x682e6ff3d6b2b8a3ull,
    0x748f82ee5defb2fcull, 0x78a5636f43172f60ull, 0x84c87814a1f0ab72ull, 0x8cc702081a6439ecull,
    0x90befffa23631e28ull, 0xa4506cebde82bde9ull, 0xbef9a3f7b2c67915ull, 0xc67178f2e372532bull,
    0xca273eceea26619cull, 0xd186b8c721c0c207ull, 0xeada7dd6cde0eb1eull, 0xf57d4f7fee6ed178ull,
    0x06f067aa72176fbaull, 0x0a637dc5a2c898a6ull, 0x113f9804bef90daeull, 0x1b710b35131c471bull,
    0x28db77f523047d84ull, 0x32caab7b40c72493ull, 0x3c9ebe0a15c9bebcull, 0x431d67c49c100d4cull,
    0x4cc5d4becb3e42b6ull, 0x597f299cfc657e2aull, 0x5fcb6fab3ad6faecull, 0x6c44198c4a475817ull,
};

// 64-bit words are handled as pairs of 32-bit registers, written out so that every rotation is two funnel
// shifts and every three-input boolean function one LOP3 per half (left to itself the compiler splits the
// 64-bit expressions but does not merge the two XORs of a Sigma into one three-input operation).
__device__ __forceinline__ uint32_t lo32(uint64_t x) { return (uint32_t)x; }
__device__ __forceinline__ uint32_t hi32(uint64_t x) { return (uint32_t)(x >> 32); }
__device__ __forceinline__ uint64_t pack64(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
template <int LUT>
__device__ __forceinline__ uint32_t lop3_512(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(r) : "r"(a), "r"(b), "r"(c), "n"(LUT));
    return r;
}
// low and high half of rotr(x, N) and of x >> N
template <int N>
__device__ __forceinline__ uint32_t rotr64_lo(uint32_t lo, uint32_t hi) {
    return N < 32 ? __funnelshift_r(lo, hi, N) : __funnelshift_r(hi, lo, N - 32);
}
template <int N>
__device__ __forceinline__ uint32_t rotr64_hi(uint32_t lo, uint32_t hi) {
    return N < 32 ? __funnelshift_r(hi, lo, N) : __funnelshift_r(lo, hi, N - 32);
}
// xor of three rotations (FIPS 180-4 equations 4.10, 4.11)
template <int A, int B, int C>
__device__ __forceinline__ uint64_t sigma_rrr(uint64_t x) {
    const uint32_t l = lo32(x), h = hi32(x);
    return pack64(lop3_512<0x96>(rotr64_lo<A>(l, h), rotr64_lo<B>(l, h), rotr64_lo<C>(l, h)),
                  lop3_512<0x96>(rotr64_hi<A>(l, h), rotr64_hi<B>(l, h), rotr64_hi<C>(l, h)));
}
// xor of two rotations and a right shift by S < 32 (equations 4.12, 4.13)
template <int A, int B, int S>
__device__ __forceinline__ uint64_t sigma_rrs(uint64_t x) {
    const uint32_t l = lo32(x), h = hi32(x);
    return pack64(lop3_512<0x96>(rotr64_lo<A>(l, h), rotr64_lo<B>(l, h), __funnelshift_r(l, h, S)),
                  lop3_512<0x96>(rotr64_hi<A>(l, h), rotr64_hi<B>(l, h), h >> S));
}
// FIPS 180-4 section 4.1.3, equations 4.8 - 4.13.
__device__ __forceinline__ uint64_t ch64(uint64_t x, uint64_t y, uint64_t z) {
    return pack64(lop3_512<0xCA>(lo32(x), lo32(y), lo32(z)), lop3_512<0xCA>(hi32(x), hi32(y), hi32(z)));
}
__device__ __forceinline__ uint64_t maj64(uint64_t x, uint64_t y, uint64_t z) {
    return pack64(lop3_512<0xE8>(lo32(x), lo32(y), lo32(z)), lop3_512<0xE8>(hi32(x), hi32(y), hi32(z)));
}
__device__ __forceinline__ uint64_t big_s0_512(uint64_t x) { return sigma_rrr<28, 34, 39>(x); }
__device__ __forceinline__ uint64_t big_s1_512(uint64_t x) { return sigma_rrr<14, 18, 41>(x); }
__device__ __forceinline__ uint64_t small_s0_512(uint64_t x) { return sigma_rrs<1, 8, 7>(x); }
__device__ __forceinline__ uint64_t small_s1_512(uint64_t x) { return sigma_rrs<19, 61, 6>(x); }

// Initial hash value of SHA-384, FIPS 180-4 section 5.3.4.
__device__ __forceinline__ void sha384_init(uint64_t (&st)[8]) {
    st[0] = 0xcbbb9d5dc1059ed8ull; st[1] = 0x629a292a367cd507ull; st[2] = 0x9159015a3070dd17ull;
    st[3] = 0x152fecd8f70e5939ull; st[4] = 0x67332667ffc00b31ull; st[5] = 0x8eb44a8768581511ull;
    st[6] = 0xdb0c2e0d64f98fa7ull; st[7] = 0x47b5481dbefa4fa4ull;
}

// Initial hash value of SHA-512, FIPS 180-4 section 5.3.5.
__device__ __forceinline__ void sha512_init(uint64_t (&st)[8]) {
    st[0] = 0x6a09e667f3bcc908ull; st[1] = 0xbb67ae8584caa73bull; st[2] = 0x3c6ef372fe94f82bull;
    st[3] = 0xa54ff53a5f1d36f1ull; st[4] = 0x510e527fade682d1ull; st[5] = 0x9b05688c2b3e6c1full;
    st[6] = 0x1f83d9abfb41bd6bull; st[7] = 0x5be0cd19137e2179ull;
}
template <int DIGEST_WORDS>
__device__ __forceinline__ void sha512_family_init(uint64_t (&st)[8]) {
    static_assert(DIGEST_WORDS == 6 || DIGEST_WORDS == 8, "SHA-384 keeps six words, SHA-512 eight");
    if (DIGEST_WORDS == 6) sha384_init(st);
    else sha512_init(st);
}

// st <- compress(st, block); w[0..15] holds the 128-byte block as big-endian 64-bit words and is
// destroyed (rolling schedule window).  Sixteen rounds per loop trip, five trips, names rotated.
__device__ __forceinline__ void sha512_compress(uint64_t (&st)[8], uint64_t (&w)[16]) {
    uint64_t v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = st[i];
#pragma unroll 1
    for (int base = 0; base < 80; base += 16) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if (base) w[i] += small_s1_512(w[(i + 14) & 15]) + w[(i + 9) & 15] + small_s0_512(w[(i + 1) & 15]);
            // round t = base + i: a = v[(8 - i) & 7], ..., h = v[(15 - i) & 7]
            uint64_t &a = v[(8 - i) & 7], &b = v[(9 - i) & 7], &c = v[(10 - i) & 7], &d = v[(11 - i) & 7];
            uint64_t &e = v[(12 - i) & 7], &f = v[(13 - i) & 7], &g = v[(14 - i) & 7], &h = v[(15 - i) & 7];
            const uint64_t t1 = h + big_s1_512(e) + ch64(e, f, g) + kSha512K[base + i] + w[i];
            d += t1;
            h = t1 + big_s0_512(a) + maj64(a, b, c);
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) st[i] += v[i];
}

// big-endian 64-bit word from eight bytes in memory order held as two little-endian 32-bit words
__device__ __forceinline__ uint64_t be64(uint32_t lo_addr_word, uint32_t hi_addr_word) {
    return pack64(__byte_perm(hi_addr_word, 0, 0x0123), __byte_perm(lo_addr_word, 0, 0x0123));
}

// Digest record: the first WORDS words, big-endian (48 bytes for SHA-384, 64 for SHA-512), at any alignment.
template <int WORDS>
__device__ __forceinline__ void store_digest512(uint8_t *dst, const uint64_t (&st)[8]) {
    uint32_t o[2 * WORDS];
#pragma unroll
    for (int i = 0; i < WORDS; ++i) {
        o[2 * i] = __byte_perm((uint32_t)(st[i] >> 32), 0, 0x0123);
        o[2 * i + 1] = __byte_perm((uint32_t)st[i], 0, 0x0123);
    }
    if ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
        uint4 *q = reinterpret_cast<uint4 *>(dst);
#pragma unroll
        for (int i = 0; i < WORDS / 2; ++i) q[i] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < 2 * WORDS; ++i)
            for (int b = 0; b < 4; ++b) dst[4 * i + b] = (uint8_t)(o[i] >> (8 * b));
    }
}

// Message tail: the last (len mod 128) bytes, then 0x80, zeros and the 128-bit bit length
// (FIPS 180-4 section 5.1.2).  tw[0..31] receives one or two blocks; returns how many.
static __device__ __noinline__ int sha512_build_tail(const uint8_t *tail_bytes, uint32_t rem, uint64_t msg_bytes,
                                                     uint64_t *tw /* [32] */) {
    for (int i = 0; i < 32; ++i) tw[i] = 0ull;
    for (uint32_t k = 0; k < rem; ++k) tw[k >> 3] |= (uint64_t)tail_bytes[k] << (56 - 8 * (k & 7));
    tw[rem >> 3] |= 0x80ull << (56 - 8 * (rem & 7));
    const int nblk = (rem + 1 + 16 <= 128) ? 1 : 2;
    tw[16 * nblk - 2] = msg_bytes >> 61;          // high 64 bits of the length in bits
    tw[16 * nblk - 1] = msg_bytes << 3;
    return nblk;
}

}  // namespace ivk
