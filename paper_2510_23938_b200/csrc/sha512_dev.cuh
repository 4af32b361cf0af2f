// SHA-384 (FIPS 180-4 sections 4.1.3, 4.2.3, 5.3.4, 6.4.2, 6.5) for one compression chain per thread:
// SHA-512's compression function on 64-bit words with SHA-384's initial value, digest = the first
// six words.  64-bit rotates compile to pairs of funnel shifts, the boolean functions to pairs of LOP3.
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

__device__ __forceinline__ uint64_t rotr64(uint64_t x, int n) { return (x >> n) | (x << (64 - n)); }
__device__ __forceinline__ uint64_t ch64(uint64_t x, uint64_t y, uint64_t z) { return (x & y) ^ (~x & z); }
__device__ __forceinline__ uint64_t maj64(uint64_t x, uint64_t y, uint64_t z) { return (x & y) | (z & (x | y)); }
__device__ __forceinline__ uint64_t big_s0_512(uint64_t x) { return rotr64(x, 28) ^ rotr64(x, 34) ^ rotr64(x, 39); }
__device__ __forceinline__ uint64_t big_s1_512(uint64_t x) { return rotr64(x, 14) ^ rotr64(x, 18) ^ rotr64(x, 41); }
__device__ __forceinline__ uint64_t small_s0_512(uint64_t x) { return rotr64(x, 1) ^ rotr64(x, 8) ^ (x >> 7); }
__device__ __forceinline__ uint64_t small_s1_512(uint64_t x) { return rotr64(x, 19) ^ rotr64(x, 61) ^ (x >> 6); }

// Initial hash value of SHA-384, FIPS 180-4 section 5.3.4.
__device__ __forceinline__ void sha384_init(uint64_t (&st)[8]) {
    st[0] = 0xcbbb9d5dc1059ed8ull; st[1] = 0x629a292a367cd507ull; st[2] = 0x9159015a3070dd17ull;
    st[3] = 0x152fecd8f70e5939ull; st[4] = 0x67332667ffc00b31ull; st[5] = 0x8eb44a8768581511ull;
    st[6] = 0xdb0c2e0d64f98fa7ull; st[7] = 0x47b5481dbefa4fa4ull;
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
    return ((uint64_t)__byte_perm(lo_addr_word, 0, 0x0123) << 32) | (uint64_t)__byte_perm(hi_addr_word, 0, 0x0123);
}

// 48-byte digest record (six big-endian words) at a 16-byte aligned address.
__device__ __forceinline__ void store_digest384(uint8_t *dst, const uint64_t (&st)[8]) {
    uint32_t o[12];
#pragma unroll
    for (int i = 0; i < 6; ++i) {
        o[2 * i] = __byte_perm((uint32_t)(st[i] >> 32), 0, 0x0123);
        o[2 * i + 1] = __byte_perm((uint32_t)st[i], 0, 0x0123);
    }
    if ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
        uint4 *q = reinterpret_cast<uint4 *>(dst);
        q[0] = make_uint4(o[0], o[1], o[2], o[3]);
        q[1] = make_uint4(o[4], o[5], o[6], o[7]);
        q[2] = make_uint4(o[8], o[9], o[10], o[11]);
    } else {
#pragma unroll
        for (int i = 0; i < 12; ++i)
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
