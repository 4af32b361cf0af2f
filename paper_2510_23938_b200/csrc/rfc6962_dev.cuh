// Device helpers of the RFC 6962 section 2.1 mode (messages that start with a one-byte prefix).
#pragma once
#include <cstdint>

namespace ivk {

// Big-endian message word from the little-endian data words (cur, prev): prev.byte3, cur.byte0..2.
__device__ __forceinline__ uint32_t shifted_word(uint32_t cur, uint32_t prev) { return __byte_perm(cur, prev, 0x7012u); }

// Tail of the prefixed message from message position mpos (a multiple of 64) to its end at msg_bytes,
// then the padding.  Message byte 0 is the prefix, message byte q >= 1 is data[q - 1].  At most 64
// message bytes remain, so the tail is one or two blocks.
static __device__ __noinline__ int prefixed_tail(const uint8_t *data, uint8_t prefix, uint64_t mpos, uint64_t msg_bytes,
                                                 uint32_t *tw /* [32] */) {
    for (int i = 0; i < 32; ++i) tw[i] = 0u;
    const uint32_t rem = (uint32_t)(msg_bytes - mpos);
    for (uint32_t k = 0; k < rem; ++k) {
        const uint64_t q = mpos + k;
        const uint32_t byte = q == 0 ? prefix : data[q - 1];
        tw[k >> 2] |= byte << (24 - 8 * (k & 3));
    }
    tw[rem >> 2] |= 0x80u << (24 - 8 * (rem & 3));
    const int nblk = (rem + 1 + 8 <= 64) ? 1 : 2;
    const uint64_t bits = msg_bytes << 3;
    tw[16 * nblk - 2] = (uint32_t)(bits >> 32);
    tw[16 * nblk - 1] = (uint32_t)bits;
    return nblk;
}

}  // namespace ivk
