// The two halves of a SHA-256 compression when it is split between a producer warp (message
// schedule plus round constants, independent of the chaining state) and a consumer warp (the
// 64 rounds): device functions shared by the split leaf kernel and the roofline probe.
#pragma once
#include "sha256_dev.cuh"
#include "tma_dev.cuh"

namespace ivk {

// Round constants, FIPS 180-4 section 4.2.2, as a compile-time function of t.
__device__ __forceinline__ constexpr uint32_t sha_k(int t) {
    constexpr uint32_t k[64] = {
        0x428a2f98u, 0x71374491u, 0xb5c0fbcfu, 0xe9b5dba5u, 0x3956c25bu, 0x59f111f1u, 0x923f82a4u, 0xab1c5ed5u,
        0xd807aa98u, 0x12835b01u, 0x243185beu, 0x550c7dc3u, 0x72be5d74u, 0x80deb1feu, 0x9bdc06a7u, 0xc19bf174u,
        0xe49b69c1u, 0xefbe4786u, 0x0fc19dc6u, 0x240ca1ccu, 0x2de92c6fu, 0x4a7484aau, 0x5cb0a9dcu, 0x76f988dau,
        0x983e5152u, 0xa831c66du, 0xb00327c8u, 0xbf597fc7u, 0xc6e00bf3u, 0xd5a79147u, 0x06ca6351u, 0x14292967u,
        0x27b70a85u, 0x2e1b2138u, 0x4d2c6dfcu, 0x53380d13u, 0x650a7354u, 0x766a0abbu, 0x81c2c92eu, 0x92722c85u,
        0xa2bfe8a1u, 0xa81a664bu, 0xc24b8b70u, 0xc76c51a3u, 0xd192e819u, 0xd6990624u, 0xf40e3585u, 0x106aa070u,
        0x19a4c116u, 0x1e376c08u, 0x2748774cu, 0x34b0bcb5u, 0x391c0cb3u, 0x4ed8aa4au, 0x5b9cca4fu, 0x682e6ff3u,
        0x748f82eeu, 0x78a5636fu, 0x84c87814u, 0x8cc70208u, 0x90befffau, 0xa4506cebu, 0xbef9a3f7u, 0xc67178f2u};
    return k[t];
}

// Stores W[t] + K[t] for the 16 values of the window (t = T0 .. T0+15) to the ring slot.
template <int T0>
__device__ __forceinline__ void store_wk16(const uint32_t (&w)[16], uint32_t dst, uint32_t one) {
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = padd<true>(w[4 * g + j], sha_k(T0 + 4 * g + j), one);
        if (g == 0) tma::st_shared_v4_at<4 * (T0 + 0)>(dst, o[0], o[1], o[2], o[3]);
        if (g == 1) tma::st_shared_v4_at<4 * (T0 + 4)>(dst, o[0], o[1], o[2], o[3]);
        if (g == 2) tma::st_shared_v4_at<4 * (T0 + 8)>(dst, o[0], o[1], o[2], o[3]);
        if (g == 3) tma::st_shared_v4_at<4 * (T0 + 12)>(dst, o[0], o[1], o[2], o[3]);
    }
}

// Sixteen schedule steps: w[i] <- W[t+16] from w[] = W[t .. t+15] (FIPS 180-4 section 6.2.2 step 1).
// Written in two phases so that the many terms that depend only on the old window (all s0
// terms but one, the W[t-16] terms, seven W[t-7] terms) are formed first with full instruction-
// level parallelism, and only the s1 recurrence (two interleaved chains) is left serial.
__device__ __forceinline__ void sched16(uint32_t (&w)[16], uint32_t one) {
    uint32_t c[16];
#pragma unroll
    for (int i = 0; i < 15; ++i) c[i] = padd<true>(small_s0(w[i + 1]), w[i], one);
#pragma unroll
    for (int i = 0; i < 7; ++i) c[i] = padd<true>(c[i], w[i + 9], one);
    const uint32_t w15_old = w[15];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        uint32_t acc = (i < 15) ? c[i] : padd<true>(small_s0(w[0]), w15_old, one);
        if (i >= 7) acc = padd<true>(acc, w[i - 7], one);
        w[i] = padd<true>(acc, small_s1(w[(i + 14) & 15]), one);
    }
}

// All 64 values of one block.
__device__ __forceinline__ void produce_wk(uint32_t (&w)[16], uint32_t dst, uint32_t one) {
    store_wk16<0>(w, dst, one);
    sched16(w, one);
    store_wk16<16>(w, dst, one);
    sched16(w, one);
    store_wk16<32>(w, dst, one);
    sched16(w, one);
    store_wk16<48>(w, dst, one);
}

// One round with kw = W[t] + K[t] already formed.  The ten SHF/LOP3 of a round must run on the ALU pipe.  Of
// the additions, the two that close the state recurrences (e and a) stay three-input ALU adds; the ones that
// feed them from values a round old go to the FMA pipe (`one` is a register that holds 1, so that
// a * one + b is a real multiply-add there).  The fastest of the placements measured.
__device__ __forceinline__ void round_kw(uint32_t a, uint32_t b, uint32_t c, uint32_t &d, uint32_t e, uint32_t f,
                                         uint32_t g, uint32_t &h, uint32_t kw, uint32_t one) {
    const uint32_t x = padd<true>(h, kw, one);
    const uint32_t y = padd<true>(x, f_ch(e, f, g), one);
    const uint32_t s1 = big_s1(e);
    const uint32_t t1 = padd<true>(y, s1, one);
    d = d + y + s1;
    h = t1 + big_s0(a) + f_maj(a, b, c);
}

// Four rounds (T0 a multiple of 4) on W + K values already in registers.
template <int T0>
__device__ __forceinline__ void rounds4(uint32_t (&v)[8], const uint32_t (&k)[4], uint32_t one) {
    constexpr int r = T0 & 7;   // 0 or 4: position in the eight-round rotation of the variable names
    round_kw(v[(8 - r) & 7], v[(9 - r) & 7], v[(10 - r) & 7], v[(11 - r) & 7], v[(12 - r) & 7],
                   v[(13 - r) & 7], v[(14 - r) & 7], v[(15 - r) & 7], k[0], one);
    round_kw(v[(7 - r) & 7], v[(8 - r) & 7], v[(9 - r) & 7], v[(10 - r) & 7], v[(11 - r) & 7],
                   v[(12 - r) & 7], v[(13 - r) & 7], v[(14 - r) & 7], k[1], one);
    round_kw(v[(6 - r) & 7], v[(7 - r) & 7], v[(8 - r) & 7], v[(9 - r) & 7], v[(10 - r) & 7],
                   v[(11 - r) & 7], v[(12 - r) & 7], v[(13 - r) & 7], k[2], one);
    round_kw(v[(5 - r) & 7], v[(6 - r) & 7], v[(7 - r) & 7], v[(8 - r) & 7], v[(9 - r) & 7],
                   v[(10 - r) & 7], v[(11 - r) & 7], v[(12 - r) & 7], k[3], one);
}

// Rounds T0 .. T0+3 with the W + K values of rounds T0+AHEAD .. fetched first (software prefetch).
template <int T0, int AHEAD>
__device__ __forceinline__ void rounds4_step(uint32_t (&v)[8], uint32_t (&kbuf)[16], uint32_t src, uint32_t one) {
    constexpr int TN = T0 + AHEAD;
    if (TN < 64) {
        constexpr int o = TN & 15;
        tma::ld_shared_v4_at<4 * (TN < 64 ? TN : 0)>(src, kbuf[o], kbuf[o + 1], kbuf[o + 2], kbuf[o + 3]);
    }
    const uint32_t k[4] = {kbuf[(T0 & 15)], kbuf[(T0 & 15) + 1], kbuf[(T0 & 15) + 2], kbuf[(T0 & 15) + 3]};
    rounds4<T0>(v, k, one);
}

// All 64 rounds of one block, W[t] + K[t] read from the shared-memory slot at `src`.
__device__ __forceinline__ void rounds64(uint32_t (&v)[8], uint32_t src, uint32_t one) {
    constexpr int AHEAD = 12;          // W + K values are requested three groups of four rounds early
    uint32_t kbuf[16];
    tma::ld_shared_v4_at<0>(src, kbuf[0], kbuf[1], kbuf[2], kbuf[3]);
    tma::ld_shared_v4_at<16>(src, kbuf[4], kbuf[5], kbuf[6], kbuf[7]);
    tma::ld_shared_v4_at<32>(src, kbuf[8], kbuf[9], kbuf[10], kbuf[11]);
    rounds4_step<0, AHEAD>(v, kbuf, src, one);  rounds4_step<4, AHEAD>(v, kbuf, src, one);
    rounds4_step<8, AHEAD>(v, kbuf, src, one);  rounds4_step<12, AHEAD>(v, kbuf, src, one);
    rounds4_step<16, AHEAD>(v, kbuf, src, one); rounds4_step<20, AHEAD>(v, kbuf, src, one);
    rounds4_step<24, AHEAD>(v, kbuf, src, one); rounds4_step<28, AHEAD>(v, kbuf, src, one);
    rounds4_step<32, AHEAD>(v, kbuf, src, one); rounds4_step<36, AHEAD>(v, kbuf, src, one);
    rounds4_step<40, AHEAD>(v, kbuf, src, one); rounds4_step<44, AHEAD>(v, kbuf, src, one);
    rounds4_step<48, AHEAD>(v, kbuf, src, one); rounds4_step<52, AHEAD>(v, kbuf, src, one);
    rounds4_step<56, AHEAD>(v, kbuf, src, one); rounds4_step<60, AHEAD>(v, kbuf, src, one);
}

}  // namespace ivk
