// Microbenchmarks that measure the denominators of the integer roofline on the
// device at hand: lane-operations per clock per SM for the instruction kinds
// SHA-256 is made of, and the cycles one register-only compression takes.
// They time themselves with the SM cycle counter, so the result does not
// depend on the clock the GPU happens to run at.
#include "iv_internal.h"
#include "sha256_dev.cuh"

namespace ivk {
namespace {

constexpr int kChains = 8;      // independent dependency chains per thread
constexpr int kUnroll = 16;     // operations per chain per loop trip

template <int KIND>
__device__ __forceinline__ uint32_t probe_op(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    if (KIND == IV_PROBE_IADD3) {
        asm volatile("{ .reg .u32 t; add.u32 t, %1, %2; add.u32 %0, t, %3; }" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    } else if (KIND == IV_PROBE_LOP3) {
        asm volatile("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    } else if (KIND == IV_PROBE_SHF) {
        asm volatile("shf.r.wrap.b32 %0, %1, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    } else if (KIND == IV_PROBE_PRMT) {
        asm volatile("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    } else {   // IV_PROBE_IMAD: multiply-add with a multiplier the compiler cannot see
        asm volatile("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    }
    return r;
}

// One trip of the mixed kind: a LOP3 and an IMAD per chain, independent pipes.
__device__ __forceinline__ void mixed_pair(uint32_t &x, uint32_t &y, uint32_t b, uint32_t c) {
    x = probe_op<IV_PROBE_LOP3>(x, b, c);
    y = probe_op<IV_PROBE_IMAD>(y, b, c);
}

template <int KIND>
__global__ void probe_kernel(uint32_t iters, uint32_t active_lanes, uint32_t seed_b, uint32_t seed_c,
                             unsigned long long *cycles, uint32_t *sink) {
    const uint32_t lane = threadIdx.x & 31u;
    uint32_t acc[kChains];
#pragma unroll
    for (int k = 0; k < kChains; ++k) acc[k] = threadIdx.x * 2654435761u + k;
    const uint32_t b = seed_b | 1u, c = seed_c;
    __syncthreads();
    const long long t0 = clock64();
    if (lane < active_lanes) {
        for (uint32_t it = 0; it < iters; ++it) {
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                if (KIND == IV_PROBE_MIXED) {
#pragma unroll
                    for (int k = 0; k < kChains; k += 2) mixed_pair(acc[k], acc[k + 1], b, c);
                } else {
#pragma unroll
                    for (int k = 0; k < kChains; ++k) acc[k] = probe_op<KIND>(acc[k], b, c);
                }
            }
        }
    }
    __syncthreads();
    const long long t1 = clock64();
    uint32_t x = 0;
#pragma unroll
    for (int k = 0; k < kChains; ++k) x ^= acc[k];
    if (x == 0x12345u) sink[0] = x;        // keeps the chains alive
    if (threadIdx.x == 0) cycles[blockIdx.x] = (unsigned long long)(t1 - t0);
}

// Register-only SHA-256: `iters` compressions per thread on a block derived from the state.
template <bool FMA>
__global__ void probe_sha_kernel(uint32_t iters, uint32_t active_lanes, uint32_t one, unsigned long long *cycles,
                                 uint32_t *sink) {
    const uint32_t lane = threadIdx.x & 31u;
    uint32_t st[8], w[16];
    sha256_init(st);
    st[0] ^= threadIdx.x + blockIdx.x * blockDim.x;
    __syncthreads();
    const long long t0 = clock64();
    if (lane < active_lanes) {
        for (uint32_t it = 0; it < iters; ++it) {
#pragma unroll
            for (int i = 0; i < 16; ++i) w[i] = __byte_perm(st[i & 7] + (uint32_t)i, it, 0x0123);
            sha256_compress<FMA>(st, w, one);
        }
    }
    __syncthreads();
    const long long t1 = clock64();
    if ((st[0] ^ st[5]) == 0x12345u) sink[0] = st[1];
    if (threadIdx.x == 0) cycles[blockIdx.x] = (unsigned long long)(t1 - t0);
}

}  // namespace

cudaError_t launch_probe(int kind, unsigned blocks, unsigned threads, uint32_t iters, uint32_t active_lanes,
                         unsigned long long *d_cycles, uint32_t *d_sink, cudaStream_t stream) {
    const uint32_t sb = 0x9e3779b9u, sc = 0x7f4a7c15u;
    switch (kind) {
        case IV_PROBE_IADD3: probe_kernel<IV_PROBE_IADD3><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_LOP3: probe_kernel<IV_PROBE_LOP3><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_SHF: probe_kernel<IV_PROBE_SHF><<<blocks, threads, 0, stream>>>(iters, active_lanes, 7u, sc, d_cycles, d_sink); break;
        case IV_PROBE_PRMT: probe_kernel<IV_PROBE_PRMT><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, 0x0123u, d_cycles, d_sink); break;
        case IV_PROBE_IMAD: probe_kernel<IV_PROBE_IMAD><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_MIXED: probe_kernel<IV_PROBE_MIXED><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_SHA256: probe_sha_kernel<false><<<blocks, threads, 0, stream>>>(iters, active_lanes, 1u, d_cycles, d_sink); break;
        case IV_PROBE_SHA256_FMA: probe_sha_kernel<true><<<blocks, threads, 0, stream>>>(iters, active_lanes, 1u, d_cycles, d_sink); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

uint64_t probe_ops_per_thread(int kind, uint32_t iters) {
    if (kind == IV_PROBE_SHA256 || kind == IV_PROBE_SHA256_FMA) return iters;                       // compressions
    return (uint64_t)iters * kUnroll * kChains;                      // instructions
}

}  // namespace ivk
