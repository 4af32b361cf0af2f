// Microbenchmarks that measure the denominators of the integer roofline on the
// device at hand: lane-operations per clock per SM for the instruction kinds
// SHA-256 is made of, and the cycles one register-only compression takes.
// They time themselves with the SM cycle counter, so the result does not
// depend on the clock the GPU happens to run at.
#include "iv_internal.h"
#include "sha256_dev.cuh"
#include "sha256_split_dev.cuh"

namespace ivk {
namespace {

constexpr int kThroughputChains = 8;   // independent dependency chains per thread (throughput kinds)
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

template <int KIND, int kChains>
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
                if (KIND == IV_PROBE_LAT_CROSS) {
                    // one chain that alternates pipes: ALU result -> FMA pipe -> ALU pipe ...
                    acc[0] = probe_op<IV_PROBE_LOP3>(acc[0], b, c);
                    acc[0] = probe_op<IV_PROBE_IMAD>(acc[0], b, c);
                } else if (KIND == IV_PROBE_MIXED) {
#pragma unroll
                    for (int k = 0; k + 1 < kChains; k += 2) mixed_pair(acc[k], acc[k + 1], b, c);
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
template <int ADD>
__global__ void probe_sha_kernel(uint32_t iters, uint32_t active_lanes, unsigned long long *cycles, uint32_t *sink) {
    const uint32_t one = sink[1];        // the host stored 1 there; the compiler cannot know
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
            sha256_compress<ADD>(st, w, one);
        }
    }
    __syncthreads();
    const long long t1 = clock64();
    if ((st[0] ^ st[5]) == 0x12345u) sink[0] = st[1];
    if (threadIdx.x == 0) cycles[blockIdx.x] = (unsigned long long)(t1 - t0);
}

// The consumer half of the two-warp kernel alone: 64 rounds per trip, W + K read from a (constant)
// shared-memory slot.
__global__ void probe_rounds_kernel(uint32_t iters, uint32_t active_lanes, unsigned long long *cycles, uint32_t *sink) {
    __shared__ __align__(16) uint32_t slot[32 * 68];
    for (int i = threadIdx.x; i < 32 * 68; i += blockDim.x) slot[i] = i * 2654435761u;
    __syncthreads();
    const uint32_t one = sink[1];        // the host stored 1 there; the compiler cannot know
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t src = tma::smem_u32(slot) + lane * 272;
    uint32_t v[8];
    sha256_init(v);
    v[0] ^= threadIdx.x;
    const long long t0 = clock64();
    if (lane < active_lanes)
        for (uint32_t it = 0; it < iters; ++it) rounds64(v, src, one);
    __syncthreads();
    const long long t1 = clock64();
    if ((v[0] ^ v[5]) == 0x12345u) sink[0] = v[1];
    if (threadIdx.x == 0) cycles[blockIdx.x] = (unsigned long long)(t1 - t0);
}

// The producer half alone: W + K of one block per trip into a shared-memory slot.
__global__ void probe_schedule_kernel(uint32_t iters, uint32_t active_lanes, unsigned long long *cycles, uint32_t *sink) {
    __shared__ __align__(16) uint32_t slot[32 * 68];
    const uint32_t one = sink[1];        // the host stored 1 there; the compiler cannot know
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t dst = tma::smem_u32(slot) + lane * 272;
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) w[i] = threadIdx.x * 40503u + i;
    const long long t0 = clock64();
    if (lane < active_lanes)
        for (uint32_t it = 0; it < iters; ++it) {
#pragma unroll
            for (int i = 0; i < 16; ++i) w[i] = bswap32(w[i] ^ it);
            produce_wk(w, dst, one);
        }
    __syncthreads();
    const long long t1 = clock64();
    if ((w[0] ^ w[5] ^ slot[threadIdx.x]) == 0x12345u) sink[0] = w[1];
    if (threadIdx.x == 0) cycles[blockIdx.x] = (unsigned long long)(t1 - t0);
}

}  // namespace

cudaError_t launch_probe(int kind, unsigned blocks, unsigned threads, uint32_t iters, uint32_t active_lanes,
                         unsigned long long *d_cycles, uint32_t *d_sink, cudaStream_t stream) {
    const uint32_t sb = 0x9e3779b9u, sc = 0x7f4a7c15u;
    switch (kind) {
        case IV_PROBE_IADD3: probe_kernel<IV_PROBE_IADD3, kThroughputChains><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_LOP3: probe_kernel<IV_PROBE_LOP3, kThroughputChains><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_SHF: probe_kernel<IV_PROBE_SHF, kThroughputChains><<<blocks, threads, 0, stream>>>(iters, active_lanes, 7u, sc, d_cycles, d_sink); break;
        case IV_PROBE_PRMT: probe_kernel<IV_PROBE_PRMT, kThroughputChains><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, 0x0123u, d_cycles, d_sink); break;
        case IV_PROBE_IMAD: probe_kernel<IV_PROBE_IMAD, kThroughputChains><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_MIXED: probe_kernel<IV_PROBE_MIXED, kThroughputChains><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_LAT_IADD3: probe_kernel<IV_PROBE_IADD3, 1><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_LAT_LOP3: probe_kernel<IV_PROBE_LOP3, 1><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_LAT_SHF: probe_kernel<IV_PROBE_SHF, 1><<<blocks, threads, 0, stream>>>(iters, active_lanes, 7u, sc, d_cycles, d_sink); break;
        case IV_PROBE_LAT_IMAD: probe_kernel<IV_PROBE_IMAD, 1><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_LAT_CROSS: probe_kernel<IV_PROBE_LAT_CROSS, 1><<<blocks, threads, 0, stream>>>(iters, active_lanes, sb, sc, d_cycles, d_sink); break;
        case IV_PROBE_ROUNDS: probe_rounds_kernel<<<blocks, threads, 0, stream>>>(iters, active_lanes, d_cycles, d_sink); break;
        case IV_PROBE_SCHEDULE: probe_schedule_kernel<<<blocks, threads, 0, stream>>>(iters, active_lanes, d_cycles, d_sink); break;
        case IV_PROBE_SHA256: probe_sha_kernel<0><<<blocks, threads, 0, stream>>>(iters, active_lanes, d_cycles, d_sink); break;
        case IV_PROBE_SHA256_SCHED_FMA: probe_sha_kernel<2><<<blocks, threads, 0, stream>>>(iters, active_lanes, d_cycles, d_sink); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

bool probe_counts_blocks(int kind) {
    return kind == IV_PROBE_SHA256 || kind == IV_PROBE_SHA256_SCHED_FMA || kind == IV_PROBE_ROUNDS || kind == IV_PROBE_SCHEDULE;
}

uint64_t probe_ops_per_thread(int kind, uint32_t iters) {
    if (probe_counts_blocks(kind)) return iters;                                      // compressions
    if (kind == IV_PROBE_LAT_CROSS) return (uint64_t)iters * kUnroll * 2;             // two instructions per trip
    if (kind >= IV_PROBE_LAT_IADD3) return (uint64_t)iters * kUnroll;                 // one dependent chain
    return (uint64_t)iters * kUnroll * kThroughputChains;                              // instructions
}

}  // namespace ivk
