// Leaf hashing: one SHA-256 compression chain per thread, one chunk per chain
// (Algorithm 1: H_i = GPU_HASH(M_i), FIPS 180-4 section 6.2).
#include "iv_internal.h"
#include "sha256_dev.cuh"
#include "tma_dev.cuh"

namespace ivk {

// 64 message bytes at a 16-byte aligned address, as four 128-bit loads.
struct RawBlock16 {
    uint4 q[4];
    __device__ __forceinline__ void load(const uint8_t *p) {
        const uint4 *s = reinterpret_cast<const uint4 *>(p);
        q[0] = __ldg(s + 0); q[1] = __ldg(s + 1); q[2] = __ldg(s + 2); q[3] = __ldg(s + 3);
    }
    __device__ __forceinline__ void to_words(uint32_t (&w)[16]) const {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            w[4 * i + 0] = bswap32(q[i].x); w[4 * i + 1] = bswap32(q[i].y);
            w[4 * i + 2] = bswap32(q[i].z); w[4 * i + 3] = bswap32(q[i].w);
        }
    }
};

// 64 message bytes at ANY address: the 16 (or 17) aligned 32-bit words that
// cover them; one PRMT per output word does the byte shift and the endian swap.
struct RawBlockAny {
    uint32_t x[17];
    __device__ __forceinline__ void load(const uint8_t *p) {
        const uintptr_t a = reinterpret_cast<uintptr_t>(p);
        const uint32_t s = (uint32_t)(a & 3u);
        const uint32_t *q = reinterpret_cast<const uint32_t *>(a - s);
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = __ldg(q + i);
        x[16] = s ? __ldg(q + 16) : 0u;   // never touch the word after an aligned block
    }
    __device__ __forceinline__ void to_words(uint32_t (&w)[16], uint32_t sel) const {
#pragma unroll
        for (int i = 0; i < 16; ++i) w[i] = __byte_perm(x[i], x[i + 1], sel);
    }
};

// PRMT selector for "big-endian word starting s bytes into the pair (lo, hi)".
__device__ __forceinline__ uint32_t be_selector(uint32_t s) { return 0x0123u + 0x1111u * s; }

template <bool ALIGNED16>
__global__ void __launch_bounds__(128)
hash_chunks_kernel(const uint8_t *__restrict__ data, uint64_t nbytes, uint64_t chunk_bytes,
                   uint64_t n_chunks, uint8_t *__restrict__ digests) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_chunks) return;
    const uint64_t begin = i * chunk_bytes;
    const uint64_t len = (nbytes - begin < chunk_bytes) ? (nbytes - begin) : chunk_bytes;
    const uint8_t *p = data + begin;
    const uint64_t nfull = len >> 6;

    uint32_t st[8];
    sha256_init(st);
    uint32_t w[16];

    if (ALIGNED16) {
        RawBlock16 raw;
        if (nfull) raw.load(p);
        for (uint64_t j = 0; j < nfull; ++j) {
            raw.to_words(w);
            if (j + 1 < nfull) raw.load(p + 64 * (j + 1));   // next block in flight during the rounds
            sha256_compress(st, w);
        }
    } else {
        const uint32_t sel = be_selector((uint32_t)(reinterpret_cast<uintptr_t>(p) & 3u));
        RawBlockAny raw;
        if (nfull) raw.load(p);
        for (uint64_t j = 0; j < nfull; ++j) {
            raw.to_words(w, sel);
            if (j + 1 < nfull) raw.load(p + 64 * (j + 1));
            sha256_compress(st, w);
        }
    }

    const uint32_t rem = (uint32_t)(len & 63u);
    if (rem == 0) {
        sha256_pad_only_block(w, len);
        sha256_compress(st, w);
    } else {
        uint32_t tw[32];
        const int nblk = sha256_build_tail(p + 64 * nfull, rem, len, tw);
#pragma unroll
        for (int k = 0; k < 16; ++k) w[k] = tw[k];
        sha256_compress(st, w);
        if (nblk == 2) {
#pragma unroll
            for (int k = 0; k < 16; ++k) w[k] = tw[16 + k];
            sha256_compress(st, w);
        }
    }
    store_digest(digests + 32 * i, st);
}

// ---------------------------------------------------------------------------
// Staged variant (base and chunk size multiples of 16 bytes).
//
// Global memory is chunk-major: the 32 lanes of a warp read 32 streams that lie
// chunk_bytes apart.  Each lane fetches its own stream in segments of SEG bytes
// with one bulk asynchronous copy (TMA, cp.async.bulk) into a per-warp ring in
// shared memory, completion counted by one mbarrier per stage, several stages
// ahead of the compression.  In shared memory the segments are lane-interleaved
// with a stride of SEG + 16 bytes, so the four 128-bit loads that fetch a
// 64-byte block are bank-conflict free.  A request of SEG bytes amortises the
// DRAM/TLB latency of a stream over SEG/64 compressions.
// ---------------------------------------------------------------------------

template <int SEG, int STAGES, int WARPS, bool FMA>
__global__ void __launch_bounds__(32 * WARPS)
hash_chunks_staged_kernel(const uint8_t *__restrict__ data, uint64_t nbytes, uint64_t chunk_bytes,
                          uint64_t n_chunks, uint8_t *__restrict__ digests, uint32_t one,
                          uint32_t *__restrict__ status) {
    constexpr uint32_t kLaneStride = SEG + 16;
    constexpr uint32_t kStageBytes = 32 * kLaneStride;
    constexpr int kBlocksPerSeg = SEG / 64;
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ __align__(8) uint64_t bars[WARPS][STAGES];

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    const uint32_t ring_base = tma::smem_u32(ring) + warp * (STAGES * kStageBytes) + lane * kLaneStride;
    const uint32_t bar_base = tma::smem_u32(&bars[warp][0]);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) tma::mbar_init(bar_base + 8 * s, 32);
        tma::fence_barrier_init();
    }
    __syncwarp();

    const uint64_t i = ((uint64_t)blockIdx.x * WARPS + warp) * 32 + lane;
    const bool valid = i < n_chunks;
    const uint64_t begin = valid ? i * chunk_bytes : 0;
    const uint64_t len = valid ? ((nbytes - begin < chunk_bytes) ? (nbytes - begin) : chunk_bytes) : 0;
    const uint8_t *p = data + begin;
    const uint64_t full_bytes = len & ~63ull;
    // Only the last chunk of the blob can be shorter, so lane 0 has the most segments of its warp.
    const uint64_t nseg = __shfl_sync(0xffffffffu, (full_bytes + SEG - 1) / SEG, 0);

    auto issue = [&](uint64_t seg, int stage) {
        const uint64_t off = seg * SEG;
        const uint32_t bar = bar_base + 8 * stage;
        if (off < full_bytes) {
            const uint32_t bytes = (uint32_t)((full_bytes - off < SEG) ? (full_bytes - off) : SEG);
            tma::mbar_arrive_expect_tx(bar, bytes);
            tma::bulk_g2s(ring_base + stage * kStageBytes, p + off, bytes, bar);
        } else {
            tma::mbar_arrive(bar);
        }
    };
#pragma unroll
    for (int s = 0; s < STAGES; ++s)
        if ((uint64_t)s < nseg) issue(s, s);

    // Flat loop over the warp's blocks.  The 64 bytes of block k+1 are fetched from the ring into
    // registers before the rounds of block k run, so neither the shared-memory latency nor the
    // stage hand-over sits on the chain's critical path.
    uint32_t st[8], w[16], raw[16];
    sha256_init(st);
    const uint64_t my_blocks = full_bytes >> 6;
    const uint64_t warp_blocks = __shfl_sync(0xffffffffu, my_blocks, 0);
    int stage = 0, in_stage = 0;
    uint32_t parity = 0;
    bool failed = false;
    auto fetch = [&](int blk_in_stage) {
        const uint32_t src = ring_base + stage * kStageBytes + 64 * blk_in_stage;
#pragma unroll
        for (int q = 0; q < 4; ++q)
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(raw[4 * q]), "=r"(raw[4 * q + 1]), "=r"(raw[4 * q + 2]), "=r"(raw[4 * q + 3])
                         : "r"(src + 16 * q));
    };
    if (warp_blocks) {
        failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded(bar_base, 0));
        if (!failed) fetch(0);
    }
    uint64_t next_seg = STAGES;                      // next segment to request
    for (uint64_t blk = 0; blk < warp_blocks && !failed; ++blk) {
#pragma unroll
        for (int k = 0; k < 16; ++k) w[k] = bswap32(raw[k]);
        if (blk + 1 < warp_blocks) {
            if (++in_stage == kBlocksPerSeg) {       // block blk was the last one of its stage
                in_stage = 0;
                __syncwarp();                        // every lane has taken its data out of the stage
                if (next_seg < nseg) issue(next_seg, stage);
                ++next_seg;
                if (++stage == STAGES) { stage = 0; parity ^= 1u; }
                failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded(bar_base + 8 * stage, parity));
                if (failed) break;
            }
            fetch(in_stage);
        }
        if (blk < my_blocks) sha256_compress<FMA>(st, w, one);
    }
    if (failed) {
        // Give copies still in flight a bounded chance to land before the ring is released.
        for (int s = 0; s < STAGES; ++s) (void)tma::mbar_wait_bounded(bar_base + 8 * s, 0);
        if (lane == 0) atomicExch(status, (uint32_t)IVK_DEV_TIMEOUT);
        return;
    }
    if (!valid) return;

    const uint32_t rem = (uint32_t)(len & 63u);
    if (rem == 0) {
        sha256_pad_only_block(w, len);
        sha256_compress<FMA>(st, w, one);
    } else {
        uint32_t tw[32];
        const int nblk = sha256_build_tail(p + full_bytes, rem, len, tw);
#pragma unroll 1
        for (int t = 0; t < nblk; ++t) {
#pragma unroll
            for (int k = 0; k < 16; ++k) w[k] = tw[16 * t + k];
            sha256_compress<FMA>(st, w, one);
        }
    }
    store_digest(digests + 32 * i, st);
}

template <int SEG, int STAGES, int WARPS, bool FMA>
cudaError_t launch_staged(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                          uint8_t *d_digests, uint32_t *d_status, cudaStream_t stream) {
    constexpr size_t smem = (size_t)WARPS * STAGES * 32 * (SEG + 16);
    auto kernel = hash_chunks_staged_kernel<SEG, STAGES, WARPS, FMA>;
    static bool configured[kMaxDevices] = {};
    if (cudaError_t e0 = ensure_dynamic_smem(kernel, smem, configured); e0 != cudaSuccess) return e0;
    const uint64_t per_cta = 32ull * WARPS;
    const uint64_t blocks = (n_chunks + per_cta - 1) / per_cta;
    if (blocks > 0x7fffffffull) return cudaErrorInvalidConfiguration;
    kernel<<<(unsigned)blocks, 32 * WARPS, smem, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests, 1u, d_status);
    return cudaGetLastError();
}

bool hash_chunks_wants_slices(const uint8_t *d_data, uint64_t chunk_bytes, uint64_t n_chunks, int sm_count) {
    const uint64_t warps = (n_chunks + 31) / 32;
    const bool aligned = ((reinterpret_cast<uintptr_t>(d_data) & 15u) == 0) && (chunk_bytes % 16u == 0);
    return aligned && chunk_bytes >= 4096 && warps > 2ull * (uint64_t)sm_count;
}

cudaError_t launch_hash_chunks(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                               uint64_t n_chunks, uint8_t *d_digests, int sm_count, uint32_t *d_status,
                               const uint32_t *d_one, void *d_slice_scratch, cudaStream_t stream,
                               uint64_t *launches, const char **kernel_used) {
    const char *unused = nullptr;
    if (!kernel_used) kernel_used = &unused;
    if (n_chunks == 0) return cudaSuccess;
    if (launches) ++*launches;
    const uint64_t warps = (n_chunks + 31) / 32;
    const bool aligned = ((reinterpret_cast<uintptr_t>(d_data) & 15u) == 0) && (chunk_bytes % 16u == 0);
    if (aligned && chunk_bytes >= 4096) {
        // Few chains: one warp per CTA, so every chain warp gets an SM scheduler of its own and a deep ring.
        // Two warps per 32 chains while every warp can still have an SM scheduler of its own.
        if (warps <= 2ull * sm_count) {
            *kernel_used = "hash_chunks_split_kernel";
            return launch_hash_chunks_split(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, d_one, stream);
        }
        // Many chains of sliceable size: chains migrate between schedulers (two launches: queue set-up + workers).
        if (d_slice_scratch && hash_chunks_wants_slices(d_data, chunk_bytes, n_chunks, sm_count)) {
            if (launches) ++*launches;
            // just above 2 x SMs groups: the two-warp pairs as workers on the slice FIFO
            if (hash_chunks_wants_pairs(d_data, chunk_bytes, n_chunks, sm_count)) {
                *kernel_used = "hash_chunks_pairs_kernel";
                return launch_hash_chunks_pairs(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status,
                                                d_slice_scratch, d_one, sm_count, stream);
            }
            *kernel_used = "hash_chunks_sliced_kernel";
            uint64_t covered = 0;
            cudaError_t e = launch_hash_chunks_sliced(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status,
                                                      d_slice_scratch, d_one, sm_count, stream, &covered);
            if (e != cudaSuccess || covered == n_chunks) return e;
            // a short last chunk, left out by the tiled copies: one chain through the direct kernel
            if (launches) ++*launches;
            const uint64_t off = covered * chunk_bytes;
            hash_chunks_kernel<true><<<1, 32, 0, stream>>>(d_data + off, nbytes - off, chunk_bytes, 1,
                                                          d_digests + 32 * covered);
            return cudaGetLastError();
        }
        // (no scratch supplied) two CTAs of four warps per SM keep two warps on every scheduler.
        *kernel_used = "hash_chunks_staged_kernel";
        if (warps <= 4ull * sm_count)
            return launch_staged<512, 3, 1, false>(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, stream);
        return launch_staged<256, 3, 4, false>(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, stream);
    }
    *kernel_used = "hash_chunks_kernel";
    const unsigned warps_per_cta = warps <= (uint64_t)sm_count ? 1u : (warps <= 2ull * sm_count ? 2u : 4u);
    const unsigned threads = 32u * warps_per_cta;
    const uint64_t blocks = (n_chunks + threads - 1) / threads;
    if (blocks > 0x7fffffffull) return cudaErrorInvalidConfiguration;
    if (aligned)
        hash_chunks_kernel<true><<<(unsigned)blocks, threads, 0, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests);
    else
        hash_chunks_kernel<false><<<(unsigned)blocks, threads, 0, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests);
    return cudaGetLastError();
}

}  // namespace ivk
