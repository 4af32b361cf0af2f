// Leaf hashing: one SHA-256 compression chain per thread, one chunk per chain
// (Algorithm 1: H_i = GPU_HASH(M_i), FIPS 180-4 section 6.2).
#include "iv_internal.h"
#include "sha256_dev.cuh"

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
__global__ void __launch_bounds__(128, 4)   // the stated minimum only steers the compiler (more registers): +2 to 4 %
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

bool hash_chunks_wants_slices(const uint8_t *d_data, uint64_t chunk_bytes, uint64_t n_chunks, int sm_count) {
    const uint64_t warps = (n_chunks + 31) / 32;
    const bool aligned = ((reinterpret_cast<uintptr_t>(d_data) & 15u) == 0) && (chunk_bytes % 16u == 0);
    return aligned && chunk_bytes >= 4096 && warps > 2ull * (uint64_t)sm_count;
}

cudaError_t launch_hash_chunks(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                               uint64_t n_chunks, uint8_t *d_digests, int sm_count, uint32_t *d_status,
                               const uint32_t *d_one, void *d_slice_scratch, cudaStream_t stream,
                               uint64_t *launches, const char **kernel_used, cudaStream_t tail_stream) {
    if (!tail_stream) tail_stream = stream;
    const char *unused = nullptr;
    if (!kernel_used) kernel_used = &unused;
    if (n_chunks == 0) return cudaSuccess;
    if (launches) ++*launches;
    const uint64_t warps = (n_chunks + 31) / 32;
    const bool aligned = ((reinterpret_cast<uintptr_t>(d_data) & 15u) == 0) && (chunk_bytes % 16u == 0);
    if (aligned && chunk_bytes >= 4096) {
        // Few chains: two warps per 32 chains while every warp can still have an SM scheduler of its own.
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
            // what the tiled copies left out (a short last chunk; everything if the blob could not be described to
            // the TMA unit): one chain per lane through the direct kernel, on tail_stream (beside the main kernel
            // when the caller forked that stream off, after it otherwise)
            if (launches) ++*launches;
            const uint64_t off = covered * chunk_bytes, rest = n_chunks - covered;
            const uint64_t rest_blocks = (rest + 127) / 128;
            if (rest_blocks > 0x7fffffffull) return cudaErrorInvalidConfiguration;
            hash_chunks_kernel<true><<<(unsigned)rest_blocks, 128, 0, tail_stream>>>(d_data + off, nbytes - off, chunk_bytes, rest,
                                                                              d_digests + 32 * covered);
            return cudaGetLastError();
        }
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
