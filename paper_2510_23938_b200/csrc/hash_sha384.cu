// SHA-384 / SHA-512 variants of the leaf hashing and of the tree (SHA-384 is the digest the paper's own
// listings use): chunk digests of 48 / 64 bytes and a binary tree whose parent is the same hash of
// left || right (96 / 128 bytes), odd last node promoted.  This file holds the plain leaf kernel -- one
// compression chain per lane, 128-byte blocks by 128-bit loads with the next block in flight during the 80
// rounds, byte loads at any alignment -- which serves the shapes the two-warp kernel (hash_sha512_pairs.cu)
// does not take (unaligned blobs, chunks below 4 KiB, a short last chunk), and the tree.
#include "iv_internal.h"
#include "sha512_dev.cuh"

namespace ivk {
namespace {

template <bool ALIGNED16, int DIGEST_WORDS>
__global__ void __launch_bounds__(128)
hash_chunks_sha384_kernel(const uint8_t *__restrict__ data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                          uint8_t *__restrict__ digests) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_chunks) return;
    const uint64_t begin = i * chunk_bytes;
    const uint64_t len = (nbytes - begin < chunk_bytes) ? (nbytes - begin) : chunk_bytes;
    const uint8_t *p = data + begin;
    const uint64_t nfull = len >> 7;

    uint64_t st[8], w[16];
    sha512_family_init<DIGEST_WORDS>(st);
    if (ALIGNED16) {
        uint4 raw[8];
        const uint4 *s = reinterpret_cast<const uint4 *>(p);
        if (nfull) {
#pragma unroll
            for (int q = 0; q < 8; ++q) raw[q] = __ldg(s + q);
        }
        for (uint64_t j = 0; j < nfull; ++j) {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                w[2 * q] = be64(raw[q].x, raw[q].y);
                w[2 * q + 1] = be64(raw[q].z, raw[q].w);
            }
            if (j + 1 < nfull) {
#pragma unroll
                for (int q = 0; q < 8; ++q) raw[q] = __ldg(s + 8 * (j + 1) + q);
            }
            sha512_compress(st, w);
        }
    } else {
        for (uint64_t j = 0; j < nfull; ++j) {
            const uint8_t *b = p + 128 * j;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                uint64_t v = 0;
#pragma unroll
                for (int c = 0; c < 8; ++c) v = (v << 8) | b[8 * k + c];
                w[k] = v;
            }
            sha512_compress(st, w);
        }
    }
    uint64_t tw[32];
    const int nblk = sha512_build_tail(p + 128 * nfull, (uint32_t)(len & 127u), len, tw);
#pragma unroll 1
    for (int t = 0; t < nblk; ++t) {
#pragma unroll
        for (int k = 0; k < 16; ++k) w[k] = tw[16 * t + k];
        sha512_compress(st, w);
    }
    store_digest512<DIGEST_WORDS>(digests + 8 * DIGEST_WORDS * i, st);
}

// One tree level: parent j = H(node 2j || node 2j+1), an unpaired last node moves up unchanged.
template <int DIGEST_WORDS>
__global__ void __launch_bounds__(128)
merkle384_level_kernel(const uint8_t *__restrict__ in, uint64_t n, uint8_t *__restrict__ out) {
    constexpr int REC = 8 * DIGEST_WORDS;
    const uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t parents = (n + 1) / 2;
    if (j >= parents) return;
    const uint8_t *src = in + 2 * REC * j;
    if (2 * j + 1 >= n) {                       // promotion
        for (int b = 0; b < REC; ++b) out[REC * j + b] = src[b];
        return;
    }
    uint64_t st[8], w[16];
    sha512_family_init<DIGEST_WORDS>(st);
#pragma unroll
    for (int k = 0; k < 2 * DIGEST_WORDS; ++k) {
        uint64_t v = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) v = (v << 8) | src[8 * k + c];
        w[k] = v;
    }
    if (DIGEST_WORDS == 6) {
        w[12] = 0x8000000000000000ull;          // padding of a 96-byte message: it fits the same block
        w[13] = 0;
        w[14] = 0;
        w[15] = 96 * 8;
        sha512_compress(st, w);
    } else {
        sha512_compress(st, w);                 // a 128-byte message fills its block; the padding is a block of its own
        w[0] = 0x8000000000000000ull;
#pragma unroll
        for (int k = 1; k < 15; ++k) w[k] = 0;
        w[15] = 128 * 8;
        sha512_compress(st, w);
    }
    store_digest512<DIGEST_WORDS>(out + REC * j, st);
}

template <int DIGEST_WORDS>
__global__ void sha384_of_nothing_kernel(uint8_t *out) {
    uint64_t st[8], w[16];
    sha512_family_init<DIGEST_WORDS>(st);
    w[0] = 0x8000000000000000ull;
#pragma unroll
    for (int k = 1; k < 16; ++k) w[k] = 0;
    sha512_compress(st, w);
    store_digest512<DIGEST_WORDS>(out, st);
}

template <int DIGEST_WORDS>
cudaError_t launch_plain(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks, uint8_t *d_digests,
                         int sm_count, cudaStream_t stream) {
    const uint64_t warps = (n_chunks + 31) / 32;
    const unsigned warps_per_cta = warps <= (uint64_t)sm_count ? 1u : (warps <= 2ull * sm_count ? 2u : 4u);
    const unsigned threads = 32u * warps_per_cta;
    const uint64_t blocks = (n_chunks + threads - 1) / threads;
    if (blocks > 0x7fffffffull) return cudaErrorInvalidConfiguration;
    const bool aligned = ((reinterpret_cast<uintptr_t>(d_data) & 15u) == 0) && (chunk_bytes % 16u == 0);
    if (aligned)
        hash_chunks_sha384_kernel<true, DIGEST_WORDS><<<(unsigned)blocks, threads, 0, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests);
    else
        hash_chunks_sha384_kernel<false, DIGEST_WORDS><<<(unsigned)blocks, threads, 0, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests);
    return cudaGetLastError();
}

template <int DIGEST_WORDS>
cudaError_t merkle_root_wide(const uint8_t *d_leaves, uint64_t n, uint8_t *d_root, uint8_t *d_scratch_a, uint8_t *d_scratch_b,
                             cudaStream_t stream, uint64_t *launches) {
    constexpr int REC = 8 * DIGEST_WORDS;
    if (n == 0) {
        sha384_of_nothing_kernel<DIGEST_WORDS><<<1, 1, 0, stream>>>(d_root);
        if (launches) ++*launches;
        return cudaGetLastError();
    }
    if (n == 1) return cudaMemcpyAsync(d_root, d_leaves, REC, cudaMemcpyDeviceToDevice, stream);
    const uint8_t *in = d_leaves;
    uint8_t *out = d_scratch_a, *other = d_scratch_b;
    while (n > 1) {
        const uint64_t parents = (n + 1) / 2;
        uint8_t *dst = parents == 1 ? d_root : out;
        merkle384_level_kernel<DIGEST_WORDS><<<(unsigned)((parents + 127) / 128), 128, 0, stream>>>(in, n, dst);
        if (launches) ++*launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        in = dst;
        uint8_t *t = out; out = other; other = t;
        n = parents;
    }
    return cudaSuccess;
}

}  // namespace

// digest_words = 6 (SHA-384) or 8 (SHA-512).  With d_pairs_scratch (sha512_pairs_scratch_bytes(...) bytes) and a
// shape the two-warp kernel takes (sha512_wants_pairs) the whole chunks go through it, the rest -- and every
// other shape -- through the plain kernel.
cudaError_t launch_hash_chunks_sha384(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                                      uint8_t *d_digests, int digest_words, int sm_count, uint32_t *d_status,
                                      void *d_pairs_scratch, cudaStream_t stream, uint64_t *launches,
                                      const char **kernel_used, cudaStream_t tail_stream) {
    if (n_chunks == 0) return cudaSuccess;
    if (!tail_stream || !d_pairs_scratch) tail_stream = stream;
    uint64_t covered = 0;
    if (kernel_used) *kernel_used = "hash_chunks_sha384_kernel";
    if (d_pairs_scratch && sha512_wants_pairs(d_data, nbytes, chunk_bytes, sm_count)) {
        cudaError_t e = launch_hash_sha512_pairs(d_data, nbytes, chunk_bytes, d_digests, digest_words, d_status,
                                                 d_pairs_scratch, sm_count, stream, &covered, launches);
        if (e != cudaSuccess) return e;
        if (covered && kernel_used) *kernel_used = "hash_sha512_pairs_kernel";
        if (covered == n_chunks) return cudaSuccess;
    }
    const uint64_t off = covered * chunk_bytes, rec = 8ull * (uint64_t)digest_words;
    if (launches) ++*launches;
    cudaStream_t s = covered ? tail_stream : stream;        // what the two-warp kernel left out runs beside it
    return digest_words == 6 ? launch_plain<6>(d_data + off, nbytes - off, chunk_bytes, n_chunks - covered, d_digests + rec * covered, sm_count, s)
                             : launch_plain<8>(d_data + off, nbytes - off, chunk_bytes, n_chunks - covered, d_digests + rec * covered, sm_count, s);
}

// d_scratch_a / d_scratch_b: ceil(n / 2) records each.
cudaError_t launch_merkle_root_sha384(const uint8_t *d_leaves, uint64_t n, uint8_t *d_root, uint8_t *d_scratch_a,
                                      uint8_t *d_scratch_b, int digest_words, cudaStream_t stream, uint64_t *launches) {
    return digest_words == 6 ? merkle_root_wide<6>(d_leaves, n, d_root, d_scratch_a, d_scratch_b, stream, launches)
                             : merkle_root_wide<8>(d_leaves, n, d_root, d_scratch_a, d_scratch_b, stream, launches);
}

}  // namespace ivk
