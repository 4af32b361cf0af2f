// SHA-384 variant of the leaf hashing and of the tree (the digest the paper's own listings use):
// chunk digests of 48 bytes and a binary tree whose parent is SHA-384(left || right) over 96 bytes,
// odd last node promoted.  One compression chain per lane; 128-byte blocks arrive by four-times
// 128-bit loads with the next block in flight during the 80 rounds (any alignment falls back to
// byte loads).  This variant is not tuned like the SHA-256 path: no staging ring, no chain migration.
#include "iv_internal.h"
#include "sha512_dev.cuh"

namespace ivk {
namespace {

template <bool ALIGNED16>
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
    sha384_init(st);
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
    store_digest384(digests + 48 * i, st);
}

// One tree level: parent j = SHA-384(node 2j || node 2j+1), an unpaired last node moves up unchanged.
__global__ void __launch_bounds__(128)
merkle384_level_kernel(const uint8_t *__restrict__ in, uint64_t n, uint8_t *__restrict__ out) {
    const uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t parents = (n + 1) / 2;
    if (j >= parents) return;
    const uint8_t *src = in + 96 * j;
    if (2 * j + 1 >= n) {                       // promotion
        for (int b = 0; b < 48; ++b) out[48 * j + b] = src[b];
        return;
    }
    uint64_t st[8], w[16];
    sha384_init(st);
#pragma unroll
    for (int k = 0; k < 12; ++k) {
        uint64_t v = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) v = (v << 8) | src[8 * k + c];
        w[k] = v;
    }
    w[12] = 0x8000000000000000ull;              // padding of a 96-byte message: one block
    w[13] = 0;
    w[14] = 0;
    w[15] = 96 * 8;
    sha512_compress(st, w);
    store_digest384(out + 48 * j, st);
}

__global__ void sha384_of_nothing_kernel(uint8_t *out) {
    uint64_t st[8], w[16];
    sha384_init(st);
    w[0] = 0x8000000000000000ull;
#pragma unroll
    for (int k = 1; k < 16; ++k) w[k] = 0;
    sha512_compress(st, w);
    store_digest384(out, st);
}

}  // namespace

cudaError_t launch_hash_chunks_sha384(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                                      uint8_t *d_digests, int sm_count, cudaStream_t stream, uint64_t *launches) {
    if (n_chunks == 0) return cudaSuccess;
    const uint64_t warps = (n_chunks + 31) / 32;
    const unsigned warps_per_cta = warps <= (uint64_t)sm_count ? 1u : (warps <= 2ull * sm_count ? 2u : 4u);
    const unsigned threads = 32u * warps_per_cta;
    const uint64_t blocks = (n_chunks + threads - 1) / threads;
    if (blocks > 0x7fffffffull) return cudaErrorInvalidConfiguration;
    const bool aligned = ((reinterpret_cast<uintptr_t>(d_data) & 15u) == 0) && (chunk_bytes % 16u == 0);
    if (aligned)
        hash_chunks_sha384_kernel<true><<<(unsigned)blocks, threads, 0, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests);
    else
        hash_chunks_sha384_kernel<false><<<(unsigned)blocks, threads, 0, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests);
    if (launches) ++*launches;
    return cudaGetLastError();
}

// d_scratch_a / d_scratch_b: ceil(n / 2) records of 48 bytes each.
cudaError_t launch_merkle_root_sha384(const uint8_t *d_leaves, uint64_t n, uint8_t *d_root, uint8_t *d_scratch_a,
                                      uint8_t *d_scratch_b, cudaStream_t stream, uint64_t *launches) {
    if (n == 0) {
        sha384_of_nothing_kernel<<<1, 1, 0, stream>>>(d_root);
        if (launches) ++*launches;
        return cudaGetLastError();
    }
    if (n == 1) return cudaMemcpyAsync(d_root, d_leaves, 48, cudaMemcpyDeviceToDevice, stream);
    const uint8_t *in = d_leaves;
    uint8_t *out = d_scratch_a, *other = d_scratch_b;
    while (n > 1) {
        const uint64_t parents = (n + 1) / 2;
        uint8_t *dst = parents == 1 ? d_root : out;
        merkle384_level_kernel<<<(unsigned)((parents + 127) / 128), 128, 0, stream>>>(in, n, dst);
        if (launches) ++*launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        in = dst;
        uint8_t *t = out; out = other; other = t;
        n = parents;
    }
    return cudaSuccess;
}

}  // namespace ivk
