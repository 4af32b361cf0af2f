// RFC 6962 section 2.1 mode (the tree construction the paper cites): leaf hash = SHA-256(0x00 || chunk),
// node = SHA-256(0x01 || left || right), empty list = SHA-256(""), one entry = its leaf hash, the list
// split at the largest power of two below n (the same shape as pairing level by level with the odd
// last node moved up).  The prefix shifts every message by one byte against the data: message word k of
// a block is the last byte of the previous data word followed by the first three bytes of data word
// k, which one PRMT per word produces together with the endian swap, so the shift costs nothing.
#include "iv_internal.h"
#include "rfc6962_dev.cuh"
#include "sha256_dev.cuh"

namespace ivk {
namespace {

template <bool ALIGNED16>
__global__ void __launch_bounds__(128)
hash_chunks_rfc6962_kernel(const uint8_t *__restrict__ data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                           uint8_t *__restrict__ digests) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_chunks) return;
    const uint64_t begin = i * chunk_bytes;
    const uint64_t len = (nbytes - begin < chunk_bytes) ? (nbytes - begin) : chunk_bytes;
    const uint8_t *p = data + begin;
    const uint64_t msg_bytes = len + 1;
    // Message block j takes data bytes 64j-1 .. 64j+62; the fast loop runs while data block j is whole.
    const uint64_t msg_full = msg_bytes >> 6, data_full = len >> 6;
    const uint64_t nfast = msg_full < data_full ? msg_full : data_full;

    uint32_t st[8], w[16];
    sha256_init(st);
    if (ALIGNED16) {
        uint4 raw[4];
        const uint4 *s = reinterpret_cast<const uint4 *>(p);
        uint32_t carry = 0u;                     // byte 3 of it is the byte before the block: the 0x00 prefix first
        if (nfast) {
#pragma unroll
            for (int q = 0; q < 4; ++q) raw[q] = __ldg(s + q);
        }
        for (uint64_t j = 0; j < nfast; ++j) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                w[4 * q + 0] = shifted_word(raw[q].x, q ? raw[q - 1].w : carry);
                w[4 * q + 1] = shifted_word(raw[q].y, raw[q].x);
                w[4 * q + 2] = shifted_word(raw[q].z, raw[q].y);
                w[4 * q + 3] = shifted_word(raw[q].w, raw[q].z);
            }
            carry = raw[3].w;
            if (j + 1 < nfast) {
#pragma unroll
                for (int q = 0; q < 4; ++q) raw[q] = __ldg(s + 4 * (j + 1) + q);
            }
            sha256_compress(st, w);
        }
    } else {
        uint32_t before = 0u;                    // the byte in front of the block
        for (uint64_t j = 0; j < nfast; ++j) {
            const uint8_t *b = p + 64 * j;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                w[k] = (before << 24) | ((uint32_t)b[4 * k] << 16) | ((uint32_t)b[4 * k + 1] << 8) | b[4 * k + 2];
                before = b[4 * k + 3];
            }
            sha256_compress(st, w);
        }
    }
    uint32_t tw[32];
    const int nblk = prefixed_tail(p, 0x00, 64 * nfast, msg_bytes, tw);
#pragma unroll 1
    for (int t = 0; t < nblk; ++t) {
#pragma unroll
        for (int k = 0; k < 16; ++k) w[k] = tw[16 * t + k];
        sha256_compress(st, w);
    }
    store_digest(digests + 32 * i, st);
}

// One tree level: parent j = SHA-256(0x01 || node 2j || node 2j+1), 65 bytes in two blocks; an
// unpaired last node moves up unchanged.
__global__ void __launch_bounds__(128)
merkle_rfc6962_level_kernel(const uint8_t *__restrict__ in, uint64_t n, uint8_t *__restrict__ out) {
    const uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t parents = (n + 1) / 2;
    if (j >= parents) return;
    const uint8_t *src = in + 64 * j;
    if (2 * j + 1 >= n) {
        for (int b = 0; b < 32; ++b) out[32 * j + b] = src[b];
        return;
    }
    uint32_t st[8], w[16];
    sha256_init(st);
    uint32_t before = 0x01u;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        w[k] = (before << 24) | ((uint32_t)src[4 * k] << 16) | ((uint32_t)src[4 * k + 1] << 8) | src[4 * k + 2];
        before = src[4 * k + 3];
    }
    sha256_compress(st, w);
    w[0] = (before << 24) | 0x00800000u;         // last byte of the right child, then the padding
#pragma unroll
    for (int k = 1; k < 15; ++k) w[k] = 0u;
    w[15] = 65u * 8u;
    sha256_compress(st, w);
    store_digest(out + 32 * j, st);
}

__global__ void sha256_of_nothing_kernel(uint8_t *out) {
    uint32_t st[8], w[16];
    sha256_init(st);
    sha256_pad_only_block(w, 0);
    sha256_compress(st, w);
    store_digest(out, st);
}

}  // namespace

namespace {
cudaError_t launch_direct(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                          uint8_t *d_digests, int sm_count, cudaStream_t stream) {
    const uint64_t warps = (n_chunks + 31) / 32;
    const unsigned warps_per_cta = warps <= (uint64_t)sm_count ? 1u : (warps <= 2ull * sm_count ? 2u : 4u);
    const unsigned threads = 32u * warps_per_cta;
    const uint64_t blocks = (n_chunks + threads - 1) / threads;
    if (blocks > 0x7fffffffull) return cudaErrorInvalidConfiguration;
    const bool aligned = ((reinterpret_cast<uintptr_t>(d_data) & 15u) == 0) && (chunk_bytes % 16u == 0);
    if (aligned)
        hash_chunks_rfc6962_kernel<true><<<(unsigned)blocks, threads, 0, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests);
    else
        hash_chunks_rfc6962_kernel<false><<<(unsigned)blocks, threads, 0, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests);
    return cudaGetLastError();
}
}  // namespace

cudaError_t launch_hash_chunks_rfc6962(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                                       uint8_t *d_digests, int sm_count, uint32_t *d_status, const uint32_t *d_one,
                                       void *d_slice_scratch, cudaStream_t stream, uint64_t *launches,
                                       const char **kernel_used, cudaStream_t tail_stream) {
    if (n_chunks == 0) return cudaSuccess;
    if (!tail_stream) tail_stream = stream;
    const bool aligned = ((reinterpret_cast<uintptr_t>(d_data) & 15u) == 0) && (chunk_bytes % 16u == 0);
    if (aligned && chunk_bytes >= 4096 && (n_chunks + 31) / 32 <= 2ull * (uint64_t)sm_count) {
        // few chains: the two-warp kernel, prefixed
        if (launches) ++*launches;
        if (kernel_used) *kernel_used = "hash_chunks_split_kernel";
        return launch_hash_chunks_split(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, d_one, stream, true);
    }
    if (d_slice_scratch && hash_chunks_wants_slices(d_data, chunk_bytes, n_chunks, sm_count)) {
        if (launches) *launches += 2;
        if (hash_chunks_wants_pairs(d_data, chunk_bytes, n_chunks, sm_count)) {
            if (kernel_used) *kernel_used = "hash_chunks_pairs_kernel";
            return launch_hash_chunks_pairs(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, d_slice_scratch,
                                            d_one, sm_count, stream, true);
        }
        // many chains that do not divide evenly over the schedulers: the migrating kernel, prefixed
        if (kernel_used) *kernel_used = "hash_chunks_sliced_kernel";
        uint64_t covered = 0;
        cudaError_t e = launch_hash_chunks_sliced(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status,
                                                  d_slice_scratch, d_one, sm_count, stream, &covered, true);
        if (e != cudaSuccess || covered == n_chunks) return e;
        if (launches) ++*launches;
        const uint64_t off = covered * chunk_bytes;
        return launch_direct(d_data + off, nbytes - off, chunk_bytes, n_chunks - covered, d_digests + 32 * covered,
                             sm_count, tail_stream);
    }
    if (launches) ++*launches;
    if (kernel_used) *kernel_used = "hash_chunks_rfc6962_kernel";
    return launch_direct(d_data, nbytes, chunk_bytes, n_chunks, d_digests, sm_count, stream);
}

// d_scratch_a / d_scratch_b: ceil(n / 2) records of 32 bytes each.
cudaError_t launch_merkle_root_rfc6962(const uint8_t *d_leaves, uint64_t n, uint8_t *d_root, uint8_t *d_scratch_a,
                                       uint8_t *d_scratch_b, cudaStream_t stream, uint64_t *launches) {
    if (n == 0) {
        sha256_of_nothing_kernel<<<1, 1, 0, stream>>>(d_root);
        if (launches) ++*launches;
        return cudaGetLastError();
    }
    if (n == 1) return cudaMemcpyAsync(d_root, d_leaves, 32, cudaMemcpyDeviceToDevice, stream);
    const uint8_t *in = d_leaves;
    uint8_t *out = d_scratch_a, *other = d_scratch_b;
    while (n > 1) {
        const uint64_t parents = (n + 1) / 2;
        uint8_t *dst = parents == 1 ? d_root : out;
        merkle_rfc6962_level_kernel<<<(unsigned)((parents + 127) / 128), 128, 0, stream>>>(in, n, dst);
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
