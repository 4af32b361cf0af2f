// Per-tensor digests: one SHA-256 per (offset, length) over a common base
// buffer (the paper's batch verification: one digest per payload).
//
// Messages have very different lengths, so lanes do not own a fixed message:
// each lane pops the next message index from a device-wide counter when its
// current message ends.  Every trip round the loop is "produce the next
// 64-byte block (data, or tail with padding), then one compression", so lanes
// at different points of their messages still share one instruction stream.
#include "iv_internal.h"
#include "sha256_dev.cuh"

namespace ivk {

namespace {

__device__ __forceinline__ uint32_t be_selector(uint32_t s) { return 0x0123u + 0x1111u * s; }

// The 16 (or 17) aligned words covering 64 bytes at any address.
__device__ __forceinline__ void load_raw(const uint8_t *p, uint32_t (&x)[17]) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    const uint32_t s = (uint32_t)(a & 3u);
    const uint32_t *q = reinterpret_cast<const uint32_t *>(a - s);
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] = __ldg(q + i);
    x[16] = s ? __ldg(q + 16) : 0u;
}

__global__ void __launch_bounds__(128, 4)   // the stated minimum only steers the compiler (more registers): 708 against 651 GB/s
hash_ragged_kernel(const uint8_t *__restrict__ base, const uint64_t *__restrict__ offsets,
                   const uint64_t *__restrict__ lengths, uint64_t n, uint8_t *__restrict__ digests,
                   unsigned long long *queue) {
    uint32_t st[8], w[16], raw[17];
    uint32_t tw[32];                       // tail blocks (local memory, touched once per message)
    const uint8_t *p = nullptr;
    uint64_t len = 0, nfull = 0, j = 0, idx = 0;
    uint32_t sel = 0x0123u;
    int tail_blocks = 0, tail_pos = 0;
    bool busy = false, exhausted = false;

    for (;;) {
        if (!busy && !exhausted) {
            const unsigned long long k = atomicAdd(queue, 1ull);
            if (k < n) {
                idx = k;
                p = base + offsets[k];
                len = lengths[k];
                nfull = len >> 6;
                j = 0;
                tail_blocks = 0;
                tail_pos = 0;
                sel = be_selector((uint32_t)(reinterpret_cast<uintptr_t>(p) & 3u));
                sha256_init(st);
                if (nfull) load_raw(p, raw);
                busy = true;
            } else {
                exhausted = true;
            }
        }
        if (!__any_sync(0xffffffffu, busy)) break;

        bool finishing = false;
        if (busy) {
            if (j < nfull) {
#pragma unroll
                for (int i = 0; i < 16; ++i) w[i] = __byte_perm(raw[i], raw[i + 1], sel);
                if (j + 1 < nfull) load_raw(p + 64 * (j + 1), raw);
                ++j;
            } else {
                if (tail_blocks == 0)
                    tail_blocks = sha256_build_tail(p + 64 * nfull, (uint32_t)(len & 63u), len, tw);
#pragma unroll
                for (int i = 0; i < 16; ++i) w[i] = tw[16 * tail_pos + i];
                ++tail_pos;
                finishing = (tail_pos == tail_blocks);
            }
            sha256_compress(st, w);
            if (finishing) {
                store_digest(digests + 32 * idx, st);
                busy = false;
            }
        }
    }
}

// order[r] = index of the tensor with the r-th largest length (ties by index): a rank sort, one
// thread per tensor counting the tensors that come before it.  Long messages then start first and
// the 32 lanes of a warp carry messages of similar length.
__global__ void rank_by_length_kernel(const uint64_t *__restrict__ lengths, uint32_t n, uint32_t *__restrict__ order) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint64_t mine = lengths[i];
    uint32_t rank = 0;
    for (uint32_t j = 0; j < n; ++j) {
        const uint64_t other = __ldg(lengths + j);
        rank += (other > mine || (other == mine && j < i)) ? 1u : 0u;
    }
    order[rank] = i;
}

}  // namespace

cudaError_t launch_hash_ragged(const uint8_t *d_base, const uint64_t *d_offsets,
                               const uint64_t *d_lengths, uint64_t n, uint8_t *d_digests,
                               unsigned long long *d_queue, uint32_t *d_order, uint32_t *d_status,
                               const uint32_t *d_one, int sm_count, cudaStream_t stream, uint64_t *launches,
                               const char **kernel_used) {
    const char *unused = nullptr;
    if (!kernel_used) kernel_used = &unused;
    if (n == 0) return cudaSuccess;
    if (n <= kRaggedSortMax && d_order) {
        rank_by_length_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(d_lengths, (uint32_t)n, d_order);
        cudaError_t e0 = cudaGetLastError();
        if (e0 != cudaSuccess) return e0;
        if (launches) *launches += 2;
        *kernel_used = "hash_chunks_split_kernel (tensors)";
        return launch_hash_ragged_split(d_base, d_offsets, d_lengths, d_order, n, d_digests, d_status, d_one, nullptr, 1,
                                        stream);
    }
    cudaError_t e = cudaMemsetAsync(d_queue, 0, sizeof(unsigned long long), stream);
    if (e != cudaSuccess) return e;
    // Few messages: one warp per CTA spreads the chains over all SM schedulers.
    const uint64_t lanes_1w = 32ull * 4ull * (uint64_t)sm_count;
    unsigned threads, blocks;
    if (n <= lanes_1w) {
        threads = 32;
        blocks = (unsigned)((n + 31) / 32);
    } else {
        threads = 128;
        const uint64_t want = (n + 127) / 128;
        const uint64_t cap = 2ull * (uint64_t)sm_count;
        blocks = (unsigned)(want < cap ? want : cap);
    }
    *kernel_used = "hash_ragged_kernel";
    hash_ragged_kernel<<<blocks, threads, 0, stream>>>(d_base, d_offsets, d_lengths, n, d_digests, d_queue);
    if (launches) ++*launches;
    return cudaGetLastError();
}

}  // namespace ivk
