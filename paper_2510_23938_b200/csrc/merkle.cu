// Merkle reduction of leaf digests to a root, and the comparison of computed
// digests and root with the manifest (Algorithm 1: "Construct Merkle tree from
// leaf_hashes using GPU", "Compare root hash with expected value").
//
// Tree rule: parent = SHA-256(left || right) over exactly 64 bytes, an unpaired
// last node moves up unchanged.  Because pairing is index-aligned, any aligned
// run of 2^k leaves reduces to one node of the global tree on its own, so each
// CTA reduces a run of 512 leaves through nine levels in shared memory, and the
// CTA that finishes last (a ticket, no spinning) reduces the run roots.
#include "iv_internal.h"
#include "sha256_dev.cuh"

namespace ivk {

namespace {

constexpr int kThreads = 256;

// Parent of two nodes held as eight native words each: the first block is the
// 64 message bytes, the second block is the constant padding of a 64-byte message.
__device__ __forceinline__ void merkle_parent(const uint32_t *left_right /* 16 words */, uint32_t *out /* 8 words */) {
    uint32_t st[8], w[16];
    sha256_init(st);
    const uint4 *s = reinterpret_cast<const uint4 *>(left_right);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 q = s[i];
        w[4 * i + 0] = q.x; w[4 * i + 1] = q.y; w[4 * i + 2] = q.z; w[4 * i + 3] = q.w;
    }
    sha256_compress(st, w);
    sha256_pad_only_block(w, 64);
    sha256_compress(st, w);
    uint4 *d = reinterpret_cast<uint4 *>(out);
    d[0] = make_uint4(st[0], st[1], st[2], st[3]);
    d[1] = make_uint4(st[4], st[5], st[6], st[7]);
}

// Level-by-level reduction of `count` nodes (8 words each) that sit in buffer a;
// b is the other half of the ping-pong.  Returns the buffer holding the single root.
__device__ uint32_t *reduce_in_shared(uint32_t *a, uint32_t *b, uint32_t count) {
    while (count > 1) {
        const uint32_t parents = count >> 1;
        for (uint32_t j = threadIdx.x; j < parents; j += blockDim.x) merkle_parent(a + 16 * j, b + 8 * j);
        if ((count & 1u) && threadIdx.x < 8) b[8 * parents + threadIdx.x] = a[8 * (count - 1) + threadIdx.x];
        __syncthreads();
        uint32_t *t = a; a = b; b = t;
        count = parents + (count & 1u);
    }
    return a;
}

// Copies `count` digests (byte records, big-endian words) from global memory
// into shared memory as native words.  `coherent` = the records were written
// by other CTAs of this launch, so the loads must bypass L1.
__device__ void load_nodes(const uint8_t *src, uint32_t count, uint32_t *dst, bool coherent) {
    if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
        const uint4 *s = reinterpret_cast<const uint4 *>(src);
        for (uint32_t q = threadIdx.x; q < 2 * count; q += blockDim.x) {
            const uint4 v = coherent ? __ldcg(s + q) : __ldg(s + q);
            reinterpret_cast<uint4 *>(dst)[q] = make_uint4(bswap32(v.x), bswap32(v.y), bswap32(v.z), bswap32(v.w));
        }
    } else {
        for (uint32_t q = threadIdx.x; q < 8 * count; q += blockDim.x) {
            const uint8_t *p = src + 4 * (uint64_t)q;
            dst[q] = ((uint32_t)p[0] << 24) | ((uint32_t)p[1] << 16) | ((uint32_t)p[2] << 8) | (uint32_t)p[3];
        }
    }
    __syncthreads();
}

__device__ void store_node(uint8_t *dst, const uint32_t *node) {
    if (threadIdx.x == 0) {
        uint32_t st[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) st[i] = node[i];
        store_digest(dst, st);
    }
}

// One pass: nodes_in[n] -> nodes_out[ceil(n/512)].  When fuse_top is set (at most
// 512 run roots) the CTA that takes the last ticket reduces them to d_root too.
// blockIdx.y selects one of several independent trees of the same size (batch verification): tree y
// reads nodes_in + y * in_stride, writes nodes_out + y * out_stride, d_root + 32 y and uses ticket[y].
__global__ void __launch_bounds__(kThreads)
merkle_pass_kernel(const uint8_t *__restrict__ nodes_in, uint64_t n, uint8_t *__restrict__ nodes_out,
                   uint8_t *__restrict__ d_root, uint32_t *ticket, int fuse_top, uint64_t in_stride = 0,
                   uint64_t out_stride = 0) {
    __shared__ __align__(16) uint32_t buf_a[kMerkleRun * 8];
    __shared__ __align__(16) uint32_t buf_b[kMerkleRun * 4];
    __shared__ uint32_t s_last;
    nodes_in += blockIdx.y * in_stride;
    nodes_out += blockIdx.y * out_stride;
    d_root += 32 * blockIdx.y;
    ticket += blockIdx.y;

    const uint64_t runs = (n + kMerkleRun - 1) / kMerkleRun;
    for (uint64_t r = blockIdx.x; r < runs; r += gridDim.x) {
        const uint64_t first = r * kMerkleRun;
        const uint32_t count = (uint32_t)((n - first < kMerkleRun) ? (n - first) : kMerkleRun);
        load_nodes(nodes_in + 32 * first, count, buf_a, false);
        const uint32_t *root = reduce_in_shared(buf_a, buf_b, count);
        // a lone run with fuse_top is already the root of the whole tree
        store_node((runs == 1 && fuse_top) ? d_root : nodes_out + 32 * r, root);
        __syncthreads();
    }
    if (!fuse_top || runs == 1) return;

    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1) ? 1u : 0u;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    load_nodes(nodes_out, (uint32_t)runs, buf_a, true);
    const uint32_t *root = reduce_in_shared(buf_a, buf_b, (uint32_t)runs);
    store_node(d_root, root);
    if (threadIdx.x == 0) *ticket = 0u;   // ready for the next call
}

// `levels` (1..9) levels of the reduction on every aligned block of 512 input nodes:
// nodes_in[n] -> nodes_out[ceil(n / 2^levels)].  Because pairing is index-aligned, the output is
// exactly level `levels` of the tree over nodes_in (promotion can only happen at the very end).
__global__ void __launch_bounds__(kThreads)
merkle_levels_kernel(const uint8_t *__restrict__ nodes_in, uint64_t n, uint32_t levels,
                     uint8_t *__restrict__ nodes_out) {
    __shared__ __align__(16) uint32_t buf_a[kMerkleRun * 8];
    __shared__ __align__(16) uint32_t buf_b[kMerkleRun * 4];
    const uint64_t blocks = (n + kMerkleRun - 1) / kMerkleRun;
    for (uint64_t r = blockIdx.x; r < blocks; r += gridDim.x) {
        const uint64_t first = r * kMerkleRun;
        uint32_t count = (uint32_t)((n - first < kMerkleRun) ? (n - first) : kMerkleRun);
        load_nodes(nodes_in + 32 * first, count, buf_a, false);
        uint32_t *a = buf_a, *b = buf_b;
        for (uint32_t l = 0; l < levels && count > 1; ++l) {
            const uint32_t parents = count >> 1;
            for (uint32_t j = threadIdx.x; j < parents; j += blockDim.x) merkle_parent(a + 16 * j, b + 8 * j);
            if ((count & 1u) && threadIdx.x < 8) b[8 * parents + threadIdx.x] = a[8 * (count - 1) + threadIdx.x];
            __syncthreads();
            uint32_t *t = a; a = b; b = t;
            count = parents + (count & 1u);
        }
        // a block of 512 inputs yields 512 >> levels outputs (fewer for the ragged last block)
        uint8_t *dst = nodes_out + 32 * (first >> levels);
        for (uint32_t j = threadIdx.x; j < count; j += blockDim.x) {
            uint32_t st[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) st[k] = a[8 * j + k];
            store_digest(dst + 32 * (uint64_t)j, st);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------
// Incremental re-verification on a retained tree (all levels kept in one array,
// leaves first).  After some leaves changed, only their ancestors are recomputed:
// one thread per changed leaf walks up one level per step; two changed siblings
// compute the same parent twice and store the same bytes.
// ---------------------------------------------------------------------------

struct TreeShape {
    uint64_t level_off[kTreeMaxLevels + 1];   // first record of each level
    uint64_t level_n[kTreeMaxLevels + 1];     // nodes of each level
    uint32_t levels;                          // number of parent levels (the root is level `levels`)
};

__device__ __forceinline__ void load_digest_words(const uint8_t *p, uint32_t (&w)[8]) {
    const uint4 lo = __ldcg(reinterpret_cast<const uint4 *>(p));
    const uint4 hi = __ldcg(reinterpret_cast<const uint4 *>(p) + 1);
    w[0] = bswap32(lo.x); w[1] = bswap32(lo.y); w[2] = bswap32(lo.z); w[3] = bswap32(lo.w);
    w[4] = bswap32(hi.x); w[5] = bswap32(hi.y); w[6] = bswap32(hi.z); w[7] = bswap32(hi.w);
}

// Recomputes the parent (at level l+1) of node `child` of level l; tree is 16-byte aligned.
__device__ void tree_update_parent(uint8_t *tree, const TreeShape &shape, uint32_t l, uint64_t child) {
    const uint64_t parent = child >> 1, left = parent << 1, right = left + 1;
    const uint8_t *lp = tree + 32 * (shape.level_off[l] + left);
    uint8_t *dst = tree + 32 * (shape.level_off[l + 1] + parent);
    uint32_t st[8], w[16];
    if (right < shape.level_n[l]) {
        uint32_t a[8], b[8];
        load_digest_words(lp, a);
        load_digest_words(lp + 32, b);
#pragma unroll
        for (int k = 0; k < 8; ++k) { w[k] = a[k]; w[8 + k] = b[k]; }
        sha256_init(st);
        sha256_compress(st, w);
        sha256_pad_only_block(w, 64);
        sha256_compress(st, w);
    } else {
        load_digest_words(lp, st);               // unpaired last node moves up unchanged
    }
    store_digest_aligned(dst, st);
}

// All levels in one CTA (n_dirty <= blockDim.x): a block barrier separates the levels.
__global__ void __launch_bounds__(1024)
tree_update_small_kernel(uint8_t *__restrict__ tree, TreeShape shape, const uint64_t *__restrict__ dirty,
                         uint32_t n_dirty) {
    bool active = threadIdx.x < n_dirty;
    uint64_t node = active ? dirty[threadIdx.x] : 0;
    if (node >= shape.level_n[0]) active = false;      // an index outside the tree is skipped (status set earlier)
    for (uint32_t l = 0; l < shape.levels; ++l) {
        if (active) tree_update_parent(tree, shape, l, node);
        node >>= 1;
        __threadfence_block();
        __syncthreads();
    }
}

// One level per launch for long dirty lists.
__global__ void __launch_bounds__(256)
tree_update_level_kernel(uint8_t *__restrict__ tree, TreeShape shape, uint32_t l, const uint64_t *__restrict__ dirty,
                         uint64_t n_dirty) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < n_dirty && dirty[t] < shape.level_n[0]) tree_update_parent(tree, shape, l, dirty[t] >> l);
}

// offsets / lengths of the dirty chunks for the per-tensor hashing kernels
__global__ void dirty_ranges_kernel(const uint64_t *__restrict__ dirty, uint64_t n_dirty, uint64_t nbytes,
                                    uint64_t chunk_bytes, uint64_t n_leaves, uint64_t *__restrict__ offsets,
                                    uint64_t *__restrict__ lengths, uint32_t *__restrict__ status) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_dirty) return;
    const uint64_t idx = dirty[t];
    if (idx >= n_leaves) {                      // not a chunk of this blob: hash nothing, record the fault
        offsets[t] = 0;
        lengths[t] = 0;
        atomicExch(status, (uint32_t)IVK_DEV_BOUNDS);
        return;
    }
    const uint64_t begin = idx * chunk_bytes;
    offsets[t] = begin;
    lengths[t] = (nbytes - begin < chunk_bytes) ? (nbytes - begin) : chunk_bytes;
}

// chunk ranges of several blobs of equal size as one tensor list: offsets are relative to blob 0
// (unsigned wrap-around makes blobs below blob 0 work too)
__global__ void batch_ranges_kernel(BlobList blobs, uint64_t n_chunks, uint64_t nbytes, uint64_t chunk_bytes,
                                    uint64_t *__restrict__ offsets, uint64_t *__restrict__ lengths) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_chunks * blobs.count) return;
    const uint64_t b = t / n_chunks, i = t - b * n_chunks;
    const uint64_t begin = i * chunk_bytes;
    offsets[t] = (uint64_t)(blobs.ptr[b] - blobs.ptr[0]) + begin;
    lengths[t] = (nbytes - begin < chunk_bytes) ? (nbytes - begin) : chunk_bytes;
}

// Column parts of the chunks of one window: part s of chunk i covers bytes [s * part, (s + 1) * part) of the
// chunk's whole 64-byte blocks, the last part everything that is left (tail and padding included).
// Entry s * m + i; a part that finishes no chunk is a whole number of blocks.
__global__ void column_ranges_kernel(uint64_t m, uint64_t bytes, uint64_t chunk_bytes, uint64_t part_bytes, uint32_t parts,
                                     uint64_t *__restrict__ offsets, uint64_t *__restrict__ lengths) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= m * parts) return;
    const uint64_t s = t / m, i = t - s * m;
    const uint64_t begin = i * chunk_bytes;
    const uint64_t len = (bytes - begin < chunk_bytes) ? (bytes - begin) : chunk_bytes;
    const uint64_t full = len & ~63ull;
    const uint64_t lo = s * part_bytes < full ? s * part_bytes : full;
    const uint64_t hi = (s + 1 == parts) ? len : ((s + 1) * part_bytes < full ? (s + 1) * part_bytes : full);
    offsets[t] = begin + lo;
    lengths[t] = hi - lo;
}

// new leaf digests (in dirty-list order) into the leaf level of the tree
__global__ void scatter_leaves_kernel(const uint8_t *__restrict__ fresh, const uint64_t *__restrict__ dirty,
                                      uint64_t n_dirty, uint64_t n_leaves, uint8_t *__restrict__ tree) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;   // one thread per 16 bytes
    if (t >= 2 * n_dirty || dirty[t >> 1] >= n_leaves) return;
    const uint4 v = reinterpret_cast<const uint4 *>(fresh)[t];
    reinterpret_cast<uint4 *>(tree + 32 * dirty[t >> 1])[t & 1] = v;
}

// Root of zero leaves: SHA-256 of the empty string, computed here rather than typed in.
__global__ void empty_root_kernel(uint8_t *d_root) {
    uint32_t st[8], w[16];
    sha256_init(st);
    sha256_pad_only_block(w, 0);
    sha256_compress(st, w);
    store_digest(d_root, st);
}

// ---------------------------------------------------------------------------
// Compare + ordered compaction.
// Each warp compares 32 chunk digests with the manifest and publishes the
// ballot as one mask word; the CTA that takes the last ticket turns the mask
// words into the ascending index list with a block-wide exclusive scan.
// ---------------------------------------------------------------------------

// REC: bytes per digest record (32 for SHA-256, 48 for SHA-384, 64 for SHA-512).
template <int REC>
__device__ __forceinline__ bool digest_differs(const uint8_t *a, const uint8_t *b, bool aligned) {
    uint32_t diff = 0;
    if (aligned) {
#pragma unroll
        for (int q = 0; q < REC / 16; ++q) {
            const uint4 x = __ldg(reinterpret_cast<const uint4 *>(a) + q), y = __ldg(reinterpret_cast<const uint4 *>(b) + q);
            diff |= (x.x ^ y.x) | (x.y ^ y.y) | (x.z ^ y.z) | (x.w ^ y.w);
        }
        return diff != 0u;
    }
    for (int i = 0; i < REC; ++i) diff |= (uint32_t)(a[i] ^ b[i]);
    return diff != 0u;
}

template <int REC, class Result, class Root>
__global__ void __launch_bounds__(kThreads)
verify_compare_kernel(const uint8_t *__restrict__ digests, const uint8_t *__restrict__ manifest, uint64_t n,
                      const uint8_t *__restrict__ d_root, Root manifest_root,
                      Result *__restrict__ result, uint64_t *__restrict__ idx_out, uint64_t idx_cap,
                      uint32_t *__restrict__ words, uint32_t *ticket, const uint32_t *__restrict__ dev_status) {
    __shared__ uint32_t s_last;
    __shared__ uint32_t s_warp_sum[kThreads / 32];
    __shared__ unsigned long long s_base;

    const bool aligned = (((reinterpret_cast<uintptr_t>(digests) | reinterpret_cast<uintptr_t>(manifest)) & 15u) == 0);
    const uint64_t n_words = (n + 31) / 32;
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warps_total = (uint64_t)gridDim.x * (kThreads / 32);
    for (uint64_t wi = (uint64_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5); wi < n_words; wi += warps_total) {
        const uint64_t i = wi * 32 + lane;
        const bool bad = (i < n) && digest_differs<REC>(digests + (uint64_t)REC * i, manifest + (uint64_t)REC * i, aligned);
        const uint32_t mask = __ballot_sync(0xffffffffu, bad);
        if (lane == 0) words[wi] = mask;
    }

    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1) ? 1u : 0u;
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    if (threadIdx.x == 0) s_base = 0ull;
    __syncthreads();
    for (uint64_t tile = 0; tile < n_words; tile += kThreads) {
        const uint64_t wi = tile + threadIdx.x;
        const uint32_t mask = (wi < n_words) ? __ldcg(words + wi) : 0u;
        const uint32_t cnt = __popc(mask);
        // exclusive scan of cnt across the CTA
        uint32_t incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= (uint32_t)d) incl += up;
        }
        if (lane == 31) s_warp_sum[threadIdx.x >> 5] = incl;
        __syncthreads();
        uint32_t warp_off = 0, tile_total = 0;
#pragma unroll
        for (int k = 0; k < kThreads / 32; ++k) {
            const uint32_t s = s_warp_sum[k];
            if (k < (int)(threadIdx.x >> 5)) warp_off += s;
            tile_total += s;
        }
        unsigned long long pos = s_base + warp_off + (incl - cnt);
        uint32_t m = mask;
        while (m) {
            const uint32_t b = __ffs(m) - 1;
            m &= m - 1;
            if (pos < idx_cap) idx_out[pos] = wi * 32 + b;
            ++pos;
        }
        __syncthreads();
        if (threadIdx.x == 0) s_base += tile_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        uint32_t diff = 0;
        for (int i = 0; i < REC; ++i) {
            const uint8_t r = d_root[i];
            result->root[i] = r;
            diff |= (uint32_t)(r ^ manifest_root.b[i]);
        }
        result->status = __ldcg(dev_status);   // nonzero if a kernel of this context gave up on a wait
        result->root_ok = diff == 0u ? 1u : 0u;
        result->n_mismatch = s_base;
        *ticket = 0u;
    }
}

}  // namespace

cudaError_t launch_merkle_root(const uint8_t *d_leaves, uint64_t n, uint8_t *d_root,
                               uint8_t *d_scratch_a, uint8_t *d_scratch_b, uint32_t *d_tickets,
                               cudaStream_t stream, uint64_t *launches) {
    if (n == 0) {
        empty_root_kernel<<<1, 1, 0, stream>>>(d_root);
        if (launches) ++*launches;
        return cudaGetLastError();
    }
    const uint8_t *in = d_leaves;
    uint8_t *out = d_scratch_a, *other = d_scratch_b;
    for (int pass = 0; pass < kMerkleMaxPasses; ++pass) {
        const uint64_t runs = (n + kMerkleRun - 1) / kMerkleRun;
        const int fuse_top = runs <= kMerkleRun ? 1 : 0;
        const unsigned grid = (unsigned)(runs < 4096 ? runs : 4096);
        merkle_pass_kernel<<<grid, kThreads, 0, stream>>>(in, n, out, d_root, d_tickets + pass, fuse_top);
        if (launches) ++*launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess || fuse_top) return e;
        in = out;
        uint8_t *t = out; out = other; other = t;
        n = runs;
    }
    return cudaErrorInvalidValue;   // more than 512^8 leaves cannot be addressed
}

// The roots of `trees` trees of n leaves each (n <= 512 * 512: one fused pass), leaves of tree y at
// d_leaves + y * 32 n, root y at d_roots + 32 y; d_scratch holds trees * 512 records, d_tickets `trees` zeroed words.
cudaError_t launch_merkle_roots_batch(const uint8_t *d_leaves, uint64_t n, uint32_t trees, uint8_t *d_roots,
                                      uint8_t *d_scratch, uint32_t *d_tickets, cudaStream_t stream, uint64_t *launches) {
    if (n == 0 || trees == 0 || n > (uint64_t)kMerkleRun * kMerkleRun) return cudaErrorInvalidValue;
    const uint64_t runs = (n + kMerkleRun - 1) / kMerkleRun;
    const dim3 grid((unsigned)runs, trees);
    merkle_pass_kernel<<<grid, kThreads, 0, stream>>>(d_leaves, n, d_scratch, d_roots, d_tickets, 1, 32 * n,
                                                      32ull * kMerkleRun);
    if (launches) ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_merkle_levels(const uint8_t *d_in, uint64_t n, uint32_t levels, uint8_t *d_out,
                                 cudaStream_t stream, uint64_t *launches) {
    if (n == 0 || levels == 0 || levels > 9) return cudaErrorInvalidValue;
    const uint64_t blocks = (n + kMerkleRun - 1) / kMerkleRun;
    merkle_levels_kernel<<<(unsigned)(blocks < 4096 ? blocks : 4096), kThreads, 0, stream>>>(d_in, n, levels, d_out);
    if (launches) ++*launches;
    return cudaGetLastError();
}

namespace {
TreeShape make_shape(uint64_t n_leaves) {
    TreeShape sh{};
    uint64_t n = n_leaves, off = 0;
    uint32_t l = 0;
    sh.level_off[0] = 0;
    sh.level_n[0] = n;
    while (n > 1 && l < (uint32_t)kTreeMaxLevels) {
        off += n;
        n = (n + 1) / 2;
        ++l;
        sh.level_off[l] = off;
        sh.level_n[l] = n;
    }
    sh.levels = l;
    return sh;
}
}  // namespace

uint64_t tree_records(uint64_t n_leaves) {
    if (n_leaves == 0) return 1;
    const TreeShape sh = make_shape(n_leaves);
    return sh.level_off[sh.levels] + 1;
}

cudaError_t launch_tree_build(const uint8_t *d_leaves, uint64_t n, uint8_t *d_tree, cudaStream_t stream,
                              uint64_t *launches) {
    if (n == 0) {
        empty_root_kernel<<<1, 1, 0, stream>>>(d_tree);
        if (launches) ++*launches;
        return cudaGetLastError();
    }
    cudaError_t e = cudaMemcpyAsync(d_tree, d_leaves, 32 * n, cudaMemcpyDeviceToDevice, stream);
    if (e != cudaSuccess) return e;
    const TreeShape sh = make_shape(n);
    for (uint32_t l = 0; l < sh.levels; ++l) {
        e = launch_merkle_levels(d_tree + 32 * sh.level_off[l], sh.level_n[l], 1, d_tree + 32 * sh.level_off[l + 1],
                                 stream, launches);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_batch_ranges(const BlobList &blobs, uint64_t n_chunks, uint64_t nbytes, uint64_t chunk_bytes,
                                uint64_t *d_offsets, uint64_t *d_lengths, cudaStream_t stream, uint64_t *launches) {
    const uint64_t total = n_chunks * blobs.count;
    batch_ranges_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(blobs, n_chunks, nbytes, chunk_bytes,
                                                                            d_offsets, d_lengths);
    if (launches) ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_column_ranges(uint64_t m, uint64_t bytes, uint64_t chunk_bytes, uint64_t part_bytes, uint32_t parts,
                                 uint64_t *d_offsets, uint64_t *d_lengths, cudaStream_t stream, uint64_t *launches) {
    const uint64_t total = m * parts;
    if (total == 0) return cudaSuccess;
    column_ranges_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(m, bytes, chunk_bytes, part_bytes, parts,
                                                                             d_offsets, d_lengths);
    if (launches) ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_dirty_ranges(const uint64_t *d_dirty, uint64_t n_dirty, uint64_t nbytes, uint64_t chunk_bytes,
                                uint64_t n_leaves, uint64_t *d_offsets, uint64_t *d_lengths, uint32_t *d_status,
                                cudaStream_t stream, uint64_t *launches) {
    dirty_ranges_kernel<<<(unsigned)((n_dirty + 255) / 256), 256, 0, stream>>>(d_dirty, n_dirty, nbytes, chunk_bytes,
                                                                              n_leaves, d_offsets, d_lengths, d_status);
    if (launches) ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_tree_update(uint8_t *d_tree, uint64_t n_leaves, const uint8_t *d_fresh, const uint64_t *d_dirty,
                               uint64_t n_dirty, cudaStream_t stream, uint64_t *launches) {
    if (n_dirty == 0 || n_leaves == 0) return cudaSuccess;
    scatter_leaves_kernel<<<(unsigned)((2 * n_dirty + 255) / 256), 256, 0, stream>>>(d_fresh, d_dirty, n_dirty, n_leaves,
                                                                                     d_tree);
    if (launches) ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const TreeShape sh = make_shape(n_leaves);
    if (sh.levels == 0) return cudaSuccess;
    if (n_dirty <= 1024) {
        tree_update_small_kernel<<<1, 1024, 0, stream>>>(d_tree, sh, d_dirty, (uint32_t)n_dirty);
        if (launches) ++*launches;
        return cudaGetLastError();
    }
    for (uint32_t l = 0; l < sh.levels; ++l) {
        tree_update_level_kernel<<<(unsigned)((n_dirty + 255) / 256), 256, 0, stream>>>(d_tree, sh, l, d_dirty, n_dirty);
        if (launches) ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_verify_compare(const uint8_t *d_digests, const uint8_t *d_manifest_digests,
                                  uint64_t n, const uint8_t *d_root, RootBytes manifest_root,
                                  iv_verify_result *d_result, uint64_t *d_mismatch_idx,
                                  uint64_t idx_cap, uint32_t *d_words, uint32_t *d_ticket,
                                  const uint32_t *d_status, cudaStream_t stream, uint64_t *launches) {
    const uint64_t n_words = (n + 31) / 32;
    uint64_t blocks = (n_words + (kThreads / 32) - 1) / (kThreads / 32);
    if (blocks == 0) blocks = 1;
    if (blocks > 1184) blocks = 1184;
    verify_compare_kernel<32, iv_verify_result, RootBytes><<<(unsigned)blocks, kThreads, 0, stream>>>(
        d_digests, d_manifest_digests, n, d_root, manifest_root, d_result, d_mismatch_idx, idx_cap,
        d_words, d_ticket, d_status);
    if (launches) ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_verify_compare_sha384(const uint8_t *d_digests, const uint8_t *d_manifest_digests,
                                         uint64_t n, const uint8_t *d_root, RootBytes384 manifest_root,
                                         iv_verify_result_sha384 *d_result, uint64_t *d_mismatch_idx,
                                         uint64_t idx_cap, uint32_t *d_words, uint32_t *d_ticket,
                                         const uint32_t *d_status, cudaStream_t stream, uint64_t *launches) {
    const uint64_t n_words = (n + 31) / 32;
    uint64_t blocks = (n_words + (kThreads / 32) - 1) / (kThreads / 32);
    if (blocks == 0) blocks = 1;
    if (blocks > 1184) blocks = 1184;
    verify_compare_kernel<48, iv_verify_result_sha384, RootBytes384><<<(unsigned)blocks, kThreads, 0, stream>>>(
        d_digests, d_manifest_digests, n, d_root, manifest_root, d_result, d_mismatch_idx, idx_cap,
        d_words, d_ticket, d_status);
    if (launches) ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_verify_compare_sha512(const uint8_t *d_digests, const uint8_t *d_manifest_digests,
                                         uint64_t n, const uint8_t *d_root, RootBytes512 manifest_root,
                                         iv_verify_result_sha512 *d_result, uint64_t *d_mismatch_idx,
                                         uint64_t idx_cap, uint32_t *d_words, uint32_t *d_ticket,
                                         const uint32_t *d_status, cudaStream_t stream, uint64_t *launches) {
    const uint64_t n_words = (n + 31) / 32;
    uint64_t blocks = (n_words + (kThreads / 32) - 1) / (kThreads / 32);
    if (blocks == 0) blocks = 1;
    if (blocks > 1184) blocks = 1184;
    verify_compare_kernel<64, iv_verify_result_sha512, RootBytes512><<<(unsigned)blocks, kThreads, 0, stream>>>(
        d_digests, d_manifest_digests, n, d_root, manifest_root, d_result, d_mismatch_idx, idx_cap,
        d_words, d_ticket, d_status);
    if (launches) ++*launches;
    return cudaGetLastError();
}

}  // namespace ivk

// ---------------------------------------------------------------------------
// Merkle root for callers that must not allocate.
//
// iv_merkle_root keeps the run roots and the ticket in memory that iv_create
// and the first large call obtain with cudaMalloc.  Code that runs where device
// allocation is forbidden or impossible -- inside a memory pool that already
// owns the whole device, in a latency-critical serving loop that may not touch
// the allocator's lock, after a fork where only pre-made buffers may be used --
// cannot call it.  This variant keeps the same scratch in a fixed array that is
// part of the library image, so every GPU that loads the library carries these
// 16.25 KiB until the process exits, and the number of leaves is capped.
// ---------------------------------------------------------------------------

// 512 run roots of 32 bytes, then the ticket word (offset 16384).
static __device__ __align__(256) unsigned char iv_noalloc_scratch[ivk::kMerkleRun * 32 + 256];

namespace {

constexpr int kNoAllocMaxDevices = 64;
// Device addresses of iv_noalloc_scratch, one per device, filled on first use.  The array's
// name is only a host-side handle: the address a kernel can use comes from cudaGetSymbolAddress.
unsigned char *g_noalloc_ptr[kNoAllocMaxDevices] = {};

}  // namespace

extern "C" int iv_merkle_root_noalloc(const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root,
                                      void *cuda_stream) {
    if (!d_root || (n_leaves && !d_leaves)) return IV_ERR_INVALID_ARG;
    if (n_leaves > IV_NOALLOC_MAX_LEAVES) return IV_ERR_TOO_LARGE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices) {
        (void)cudaGetLastError();
        return IV_ERR_NO_DEVICE;
    }
    unsigned char *scratch = __atomic_load_n(&g_noalloc_ptr[dev], __ATOMIC_ACQUIRE);
    if (!scratch) {
        // set-up, once per device, with that device current
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&scratch), iv_noalloc_scratch) != cudaSuccess || !scratch) {
            (void)cudaGetLastError();
            return IV_ERR_CUDA;
        }
        __atomic_store_n(&g_noalloc_ptr[dev], scratch, __ATOMIC_RELEASE);
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (n_leaves == 0) {
        ivk::empty_root_kernel<<<1, 1, 0, stream>>>(d_root);
        return cudaGetLastError() == cudaSuccess ? IV_OK : IV_ERR_CUDA;
    }
    uint32_t *ticket = reinterpret_cast<uint32_t *>(scratch + ivk::kMerkleRun * 32);
    // The array keeps whatever the previous call left; only the ticket has to start at zero.
    if (cudaMemsetAsync(ticket, 0, sizeof(uint32_t), stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return IV_ERR_CUDA;
    }
    const uint64_t runs = (n_leaves + ivk::kMerkleRun - 1) / ivk::kMerkleRun;   // <= 512: one fused pass
    ivk::merkle_pass_kernel<<<(unsigned)runs, ivk::kThreads, 0, stream>>>(d_leaves, n_leaves, scratch, d_root,
                                                                           ticket, 1);
    return cudaGetLastError() == cudaSuccess ? IV_OK : IV_ERR_CUDA;
}
