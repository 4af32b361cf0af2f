// C ABI of libiv (see include/iv.h): argument checks, scratch management,
// stream plumbing.  All arithmetic of the path runs in the kernels.
#include <cstdlib>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "iv_internal.h"

struct iv_ctx {
    int device = 0;
    int sm_count = 0;
    int last_cuda_error = 0;
    uint64_t launches = 0;
    const char *leaf_kernel = "";             // name of the leaf-hashing kernel the last call launched
    const char *leaf_instance = "";           // and, where that kernel has several launch shapes, which one

    // small fixed block: tickets, work-queue counter, root
    uint32_t *d_tickets = nullptr;            // kMerkleMaxPasses + 1 words
    unsigned long long *d_queue = nullptr;
    uint8_t *d_root = nullptr;                // 32 bytes
    uint32_t *d_status = nullptr;             // device-side status word (0 = ok), sticky until read
    uint32_t *d_one = nullptr;                // a device word holding 1 (multiplier for adds on the FMA pipe)
    void *d_small = nullptr;

    // lazily sized scratch
    uint8_t *d_merkle_a = nullptr, *d_merkle_b = nullptr;
    uint64_t merkle_cap = 0;                  // in digests, each buffer
    uint8_t *d_digests = nullptr;
    uint64_t digests_cap = 0;                 // in digests
    uint64_t digests_valid = 0;
    uint32_t *d_words = nullptr;
    uint64_t words_cap = 0;
    uint8_t *d_tree384[2] = {nullptr, nullptr};   // level ping-pong of the SHA-384 and RFC 6962 trees
    uint64_t tree384_cap = 0;                 // in records of 64 bytes, each buffer
    uint8_t *d_pairs512 = nullptr;            // FIFO, slice counters and parked chaining values of the SHA-384/512 two-warp kernel
    uint64_t pairs512_cap = 0;                // bytes
    uint8_t *d_batch = nullptr;               // offsets, lengths, roots, run roots, tickets of iv_verify_manifest_batch
    uint64_t batch_cap = 0;                   // bytes
    uint64_t batch_blobs = 0, batch_total = 0;   // shape of the last batch (the tickets' position depends on it)
    uint8_t *d_sub = nullptr;                 // sub-leaf digests of the two-level mode
    uint64_t sub_cap = 0;                     // in digests
    uint8_t *d_dirty_scratch = nullptr;       // offsets, lengths and fresh digests of iv_tree_update
    uint64_t dirty_cap = 0;                   // bytes
    uint32_t *d_order = nullptr;              // tensor order (by descending length) of iv_hash_ragged
    uint64_t order_cap = 0;
    uint8_t *d_slices = nullptr;              // FIFO, slice counters and parked chaining values of the sliced leaf kernel
    uint64_t slices_cap = 0;                  // bytes

    // streaming windows
    uint8_t *d_digests384 = nullptr;          // chunk digests of iv_verify_manifest_sha384 / _sha512, then the root
    uint64_t digests384_cap = 0;              // records of 64 bytes
    uint8_t *d_columns = nullptr;             // offsets, lengths and chaining values of a window hashed in column parts
    uint64_t columns_cap = 0;                 // bytes
    uint8_t *d_window[2] = {nullptr, nullptr};
    uint64_t window_cap = 0;
    cudaStream_t copy_stream = nullptr;
    cudaStream_t tail_stream = nullptr;       // a blob's short last chunk is hashed here, beside the main leaf kernel
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaEvent_t ev_entry = nullptr, ev_copied[2] = {nullptr, nullptr}, ev_hashed[2] = {nullptr, nullptr};

    // NVTX range of the phase the current verification call is in (leaf hashing / Merkle reduction / compare)
    nvtxRangeId_t nvtx_id = 0;
    bool nvtx_open = false;

    // phase timing: four events (start, hashed, reduced, compared) per recent call
    bool timing = false;
    uint64_t timed_calls = 0;                          // verification calls made so far
    cudaEvent_t ev_phase[IV_TIMING_RING][4] = {};
    bool slot_timed[IV_TIMING_RING] = {};
};

namespace {

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) cudaSetDevice(dev);
        else prev = -1;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

int fail_cuda(iv_ctx *ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda_error = (int)e;
    (void)cudaGetLastError();   // clear the sticky-free error state
    return e == cudaErrorMemoryAllocation ? IV_ERR_NOMEM : IV_ERR_CUDA;
}

#define IV_TRY(ctx, call)                                   \
    do {                                                    \
        cudaError_t e_ = (call);                            \
        if (e_ != cudaSuccess) return fail_cuda((ctx), e_); \
    } while (0)

uint64_t chunk_count(uint64_t nbytes, uint64_t chunk_bytes) {
    return nbytes == 0 ? 0 : (nbytes - 1) / chunk_bytes + 1;
}

// Grows a device buffer to at least `need` bytes (contents are not preserved).
template <typename T>
int grow(iv_ctx *ctx, T **buf, uint64_t *cap_items, uint64_t need_items, uint64_t item_bytes) {
    if (need_items <= *cap_items) return IV_OK;
    if (*buf) {
        IV_TRY(ctx, cudaDeviceSynchronize());
        IV_TRY(ctx, cudaFree(*buf));
        *buf = nullptr;
        *cap_items = 0;
    }
    uint64_t items = need_items + need_items / 4 + 64;
    void *p = nullptr;
    IV_TRY(ctx, cudaMalloc(&p, items * item_bytes));
    *buf = static_cast<T *>(p);
    *cap_items = items;
    return IV_OK;
}

int ensure_merkle_scratch(iv_ctx *ctx, uint64_t n_leaves) {
    const uint64_t need = (n_leaves + ivk::kMerkleRun - 1) / ivk::kMerkleRun + 1;
    if (need <= ctx->merkle_cap) return IV_OK;
    uint64_t cap_a = ctx->merkle_cap, cap_b = ctx->merkle_cap;
    int rc = grow(ctx, &ctx->d_merkle_a, &cap_a, need, 32);
    if (rc != IV_OK) return rc;
    rc = grow(ctx, &ctx->d_merkle_b, &cap_b, need, 32);
    if (rc != IV_OK) return rc;
    ctx->merkle_cap = cap_a < cap_b ? cap_a : cap_b;
    return IV_OK;
}

// Level buffers of the variant trees: two buffers of at least `records` records of up to 64 bytes.
int ensure_variant_tree_scratch(iv_ctx *ctx, uint64_t records) {
    if (records <= ctx->tree384_cap) return IV_OK;
    uint64_t cap_a = ctx->tree384_cap, cap_b = ctx->tree384_cap;
    int rc = grow(ctx, &ctx->d_tree384[0], &cap_a, records, 64);
    if (rc != IV_OK) return rc;
    rc = grow(ctx, &ctx->d_tree384[1], &cap_b, records, 64);
    if (rc != IV_OK) return rc;
    ctx->tree384_cap = cap_a < cap_b ? cap_a : cap_b;
    return IV_OK;
}

// The kernels with tiled copies hash a blob's whole chunks; a short last chunk is left to a direct kernel as one
// serial chain, which for a large chunk can take as long as the whole main launch.  It therefore runs on the
// context's second stream, forked off the caller's stream before the launches and joined after them.
int fork_tail_stream(iv_ctx *ctx, cudaStream_t stream) {
    IV_TRY(ctx, cudaEventRecord(ctx->ev_fork, stream));
    IV_TRY(ctx, cudaStreamWaitEvent(ctx->tail_stream, ctx->ev_fork, 0));
    return IV_OK;
}
int join_tail_stream(iv_ctx *ctx, cudaStream_t stream) {
    IV_TRY(ctx, cudaEventRecord(ctx->ev_join, ctx->tail_stream));
    IV_TRY(ctx, cudaStreamWaitEvent(stream, ctx->ev_join, 0));
    return IV_OK;
}

// After a leaf-hashing launch: which launch shape the kernel ran in, for the kernels that have several.
void note_leaf_instance(iv_ctx *ctx) {
    ctx->leaf_instance = std::strcmp(ctx->leaf_kernel, "hash_chunks_sliced_kernel") == 0 ? ivk::sliced_instance_name() : "";
}

// Leaf hashing with the scratch the launch shape needs.
int hash_leaves(iv_ctx *ctx, const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n,
                uint8_t *d_digests, cudaStream_t stream) {
    void *scratch = nullptr;
    if (ivk::hash_chunks_wants_slices(d_data, chunk_bytes, n, ctx->sm_count)) {
        const uint64_t need = ivk::sliced_scratch_bytes(n, chunk_bytes, nullptr, nullptr, nbytes);
        int rc = grow(ctx, &ctx->d_slices, &ctx->slices_cap, need, 1);
        if (rc != IV_OK) return rc;
        scratch = ctx->d_slices;
    }
    const bool fork = scratch && nbytes % chunk_bytes != 0;
    int rc = IV_OK;
    if (fork && (rc = fork_tail_stream(ctx, stream)) != IV_OK) return rc;
    IV_TRY(ctx, ivk::launch_hash_chunks(d_data, nbytes, chunk_bytes, n, d_digests, ctx->sm_count, ctx->d_status,
                                        ctx->d_one, scratch, stream, &ctx->launches, &ctx->leaf_kernel,
                                        fork ? ctx->tail_stream : nullptr));
    if (fork && (rc = join_tail_stream(ctx, stream)) != IV_OK) return rc;
    note_leaf_instance(ctx);
    return IV_OK;
}

// The same for the prefixed leaf hashes of the RFC 6962 mode.
int hash_leaves_rfc6962(iv_ctx *ctx, const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n,
                        uint8_t *d_digests, cudaStream_t stream) {
    void *scratch = nullptr;
    if (ivk::hash_chunks_wants_slices(d_data, chunk_bytes, n, ctx->sm_count)) {
        const uint64_t need = ivk::sliced_scratch_bytes(n, chunk_bytes, nullptr, nullptr, nbytes);
        int rc = grow(ctx, &ctx->d_slices, &ctx->slices_cap, need, 1);
        if (rc != IV_OK) return rc;
        scratch = ctx->d_slices;
    }
    const bool fork = scratch && nbytes % chunk_bytes != 0;
    int rc = IV_OK;
    if (fork && (rc = fork_tail_stream(ctx, stream)) != IV_OK) return rc;
    IV_TRY(ctx, ivk::launch_hash_chunks_rfc6962(d_data, nbytes, chunk_bytes, n, d_digests, ctx->sm_count, ctx->d_status,
                                                ctx->d_one, scratch, stream, &ctx->launches, &ctx->leaf_kernel,
                                                fork ? ctx->tail_stream : nullptr));
    if (fork && (rc = join_tail_stream(ctx, stream)) != IV_OK) return rc;
    note_leaf_instance(ctx);
    return IV_OK;
}

// SHA-384 (digest_words 6) or SHA-512 (8) leaf hashing with the scratch the launch shape needs.
int hash_leaves_wide(iv_ctx *ctx, const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n,
                     uint8_t *d_digests, int digest_words, cudaStream_t stream) {
    void *scratch = nullptr;
    if (ivk::sha512_wants_pairs(d_data, nbytes, chunk_bytes, ctx->sm_count)) {
        int rc = grow(ctx, &ctx->d_pairs512, &ctx->pairs512_cap, ivk::sha512_pairs_scratch_bytes(nbytes, chunk_bytes), 1);
        if (rc != IV_OK) return rc;
        scratch = ctx->d_pairs512;
    }
    const bool fork = scratch && nbytes % chunk_bytes != 0;
    int rc = IV_OK;
    if (fork && (rc = fork_tail_stream(ctx, stream)) != IV_OK) return rc;
    IV_TRY(ctx, ivk::launch_hash_chunks_sha384(d_data, nbytes, chunk_bytes, n, d_digests, digest_words, ctx->sm_count,
                                               ctx->d_status, scratch, stream, &ctx->launches, &ctx->leaf_kernel,
                                               fork ? ctx->tail_stream : nullptr));
    if (fork && (rc = join_tail_stream(ctx, stream)) != IV_OK) return rc;
    ctx->leaf_instance = std::strcmp(ctx->leaf_kernel, "hash_sha512_pairs_kernel") == 0 ? ivk::sha512_pairs_instance_name() : "";
    return IV_OK;
}

int check_manifest(const iv_manifest *m, uint64_t nbytes) {
    if (!m || m->chunk_bytes == 0) return IV_ERR_INVALID_ARG;
    if (m->total_bytes != nbytes) return IV_ERR_INVALID_ARG;
    if (m->n_chunks != chunk_count(nbytes, m->chunk_bytes)) return IV_ERR_INVALID_ARG;
    if (m->n_chunks && !m->d_digests) return IV_ERR_INVALID_ARG;
    return IV_OK;
}

// One window of a streamed blob, copied and hashed in column parts (see iv_verify_streamed).  The window has m
// chunks of which the last may be short; it lands in ctx->d_window[b], its digests at d_digests.
int hash_window_in_columns(iv_ctx *ctx, const void *h_window, uint64_t bytes, uint64_t chunk, uint64_t m, uint32_t parts,
                           int b, uint8_t *d_digests, cudaStream_t stream) {
    const uint64_t part = (chunk / parts) & ~4095ull;              // a whole number of blocks, at least 16 KiB
    const uint64_t whole = bytes / chunk;                          // m or m - 1
    const uint64_t need = 2 * 8 * m * parts + sizeof(iv_sha_state) * m + 64;
    int rc = grow(ctx, &ctx->d_columns, &ctx->columns_cap, need, 1);
    if (rc != IV_OK) return rc;
    uint64_t *d_off = reinterpret_cast<uint64_t *>(ctx->d_columns);
    uint64_t *d_len = d_off + m * parts;
    iv_sha_state *d_states = reinterpret_cast<iv_sha_state *>(d_len + m * parts);
    IV_TRY(ctx, ivk::launch_column_ranges(m, bytes, chunk, part, parts, d_off, d_len, stream, &ctx->launches));
    IV_TRY(ctx, cudaMemsetAsync(d_states, 0, sizeof(iv_sha_state) * m, stream));
    uint8_t *dst = ctx->d_window[b];
    const uint8_t *src = static_cast<const uint8_t *>(h_window);
    for (uint32_t s = 0; s < parts; ++s) {
        const uint64_t lo = (uint64_t)s * part;
        const uint64_t width = (s + 1 == parts) ? chunk - lo : part;
        if (whole)
            IV_TRY(ctx, cudaMemcpy2DAsync(dst + lo, chunk, src + lo, chunk, width, whole, cudaMemcpyHostToDevice,
                                          ctx->copy_stream));
        if (s == 0 && whole < m)                                   // the blob's short last chunk comes with the first part
            IV_TRY(ctx, cudaMemcpyAsync(dst + whole * chunk, src + whole * chunk, bytes - whole * chunk,
                                        cudaMemcpyHostToDevice, ctx->copy_stream));
        IV_TRY(ctx, cudaEventRecord(ctx->ev_copied[b], ctx->copy_stream));
        IV_TRY(ctx, cudaStreamWaitEvent(stream, ctx->ev_copied[b], 0));
        IV_TRY(ctx, ivk::launch_hash_ragged_split(dst, d_off + (uint64_t)s * m, d_len + (uint64_t)s * m, nullptr, m, d_digests,
                                                  ctx->d_status, ctx->d_one, d_states, s + 1 == parts ? 1 : 0, stream));
        ++ctx->launches;
    }
    ctx->leaf_kernel = "hash_chunks_split_kernel (tensors)";
    return IV_OK;
}

// Phase boundary `which` (0 = leaf hashing begins, 1 = tree reduction begins, 2 = comparison begins, 3 = done) of
// the current verification call: closes and opens the NVTX range of the phase (profilers show the launches of a
// phase under its name; without a tool attached the calls do nothing) and, when timing is on, records the event.
int mark_phase(iv_ctx *ctx, int which, cudaStream_t stream) {
    static const char *const names[3] = {"iv: leaf hashing", "iv: Merkle reduction", "iv: manifest compare"};
    if (ctx->nvtx_open) {
        nvtxRangeEnd(ctx->nvtx_id);
        ctx->nvtx_open = false;
    }
    if (which < 3) {
        ctx->nvtx_id = nvtxRangeStartA(names[which]);
        ctx->nvtx_open = true;
    }
    if (!ctx->timing) return IV_OK;
    const uint32_t slot = (uint32_t)(ctx->timed_calls % IV_TIMING_RING);
    for (int k = 0; k < 4; ++k)
        if (!ctx->ev_phase[slot][k]) IV_TRY(ctx, cudaEventCreate(&ctx->ev_phase[slot][k]));
    IV_TRY(ctx, cudaEventRecord(ctx->ev_phase[slot][which], stream));
    return IV_OK;
}

// Root + compare, shared by the resident and the streamed verification.
int finish_verification(iv_ctx *ctx, const iv_manifest *m, iv_verify_result *d_result,
                        uint64_t *d_mismatch_idx, uint64_t idx_cap, cudaStream_t stream, bool rfc6962 = false) {
    const uint64_t n = m->n_chunks;
    int rc = ensure_merkle_scratch(ctx, n);
    if (rc != IV_OK) return rc;
    rc = grow(ctx, &ctx->d_words, &ctx->words_cap, (n + 31) / 32 + 1, sizeof(uint32_t));
    if (rc != IV_OK) return rc;
    if (rfc6962 && (rc = ensure_variant_tree_scratch(ctx, (n + 1) / 2 + 1)) != IV_OK) return rc;
    if ((rc = mark_phase(ctx, 1, stream)) != IV_OK) return rc;
    if (rfc6962)
        IV_TRY(ctx, ivk::launch_merkle_root_rfc6962(ctx->d_digests, n, ctx->d_root, ctx->d_tree384[0], ctx->d_tree384[1],
                                                    stream, &ctx->launches));
    else
        IV_TRY(ctx, ivk::launch_merkle_root(ctx->d_digests, n, ctx->d_root, ctx->d_merkle_a, ctx->d_merkle_b,
                                            ctx->d_tickets, stream, &ctx->launches));
    if ((rc = mark_phase(ctx, 2, stream)) != IV_OK) return rc;
    ivk::RootBytes expect;
    std::memcpy(expect.b, m->root, 32);
    IV_TRY(ctx, ivk::launch_verify_compare(ctx->d_digests, m->d_digests, n, ctx->d_root, expect, d_result,
                                           d_mismatch_idx, idx_cap, ctx->d_words,
                                           ctx->d_tickets + ivk::kMerkleMaxPasses, ctx->d_status, stream,
                                           &ctx->launches));
    if ((rc = mark_phase(ctx, 3, stream)) != IV_OK) return rc;
    ctx->slot_timed[ctx->timed_calls % IV_TIMING_RING] = ctx->timing;
    ++ctx->timed_calls;
    ctx->digests_valid = n;
    return IV_OK;
}

}  // namespace

extern "C" {

const char *iv_strerror(int code) {
    switch (code) {
        case IV_OK: return "ok";
        case IV_ERR_INVALID_ARG: return "invalid argument";
        case IV_ERR_NOMEM: return "out of memory";
        case IV_ERR_CUDA: return "CUDA runtime error";
        case IV_ERR_NO_DEVICE: return "no usable CUDA device (compute capability 10.x required)";
        case IV_ERR_TOO_LARGE: return "size exceeds the fixed limit of this entry point";
        default: return "unknown status";
    }
}

int iv_create(iv_ctx **out, int cuda_device) {
    if (!out) return IV_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || cuda_device < 0 || cuda_device >= count) {
        (void)cudaGetLastError();
        return IV_ERR_NO_DEVICE;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cuda_device) != cudaSuccess || prop.major != 10) {
        (void)cudaGetLastError();
        return IV_ERR_NO_DEVICE;   // the kernels are built for sm_100a only
    }
    iv_ctx *ctx = new (std::nothrow) iv_ctx();
    if (!ctx) return IV_ERR_NOMEM;
    ctx->device = cuda_device;
    ctx->sm_count = prop.multiProcessorCount;
    DeviceGuard guard(cuda_device);

    const size_t small_bytes = 256;
    cudaError_t e = cudaMalloc(&ctx->d_small, small_bytes);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_small, 0, small_bytes);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->tail_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_entry, cudaEventDisableTiming);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&ctx->ev_copied[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_hashed[i], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        int rc = fail_cuda(nullptr, e);
        iv_destroy(ctx);
        return rc;
    }
    uint8_t *base = static_cast<uint8_t *>(ctx->d_small);
    ctx->d_root = base;                                                   // 32 bytes
    ctx->d_queue = reinterpret_cast<unsigned long long *>(base + 64);     // 8 bytes
    ctx->d_tickets = reinterpret_cast<uint32_t *>(base + 128);            // kMerkleMaxPasses + 1 words
    ctx->d_status = reinterpret_cast<uint32_t *>(base + 192);
    ctx->d_one = reinterpret_cast<uint32_t *>(base + 224);
    {
        const uint32_t one = 1u;
        e = cudaMemcpy(ctx->d_one, &one, sizeof one, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            int rc = fail_cuda(nullptr, e);
            iv_destroy(ctx);
            return rc;
        }
    }
    *out = ctx;
    return IV_OK;
}

int iv_destroy(iv_ctx *ctx) {
    if (!ctx) return IV_OK;
    DeviceGuard guard(ctx->device);
    if (ctx->nvtx_open) nvtxRangeEnd(ctx->nvtx_id);
    cudaDeviceSynchronize();
    cudaFree(ctx->d_small);
    cudaFree(ctx->d_merkle_a);
    cudaFree(ctx->d_merkle_b);
    cudaFree(ctx->d_digests);
    cudaFree(ctx->d_words);
    cudaFree(ctx->d_slices);
    cudaFree(ctx->d_order);
    cudaFree(ctx->d_dirty_scratch);
    cudaFree(ctx->d_columns);
    cudaFree(ctx->d_digests384);
    cudaFree(ctx->d_pairs512);
    cudaFree(ctx->d_sub);
    cudaFree(ctx->d_batch);
    cudaFree(ctx->d_tree384[0]);
    cudaFree(ctx->d_tree384[1]);
    cudaFree(ctx->d_window[0]);
    cudaFree(ctx->d_window[1]);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->tail_stream) cudaStreamDestroy(ctx->tail_stream);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->ev_entry) cudaEventDestroy(ctx->ev_entry);
    for (int i = 0; i < 2; ++i) {
        if (ctx->ev_copied[i]) cudaEventDestroy(ctx->ev_copied[i]);
        if (ctx->ev_hashed[i]) cudaEventDestroy(ctx->ev_hashed[i]);
    }
    for (int r = 0; r < IV_TIMING_RING; ++r)
        for (int k = 0; k < 4; ++k)
            if (ctx->ev_phase[r][k]) cudaEventDestroy(ctx->ev_phase[r][k]);
    (void)cudaGetLastError();
    delete ctx;
    return IV_OK;
}

int iv_last_cuda_error(const iv_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

uint64_t iv_kernel_launches(const iv_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *iv_last_leaf_kernel(const iv_ctx *ctx) { return ctx ? ctx->leaf_kernel : ""; }

const char *iv_last_leaf_instance(const iv_ctx *ctx) { return ctx ? ctx->leaf_instance : ""; }

int iv_selftest_wait_timeout(iv_ctx *ctx, uint64_t limit_cycles, uint64_t *h_waited_cycles, void *cuda_stream) {
    if (!ctx || limit_cycles == 0 || limit_cycles > 4000000000ull) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    IV_TRY(ctx, ivk::launch_wait_timeout_selftest(limit_cycles, ctx->d_status, ctx->d_queue, stream, &ctx->launches));
    if (h_waited_cycles) {
        unsigned long long waited = 0;
        IV_TRY(ctx, cudaMemcpyAsync(&waited, ctx->d_queue, sizeof waited, cudaMemcpyDeviceToHost, stream));
        IV_TRY(ctx, cudaStreamSynchronize(stream));
        *h_waited_cycles = waited;
    }
    return IV_OK;
}

int iv_device_status(iv_ctx *ctx, uint32_t *h_status) {
    if (!ctx || !h_status) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    IV_TRY(ctx, cudaDeviceSynchronize());
    IV_TRY(ctx, cudaMemcpy(h_status, ctx->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost));
    if (*h_status != 0) IV_TRY(ctx, cudaMemset(ctx->d_status, 0, sizeof(uint32_t)));
    return IV_OK;
}

const uint8_t *iv_ctx_digests(const iv_ctx *ctx) {
    return (ctx && ctx->digests_valid) ? ctx->d_digests : nullptr;
}

int iv_hash_chunks(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                   uint8_t *d_digests, uint64_t digests_cap, uint64_t *h_n_chunks, void *cuda_stream) {
    if (!ctx || chunk_bytes == 0) return IV_ERR_INVALID_ARG;
    const uint64_t n = chunk_count(nbytes, chunk_bytes);
    if (n > digests_cap) return IV_ERR_INVALID_ARG;
    if (n && (!d_data || !d_digests)) return IV_ERR_INVALID_ARG;
    if (h_n_chunks) *h_n_chunks = n;
    if (n == 0) return IV_OK;
    DeviceGuard guard(ctx->device);
    return hash_leaves(ctx, static_cast<const uint8_t *>(d_data), nbytes, chunk_bytes, n, d_digests,
                       static_cast<cudaStream_t>(cuda_stream));
}

int iv_merkle_root(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root, void *cuda_stream) {
    if (!ctx || !d_root || (n_leaves && !d_leaves)) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    int rc = ensure_merkle_scratch(ctx, n_leaves);
    if (rc != IV_OK) return rc;
    IV_TRY(ctx, ivk::launch_merkle_root(d_leaves, n_leaves, d_root, ctx->d_merkle_a, ctx->d_merkle_b,
                                        ctx->d_tickets, static_cast<cudaStream_t>(cuda_stream), &ctx->launches));
    return IV_OK;
}

int iv_merkle_levels(iv_ctx *ctx, const uint8_t *d_nodes, uint64_t n, uint32_t levels, uint8_t *d_out,
                     uint64_t out_cap, uint64_t *h_n_out, void *cuda_stream) {
    if (!ctx || levels > 63) return IV_ERR_INVALID_ARG;
    uint64_t n_out = n;
    for (uint32_t l = 0; l < levels && n_out > 1; ++l) n_out = (n_out + 1) / 2;
    if (h_n_out) *h_n_out = n_out;
    if (n == 0) return IV_OK;
    if (!d_nodes || !d_out || n_out > out_cap) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (levels == 0 || n == 1) {
        IV_TRY(ctx, cudaMemcpyAsync(d_out, d_nodes, 32 * n, cudaMemcpyDeviceToDevice, stream));
        return IV_OK;
    }
    // up to nine levels per launch; intermediate level arrays ping-pong through the context's scratch
    int rc = ensure_merkle_scratch(ctx, n);       // an intermediate array exists only after nine levels: n / 512 records
    if (rc != IV_OK) return rc;
    const uint8_t *in = d_nodes;
    uint64_t cur = n;
    uint32_t left = levels;
    uint8_t *ping = ctx->d_merkle_a, *pong = ctx->d_merkle_b;
    while (left > 0 && cur > 1) {
        const uint32_t step = left > 9 ? 9 : left;
        uint64_t next = cur;
        for (uint32_t l = 0; l < step && next > 1; ++l) next = (next + 1) / 2;
        const bool last = (left == step) || next == 1;
        uint8_t *out = last ? d_out : ping;
        IV_TRY(ctx, ivk::launch_merkle_levels(in, cur, step, out, stream, &ctx->launches));
        in = out;
        uint8_t *t = ping; ping = pong; pong = t;
        cur = next;
        left -= step;
        if (last) break;
    }
    return IV_OK;
}

namespace {

// log2(chunk_bytes / sub_bytes) when the ratio is a power of two, -1 otherwise.
int two_level_shift(uint64_t chunk_bytes, uint64_t sub_bytes) {
    if (sub_bytes == 0 || chunk_bytes < sub_bytes || chunk_bytes % sub_bytes) return -1;
    uint64_t ratio = chunk_bytes / sub_bytes;
    int k = 0;
    while ((ratio & 1u) == 0) { ratio >>= 1; ++k; }
    return ratio == 1 ? k : -1;
}

// Two-level leaf digests into d_out (n = ceil(nbytes / chunk_bytes) records).
int hash_leaves_two_level(iv_ctx *ctx, const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t sub_bytes,
                          uint8_t *d_out, uint64_t n, cudaStream_t stream) {
    const int k = two_level_shift(chunk_bytes, sub_bytes);
    if (k < 0) return IV_ERR_INVALID_ARG;
    if (k == 0) return hash_leaves(ctx, d_data, nbytes, chunk_bytes, n, d_out, stream);
    const uint64_t n_sub = chunk_count(nbytes, sub_bytes);
    int rc = grow(ctx, &ctx->d_sub, &ctx->sub_cap, n_sub + 1, 32);
    if (rc != IV_OK) return rc;
    rc = hash_leaves(ctx, d_data, nbytes, sub_bytes, n_sub, ctx->d_sub, stream);
    if (rc != IV_OK) return rc;
    // the sub-leaves of chunk i are the aligned run [i * 2^k, (i+1) * 2^k): k levels up they are one node
    return iv_merkle_levels(ctx, ctx->d_sub, n_sub, (uint32_t)k, d_out, n, nullptr, stream);
}

}  // namespace

uint64_t iv_tree_records(uint64_t n_leaves) { return ivk::tree_records(n_leaves); }

int iv_hash_chunks_two_level(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t sub_bytes,
                             uint8_t *d_digests, uint64_t digests_cap, uint64_t *h_n_chunks, void *cuda_stream) {
    if (!ctx || chunk_bytes == 0 || two_level_shift(chunk_bytes, sub_bytes) < 0) return IV_ERR_INVALID_ARG;
    const uint64_t n = chunk_count(nbytes, chunk_bytes);
    if (n > digests_cap) return IV_ERR_INVALID_ARG;
    if (n && (!d_data || !d_digests)) return IV_ERR_INVALID_ARG;
    if (h_n_chunks) *h_n_chunks = n;
    if (n == 0) return IV_OK;
    DeviceGuard guard(ctx->device);
    return hash_leaves_two_level(ctx, static_cast<const uint8_t *>(d_data), nbytes, chunk_bytes, sub_bytes, d_digests, n,
                                 static_cast<cudaStream_t>(cuda_stream));
}

int iv_verify_manifest_two_level(iv_ctx *ctx, const void *d_data, uint64_t nbytes, const iv_manifest *h_manifest,
                                 uint64_t sub_bytes, iv_verify_result *d_result, uint64_t *d_mismatch_idx,
                                 uint64_t idx_cap, void *cuda_stream) {
    if (!ctx || !d_result || (idx_cap && !d_mismatch_idx)) return IV_ERR_INVALID_ARG;
    int rc = check_manifest(h_manifest, nbytes);
    if (rc != IV_OK) return rc;
    if (two_level_shift(h_manifest->chunk_bytes, sub_bytes) < 0) return IV_ERR_INVALID_ARG;
    if (nbytes && !d_data) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint64_t n = h_manifest->n_chunks;
    rc = grow(ctx, &ctx->d_digests, &ctx->digests_cap, n + 1, 32);
    if (rc != IV_OK) return rc;
    // grow everything the phases need before the first phase event, so that no allocation sits between events
    rc = grow(ctx, &ctx->d_sub, &ctx->sub_cap, chunk_count(nbytes, sub_bytes) + 1, 32);
    if (rc != IV_OK) return rc;
    if ((rc = mark_phase(ctx, 0, stream)) != IV_OK) return rc;
    if (n) {
        rc = hash_leaves_two_level(ctx, static_cast<const uint8_t *>(d_data), nbytes, h_manifest->chunk_bytes, sub_bytes,
                                   ctx->d_digests, n, stream);
        if (rc != IV_OK) return rc;
    }
    return finish_verification(ctx, h_manifest, d_result, d_mismatch_idx, idx_cap, stream);
}

int iv_tree_build(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_tree, uint64_t tree_cap,
                  void *cuda_stream) {
    if (!ctx || !d_tree || (n_leaves && !d_leaves)) return IV_ERR_INVALID_ARG;
    if (tree_cap < ivk::tree_records(n_leaves)) return IV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_tree) | reinterpret_cast<uintptr_t>(d_leaves)) & 15u) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    IV_TRY(ctx, ivk::launch_tree_build(d_leaves, n_leaves, d_tree, static_cast<cudaStream_t>(cuda_stream),
                                       &ctx->launches));
    return IV_OK;
}

int iv_tree_update(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes, const uint64_t *d_dirty,
                   uint64_t n_dirty, uint8_t *d_tree, uint64_t tree_cap, void *cuda_stream) {
    if (!ctx || chunk_bytes == 0 || !d_tree) return IV_ERR_INVALID_ARG;
    const uint64_t n = chunk_count(nbytes, chunk_bytes);
    if (tree_cap < ivk::tree_records(n)) return IV_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_tree) & 15u) return IV_ERR_INVALID_ARG;
    if (n_dirty == 0) return IV_OK;
    if (!d_dirty || !d_data || n == 0) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // scratch: offsets[n_dirty] | lengths[n_dirty] | fresh digests[n_dirty * 32]
    int rc = grow(ctx, &ctx->d_dirty_scratch, &ctx->dirty_cap, 48 * n_dirty + 64, 1);
    if (rc != IV_OK) return rc;
    uint64_t *d_off = reinterpret_cast<uint64_t *>(ctx->d_dirty_scratch);
    uint64_t *d_len = d_off + n_dirty;
    uint8_t *d_fresh = reinterpret_cast<uint8_t *>(d_len + n_dirty);
    if (n_dirty <= ivk::kRaggedSortMax) {
        rc = grow(ctx, &ctx->d_order, &ctx->order_cap, n_dirty, sizeof(uint32_t));
        if (rc != IV_OK) return rc;
    }
    IV_TRY(ctx, ivk::launch_dirty_ranges(d_dirty, n_dirty, nbytes, chunk_bytes, n, d_off, d_len, ctx->d_status, stream,
                                         &ctx->launches));
    IV_TRY(ctx, ivk::launch_hash_ragged(static_cast<const uint8_t *>(d_data), d_off, d_len, n_dirty, d_fresh,
                                        ctx->d_queue, n_dirty <= ivk::kRaggedSortMax ? ctx->d_order : nullptr,
                                        ctx->d_status, ctx->d_one, ctx->sm_count, stream, &ctx->launches,
                                        &ctx->leaf_kernel));
    IV_TRY(ctx, ivk::launch_tree_update(d_tree, n, d_fresh, d_dirty, n_dirty, stream, &ctx->launches));
    return IV_OK;
}

int iv_verify_manifest(iv_ctx *ctx, const void *d_data, uint64_t nbytes, const iv_manifest *h_manifest,
                       iv_verify_result *d_result, uint64_t *d_mismatch_idx, uint64_t idx_cap,
                       void *cuda_stream) {
    if (!ctx || !d_result || (idx_cap && !d_mismatch_idx)) return IV_ERR_INVALID_ARG;
    int rc = check_manifest(h_manifest, nbytes);
    if (rc != IV_OK) return rc;
    if (nbytes && !d_data) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint64_t n = h_manifest->n_chunks;
    rc = grow(ctx, &ctx->d_digests, &ctx->digests_cap, n + 1, 32);
    if (rc != IV_OK) return rc;
    if ((rc = mark_phase(ctx, 0, stream)) != IV_OK) return rc;
    rc = hash_leaves(ctx, static_cast<const uint8_t *>(d_data), nbytes, h_manifest->chunk_bytes, n, ctx->d_digests,
                     stream);
    if (rc != IV_OK) return rc;
    return finish_verification(ctx, h_manifest, d_result, d_mismatch_idx, idx_cap, stream);
}

int iv_verify_manifest_batch(iv_ctx *ctx, const void *const *h_d_blobs, uint64_t n_blobs, uint64_t nbytes,
                             const iv_manifest *h_manifest, iv_verify_result *d_results, uint64_t *d_mismatch_idx,
                             uint64_t idx_cap, void *cuda_stream) {
    if (!ctx || !d_results || (idx_cap && !d_mismatch_idx)) return IV_ERR_INVALID_ARG;
    if (n_blobs == 0) return IV_OK;
    if (!h_d_blobs) return IV_ERR_INVALID_ARG;
    if (n_blobs > ivk::kMaxBatch) return IV_ERR_TOO_LARGE;
    int rc = check_manifest(h_manifest, nbytes);
    if (rc != IV_OK) return rc;
    ivk::BlobList blobs{};
    blobs.count = (uint32_t)n_blobs;
    for (uint64_t b = 0; b < n_blobs; ++b) {
        if (nbytes && !h_d_blobs[b]) return IV_ERR_INVALID_ARG;
        blobs.ptr[b] = static_cast<const uint8_t *>(h_d_blobs[b]);
    }
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint64_t n = h_manifest->n_chunks, total = n * n_blobs;
    rc = grow(ctx, &ctx->d_digests, &ctx->digests_cap, total + 1, 32);
    if (rc != IV_OK) return rc;
    // scratch: offsets[total] | lengths[total] | one root per blob | 512 run roots per blob | one ticket per blob
    const uint64_t batch_bytes = 16 * total + 32 * n_blobs + 32ull * ivk::kMerkleRun * n_blobs + 4 * n_blobs + 64;
    const bool fresh = batch_bytes > ctx->batch_cap;
    rc = grow(ctx, &ctx->d_batch, &ctx->batch_cap, batch_bytes, 1);
    if (rc != IV_OK) return rc;
    uint64_t *d_off = reinterpret_cast<uint64_t *>(ctx->d_batch);
    uint64_t *d_len = d_off + total;
    uint8_t *d_roots = reinterpret_cast<uint8_t *>(d_len + total);
    uint8_t *d_runs = d_roots + 32 * n_blobs;
    uint32_t *d_btickets = reinterpret_cast<uint32_t *>(d_runs + 32ull * ivk::kMerkleRun * n_blobs);
    // tickets must start at zero (the kernel leaves them at zero); a regrown or differently shaped scratch is cleared
    if (fresh || ctx->batch_blobs != n_blobs || ctx->batch_total != total) {
        IV_TRY(ctx, cudaMemsetAsync(d_btickets, 0, 4 * n_blobs, stream));
        ctx->batch_blobs = n_blobs;
        ctx->batch_total = total;
    }
    if (total && total <= ivk::kRaggedSortMax) {
        rc = grow(ctx, &ctx->d_order, &ctx->order_cap, total, sizeof(uint32_t));
        if (rc != IV_OK) return rc;
    }
    rc = ensure_merkle_scratch(ctx, n);
    if (rc != IV_OK) return rc;
    rc = grow(ctx, &ctx->d_words, &ctx->words_cap, (n + 31) / 32 + 1, sizeof(uint32_t));
    if (rc != IV_OK) return rc;
    if (total) {
        // all blobs' chunks are independent chains of one launch
        IV_TRY(ctx, ivk::launch_batch_ranges(blobs, n, nbytes, h_manifest->chunk_bytes, d_off, d_len, stream,
                                             &ctx->launches));
        IV_TRY(ctx, ivk::launch_hash_ragged(blobs.ptr[0], d_off, d_len, total, ctx->d_digests, ctx->d_queue,
                                            total <= ivk::kRaggedSortMax ? ctx->d_order : nullptr, ctx->d_status,
                                            ctx->d_one, ctx->sm_count, stream, &ctx->launches, &ctx->leaf_kernel));
    }
    ivk::RootBytes expect;
    std::memcpy(expect.b, h_manifest->root, 32);
    const bool one_pass = n > 0 && n <= (uint64_t)ivk::kMerkleRun * ivk::kMerkleRun;
    if (one_pass)      // all trees in one launch
        IV_TRY(ctx, ivk::launch_merkle_roots_batch(ctx->d_digests, n, (uint32_t)n_blobs, d_roots, d_runs, d_btickets, stream,
                                                   &ctx->launches));
    for (uint64_t b = 0; b < n_blobs; ++b) {
        const uint8_t *dig = ctx->d_digests + 32 * n * b;
        if (!one_pass)
            IV_TRY(ctx, ivk::launch_merkle_root(dig, n, d_roots + 32 * b, ctx->d_merkle_a, ctx->d_merkle_b, ctx->d_tickets,
                                                stream, &ctx->launches));
        IV_TRY(ctx, ivk::launch_verify_compare(dig, h_manifest->d_digests, n, d_roots + 32 * b, expect, d_results + b,
                                               idx_cap ? d_mismatch_idx + b * idx_cap : nullptr, idx_cap, ctx->d_words,
                                               ctx->d_tickets + ivk::kMerkleMaxPasses, ctx->d_status, stream,
                                               &ctx->launches));
    }
    ctx->digests_valid = total;
    return IV_OK;
}

int iv_verify_streamed(iv_ctx *ctx, const void *const *h_windows, uint64_t n_windows, uint64_t window_bytes,
                       uint64_t nbytes, const iv_manifest *h_manifest, iv_verify_result *d_result,
                       uint64_t *d_mismatch_idx, uint64_t idx_cap, void *cuda_stream) {
    if (!ctx || !d_result || (idx_cap && !d_mismatch_idx)) return IV_ERR_INVALID_ARG;
    int rc = check_manifest(h_manifest, nbytes);
    if (rc != IV_OK) return rc;
    const uint64_t chunk = h_manifest->chunk_bytes;
    if (window_bytes == 0 || window_bytes % chunk != 0) return IV_ERR_INVALID_ARG;
    if (n_windows != chunk_count(nbytes, window_bytes)) return IV_ERR_INVALID_ARG;
    if (n_windows && !h_windows) return IV_ERR_INVALID_ARG;
    for (uint64_t w = 0; w < n_windows; ++w)
        if (!h_windows[w]) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint64_t n = h_manifest->n_chunks;
    rc = grow(ctx, &ctx->d_digests, &ctx->digests_cap, n + 1, 32);
    if (rc != IV_OK) return rc;

    const uint64_t win = window_bytes < nbytes ? window_bytes : nbytes;
    if (win > ctx->window_cap) {
        IV_TRY(ctx, cudaDeviceSynchronize());
        for (int i = 0; i < 2; ++i) {
            if (ctx->d_window[i]) IV_TRY(ctx, cudaFree(ctx->d_window[i]));
            ctx->d_window[i] = nullptr;
        }
        ctx->window_cap = 0;
        for (int i = 0; i < 2; ++i) {
            void *p = nullptr;
            IV_TRY(ctx, cudaMalloc(&p, win));
            ctx->d_window[i] = static_cast<uint8_t *>(p);
        }
        ctx->window_cap = win;
    }

    if ((rc = mark_phase(ctx, 0, stream)) != IV_OK) return rc;
    // The copy stream starts after everything already enqueued on the caller's
    // stream (which includes the previous call's use of the windows).
    IV_TRY(ctx, cudaEventRecord(ctx->ev_entry, stream));
    IV_TRY(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_entry, 0));
    const uint64_t chunks_per_window = window_bytes / chunk;
    for (uint64_t w = 0; w < n_windows; ++w) {
        const int b = (int)(w & 1u);
        const uint64_t off = w * window_bytes;
        const uint64_t bytes = nbytes - off < window_bytes ? nbytes - off : window_bytes;
        if (w >= 2) IV_TRY(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_hashed[b], 0));
        {
            // With few chunks the hashing of a window lasts as long as ONE chunk's serial chain, whatever the
            // window's size, and it can start only when the window has arrived: the hashing runs a window
            // behind the copies and nothing overlaps the last one.  So a window arrives in column parts (part s
            // of every chunk, one strided copy) and part s is hashed, from the chaining values part s - 1 left,
            // while part s + 1 is on its way: what remains after the last byte is one part's time.
            const uint64_t m = chunk_count(bytes, chunk);
            const uint64_t parts = chunk / 16384 < 16 ? chunk / 16384 : 16;     // parts of at least 16 KiB
            if (parts >= 2 && chunk < (1ull << 31) && m <= 2ull * 32 * (uint64_t)ctx->sm_count && m <= ivk::kRaggedSortMax) {
                rc = hash_window_in_columns(ctx, h_windows[w], bytes, chunk, m, (uint32_t)parts, b,
                                            ctx->d_digests + 32 * w * chunks_per_window, stream);
                if (rc != IV_OK) return rc;
                IV_TRY(ctx, cudaEventRecord(ctx->ev_hashed[b], stream));
                continue;
            }
        }
        IV_TRY(ctx, cudaMemcpyAsync(ctx->d_window[b], h_windows[w], bytes, cudaMemcpyHostToDevice, ctx->copy_stream));
        IV_TRY(ctx, cudaEventRecord(ctx->ev_copied[b], ctx->copy_stream));
        IV_TRY(ctx, cudaStreamWaitEvent(stream, ctx->ev_copied[b], 0));
        rc = hash_leaves(ctx, ctx->d_window[b], bytes, chunk, chunk_count(bytes, chunk),
                         ctx->d_digests + 32 * w * chunks_per_window, stream);
        if (rc != IV_OK) return rc;
        IV_TRY(ctx, cudaEventRecord(ctx->ev_hashed[b], stream));
    }
    return finish_verification(ctx, h_manifest, d_result, d_mismatch_idx, idx_cap, stream);
}

int iv_set_timing(iv_ctx *ctx, int enabled) {
    if (!ctx) return IV_ERR_INVALID_ARG;
    ctx->timing = enabled != 0;
    return IV_OK;
}

int iv_phase_times(iv_ctx *ctx, uint32_t calls_back, float *h_ms) {
    if (!ctx || !h_ms || calls_back >= IV_TIMING_RING || calls_back >= ctx->timed_calls) return IV_ERR_INVALID_ARG;
    const uint32_t slot = (uint32_t)((ctx->timed_calls - 1 - calls_back) % IV_TIMING_RING);
    if (!ctx->slot_timed[slot]) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    IV_TRY(ctx, cudaEventSynchronize(ctx->ev_phase[slot][3]));
    for (int k = 0; k < 3; ++k)
        IV_TRY(ctx, cudaEventElapsedTime(&h_ms[k], ctx->ev_phase[slot][k], ctx->ev_phase[slot][k + 1]));
    return IV_OK;
}

int iv_hash_ragged(iv_ctx *ctx, const void *d_base, const uint64_t *d_offsets, const uint64_t *d_lengths,
                   uint64_t n, uint8_t *d_digests, void *cuda_stream) {
    if (!ctx) return IV_ERR_INVALID_ARG;
    if (n == 0) return IV_OK;
    if (!d_base || !d_offsets || !d_lengths || !d_digests) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (n <= ivk::kRaggedSortMax) {
        int rc = grow(ctx, &ctx->d_order, &ctx->order_cap, n, sizeof(uint32_t));
        if (rc != IV_OK) return rc;
    }
    IV_TRY(ctx, ivk::launch_hash_ragged(static_cast<const uint8_t *>(d_base), d_offsets, d_lengths, n, d_digests,
                                        ctx->d_queue, n <= ivk::kRaggedSortMax ? ctx->d_order : nullptr,
                                        ctx->d_status, ctx->d_one, ctx->sm_count,
                                        static_cast<cudaStream_t>(cuda_stream), &ctx->launches, &ctx->leaf_kernel));
    return IV_OK;
}

int iv_hash_ragged_update(iv_ctx *ctx, const void *d_base, const uint64_t *d_offsets, const uint64_t *d_lengths,
                          uint64_t n, iv_sha_state *d_states, int finish, uint8_t *d_digests, void *cuda_stream) {
    if (!ctx) return IV_ERR_INVALID_ARG;
    if (n == 0) return IV_OK;
    if (!d_base || !d_offsets || !d_lengths || !d_states || (finish && !d_digests)) return IV_ERR_INVALID_ARG;
    if (n > ivk::kRaggedSortMax) return IV_ERR_TOO_LARGE;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // index order: the parts of one tensor set keep the same message-to-lane assignment from call to call
    IV_TRY(ctx, ivk::launch_hash_ragged_split(static_cast<const uint8_t *>(d_base), d_offsets, d_lengths, nullptr, n,
                                              d_digests, ctx->d_status, ctx->d_one, d_states, finish, stream));
    ++ctx->launches;
    ctx->leaf_kernel = "hash_chunks_split_kernel (tensors)";
    return IV_OK;
}

namespace {

int hash_chunks_wide(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint8_t *d_digests,
                     uint64_t digests_cap, uint64_t *h_n_chunks, int digest_words, void *cuda_stream) {
    if (!ctx || chunk_bytes == 0) return IV_ERR_INVALID_ARG;
    const uint64_t n = chunk_count(nbytes, chunk_bytes);
    if (n > digests_cap) return IV_ERR_INVALID_ARG;
    if (n && (!d_data || !d_digests)) return IV_ERR_INVALID_ARG;
    if (h_n_chunks) *h_n_chunks = n;
    if (n == 0) return IV_OK;
    DeviceGuard guard(ctx->device);
    return hash_leaves_wide(ctx, static_cast<const uint8_t *>(d_data), nbytes, chunk_bytes, n, d_digests, digest_words,
                            static_cast<cudaStream_t>(cuda_stream));
}

int merkle_root_wide(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root, int digest_words,
                     void *cuda_stream) {
    if (!ctx || !d_root || (n_leaves && !d_leaves)) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    int rc = ensure_variant_tree_scratch(ctx, (n_leaves + 1) / 2 + 1);
    if (rc != IV_OK) return rc;
    IV_TRY(ctx, ivk::launch_merkle_root_sha384(d_leaves, n_leaves, d_root, ctx->d_tree384[0], ctx->d_tree384[1], digest_words,
                                               static_cast<cudaStream_t>(cuda_stream), &ctx->launches));
    return IV_OK;
}

}  // namespace

int iv_hash_chunks_sha384(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint8_t *d_digests,
                          uint64_t digests_cap, uint64_t *h_n_chunks, void *cuda_stream) {
    return hash_chunks_wide(ctx, d_data, nbytes, chunk_bytes, d_digests, digests_cap, h_n_chunks, 6, cuda_stream);
}

int iv_merkle_root_sha384(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root, void *cuda_stream) {
    return merkle_root_wide(ctx, d_leaves, n_leaves, d_root, 6, cuda_stream);
}

int iv_hash_chunks_sha512(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint8_t *d_digests,
                          uint64_t digests_cap, uint64_t *h_n_chunks, void *cuda_stream) {
    return hash_chunks_wide(ctx, d_data, nbytes, chunk_bytes, d_digests, digests_cap, h_n_chunks, 8, cuda_stream);
}

int iv_merkle_root_sha512(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root, void *cuda_stream) {
    return merkle_root_wide(ctx, d_leaves, n_leaves, d_root, 8, cuda_stream);
}

extern "C++" {
namespace {

// iv_verify_manifest over SHA-384 (WORDS 6) or SHA-512 (8) records: hash, tree, compare.
template <int WORDS, class Manifest, class Result, class Root>
int verify_manifest_wide(iv_ctx *ctx, const void *d_data, uint64_t nbytes, const Manifest *m, Result *d_result,
                         uint64_t *d_mismatch_idx, uint64_t idx_cap, void *cuda_stream,
                         cudaError_t (*compare)(const uint8_t *, const uint8_t *, uint64_t, const uint8_t *, Root, Result *,
                                                uint64_t *, uint64_t, uint32_t *, uint32_t *, const uint32_t *, cudaStream_t,
                                                uint64_t *)) {
    constexpr uint64_t REC = 8 * WORDS;
    if (!ctx || !d_result || (idx_cap && !d_mismatch_idx)) return IV_ERR_INVALID_ARG;
    if (!m || m->chunk_bytes == 0 || m->total_bytes != nbytes) return IV_ERR_INVALID_ARG;
    const uint64_t n = chunk_count(nbytes, m->chunk_bytes);
    if (m->n_chunks != n || (n && !m->d_digests) || (nbytes && !d_data)) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int rc = grow(ctx, &ctx->d_digests384, &ctx->digests384_cap, n + 2, 64);      // digests, then the root
    if (rc != IV_OK) return rc;
    if ((rc = ensure_variant_tree_scratch(ctx, (n + 1) / 2 + 1)) != IV_OK) return rc;
    if ((rc = grow(ctx, &ctx->d_words, &ctx->words_cap, (n + 31) / 32 + 1, sizeof(uint32_t))) != IV_OK) return rc;
    uint8_t *d_root = ctx->d_digests384 + REC * (n + 1);
    if (n && (rc = hash_leaves_wide(ctx, static_cast<const uint8_t *>(d_data), nbytes, m->chunk_bytes, n, ctx->d_digests384,
                                    WORDS, stream)) != IV_OK)
        return rc;
    IV_TRY(ctx, ivk::launch_merkle_root_sha384(ctx->d_digests384, n, d_root, ctx->d_tree384[0], ctx->d_tree384[1], WORDS,
                                               stream, &ctx->launches));
    Root expect;
    std::memcpy(expect.b, m->root, REC);
    IV_TRY(ctx, compare(ctx->d_digests384, m->d_digests, n, d_root, expect, d_result, d_mismatch_idx, idx_cap, ctx->d_words,
                        ctx->d_tickets + ivk::kMerkleMaxPasses, ctx->d_status, stream, &ctx->launches));
    return IV_OK;
}

}  // namespace
}  // extern "C++"

int iv_verify_manifest_sha384(iv_ctx *ctx, const void *d_data, uint64_t nbytes, const iv_manifest_sha384 *m,
                              iv_verify_result_sha384 *d_result, uint64_t *d_mismatch_idx, uint64_t idx_cap,
                              void *cuda_stream) {
    return verify_manifest_wide<6, iv_manifest_sha384, iv_verify_result_sha384, ivk::RootBytes384>(
        ctx, d_data, nbytes, m, d_result, d_mismatch_idx, idx_cap, cuda_stream, ivk::launch_verify_compare_sha384);
}

int iv_verify_manifest_sha512(iv_ctx *ctx, const void *d_data, uint64_t nbytes, const iv_manifest_sha512 *m,
                              iv_verify_result_sha512 *d_result, uint64_t *d_mismatch_idx, uint64_t idx_cap,
                              void *cuda_stream) {
    return verify_manifest_wide<8, iv_manifest_sha512, iv_verify_result_sha512, ivk::RootBytes512>(
        ctx, d_data, nbytes, m, d_result, d_mismatch_idx, idx_cap, cuda_stream, ivk::launch_verify_compare_sha512);
}

int iv_hash_chunks_rfc6962(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint8_t *d_digests,
                           uint64_t digests_cap, uint64_t *h_n_chunks, void *cuda_stream) {
    if (!ctx || chunk_bytes == 0) return IV_ERR_INVALID_ARG;
    const uint64_t n = chunk_count(nbytes, chunk_bytes);
    if (n > digests_cap) return IV_ERR_INVALID_ARG;
    if (n && (!d_data || !d_digests)) return IV_ERR_INVALID_ARG;
    if (h_n_chunks) *h_n_chunks = n;
    if (n == 0) return IV_OK;
    DeviceGuard guard(ctx->device);
    return hash_leaves_rfc6962(ctx, static_cast<const uint8_t *>(d_data), nbytes, chunk_bytes, n, d_digests,
                               static_cast<cudaStream_t>(cuda_stream));
}

int iv_verify_manifest_rfc6962(iv_ctx *ctx, const void *d_data, uint64_t nbytes, const iv_manifest *h_manifest,
                               iv_verify_result *d_result, uint64_t *d_mismatch_idx, uint64_t idx_cap,
                               void *cuda_stream) {
    if (!ctx || !d_result || (idx_cap && !d_mismatch_idx)) return IV_ERR_INVALID_ARG;
    int rc = check_manifest(h_manifest, nbytes);
    if (rc != IV_OK) return rc;
    if (nbytes && !d_data) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint64_t n = h_manifest->n_chunks;
    rc = grow(ctx, &ctx->d_digests, &ctx->digests_cap, n + 1, 32);
    if (rc != IV_OK) return rc;
    if ((rc = mark_phase(ctx, 0, stream)) != IV_OK) return rc;
    rc = hash_leaves_rfc6962(ctx, static_cast<const uint8_t *>(d_data), nbytes, h_manifest->chunk_bytes, n,
                             ctx->d_digests, stream);
    if (rc != IV_OK) return rc;
    return finish_verification(ctx, h_manifest, d_result, d_mismatch_idx, idx_cap, stream, true);
}

int iv_merkle_root_rfc6962(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root, void *cuda_stream) {
    if (!ctx || !d_root || (n_leaves && !d_leaves)) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    int rc = ensure_variant_tree_scratch(ctx, (n_leaves + 1) / 2 + 1);
    if (rc != IV_OK) return rc;
    IV_TRY(ctx, ivk::launch_merkle_root_rfc6962(d_leaves, n_leaves, d_root, ctx->d_tree384[0], ctx->d_tree384[1],
                                                static_cast<cudaStream_t>(cuda_stream), &ctx->launches));
    return IV_OK;
}

int iv_probe_alu(iv_ctx *ctx, int kind, uint32_t warps_per_block, uint32_t blocks_per_sm, uint32_t active_lanes,
                 uint32_t iters, double *h_out) {
    if (!ctx || !h_out || warps_per_block == 0 || warps_per_block > 32 || blocks_per_sm == 0 ||
        blocks_per_sm > 32 || active_lanes == 0 || active_lanes > 32 || iters == 0)
        return IV_ERR_INVALID_ARG;
    if (kind < IV_PROBE_IADD3 || kind > IV_PROBE_SCHEDULE) return IV_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    const unsigned blocks = blocks_per_sm * (unsigned)ctx->sm_count;
    unsigned long long *d_cycles = nullptr;
    IV_TRY(ctx, cudaMalloc(&d_cycles, sizeof(unsigned long long) * blocks + 64));
    uint32_t *d_sink = reinterpret_cast<uint32_t *>(d_cycles + blocks);
    const uint32_t sink_init[2] = {0u, 1u};     // word 1 is the multiplier "1" some probe kernels read
    unsigned long long *h_cycles = static_cast<unsigned long long *>(std::malloc(sizeof(unsigned long long) * blocks));
    int rc = IV_OK;
    cudaError_t e = h_cycles ? cudaSuccess : cudaErrorMemoryAllocation;
    if (e == cudaSuccess) e = cudaMemcpy(d_sink, sink_init, sizeof sink_init, cudaMemcpyHostToDevice);
    for (int rep = 0; rep < 2 && e == cudaSuccess; ++rep) {   // first launch warms the instruction cache
        e = ivk::launch_probe(kind, blocks, 32u * warps_per_block, iters, active_lanes, d_cycles, d_sink, nullptr);
        ++ctx->launches;
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
    }
    if (e == cudaSuccess)
        e = cudaMemcpy(h_cycles, d_cycles, sizeof(unsigned long long) * blocks, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) {
        double sum = 0.0;
        for (unsigned b = 0; b < blocks; ++b) sum += (double)h_cycles[b];
        const double mean = sum / blocks;
        double per_thread = (double)ivk::probe_ops_per_thread(kind, iters);
        if (ivk::probe_counts_blocks(kind)) per_thread *= 64.0;       // bytes per compression
        h_out[0] = (double)blocks_per_sm * warps_per_block * active_lanes * per_thread / mean;
        h_out[1] = mean;
    } else {
        rc = fail_cuda(ctx, e);
    }
    std::free(h_cycles);
    cudaFree(d_cycles);
    return rc;
}

}  // extern "C"
