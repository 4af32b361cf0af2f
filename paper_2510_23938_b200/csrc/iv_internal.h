// Internal interfaces between the C-ABI layer (iv_api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

#include "../../include/iv.h"

namespace ivk {

// Opts a kernel into `bytes` of dynamic shared memory on the CURRENT device, once per device and
// kernel (the attribute is per device; a process may drive several GPUs).  `done` is the caller's
// static table, one flag per device ordinal.
constexpr int kMaxDevices = 64;
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, size_t bytes, bool (&done)[kMaxDevices]) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) done[dev] = true;
    return e;
}

// Device-side status values written to iv_verify_result::status.
enum : uint32_t { IVK_DEV_OK = 0, IVK_DEV_TIMEOUT = 1, IVK_DEV_BOUNDS = 2 };

// Leaves reduced by one CTA of the Merkle kernel (2^9): nine tree levels per pass.
constexpr uint32_t kMerkleRun = 512;

// hash_chunks.cu -----------------------------------------------------------
// One SHA-256 per chunk: digest i <- SHA-256(data[i*C .. min((i+1)*C, nbytes))).
cudaError_t launch_hash_chunks(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                               uint64_t n_chunks, uint8_t *d_digests, int sm_count, uint32_t *d_status,
                               const uint32_t *d_one, void *d_slice_scratch, cudaStream_t stream,
                               uint64_t *launches, const char **kernel_used, cudaStream_t tail_stream = nullptr);
// tail_stream (here and in the variants' launchers): where the kernel for what the tiled copies leave out -- a blob's
// short last chunk, one long serial chain -- is launched; NULL = on `stream`, after the main kernel.  A caller that
// has forked a second stream off `stream` passes it, and the chain runs beside the main kernel.
// True when launch_hash_chunks would use the sliced kernel (and so needs its scratch).
bool hash_chunks_wants_slices(const uint8_t *d_data, uint64_t chunk_bytes, uint64_t n_chunks, int sm_count);

// hash_chunks_split.cu ------------------------------------------------------
// Same result for base and chunk size multiples of 16 bytes; two warps per 32 chains
// (schedule producer + round consumer), for launches with few chains.
cudaError_t launch_hash_chunks_split(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                                     uint64_t n_chunks, uint8_t *d_digests, uint32_t *d_status,
                                     const uint32_t *d_one, cudaStream_t stream, bool zero_prefix = false);

// hash_chunks_sliced.cu -----------------------------------------------------
// Same result for many chunks of at least 32 KiB (16-byte aligned): chunks are cut into slices
// that persistent warps take from a FIFO, so chains migrate between SM schedulers and the load
// stays level.  d_scratch must hold sliced_scratch_bytes(...) bytes.
uint64_t sliced_scratch_bytes(uint64_t n_chunks, uint64_t chunk_bytes, uint64_t *slice_bytes_out,
                              uint64_t *total_tasks_out, uint64_t nbytes);
// *covered receives the number of leading chunks the launch hashes (all, or all but a short last chunk).
// zero_prefix: hash 0x00 || chunk instead of the chunk (the RFC 6962 leaf hash).
cudaError_t launch_hash_chunks_sliced(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                                      uint64_t n_chunks, uint8_t *d_digests, uint32_t *d_status, void *d_scratch,
                                      const uint32_t *d_one, int sm_count, cudaStream_t stream, uint64_t *covered,
                                      bool zero_prefix = false);
// Which instance of the sliced kernel the calling host thread's last launch_hash_chunks_sliced picked
// (worker count and service order); static text.
const char *sliced_instance_name();

// The same two-warp kernel for tensors at any alignment; message k of the launch is tensor d_order[k]
// (d_order may be NULL for index order).
// d_states (may be NULL): resumable hashing, see iv_hash_ragged_update; finish = 0 leaves the messages open.
cudaError_t launch_hash_ragged_split(const uint8_t *d_base, const uint64_t *d_offsets, const uint64_t *d_lengths,
                                     const uint32_t *d_order, uint64_t n, uint8_t *d_digests, uint32_t *d_status,
                                     const uint32_t *d_one, iv_sha_state *d_states, int finish, cudaStream_t stream);

// hash_ragged.cu -----------------------------------------------------------
// One SHA-256 per (offset, length).  Up to kRaggedSortMax tensors are ordered by descending length
// (d_order: n uint32 of scratch) and hashed by the two-warp kernel; larger sets go through the
// per-lane work queue (d_queue: one uint64 counter).
constexpr uint64_t kRaggedSortMax = 32768;
cudaError_t launch_hash_ragged(const uint8_t *d_base, const uint64_t *d_offsets,
                               const uint64_t *d_lengths, uint64_t n, uint8_t *d_digests,
                               unsigned long long *d_queue, uint32_t *d_order, uint32_t *d_status,
                               const uint32_t *d_one, int sm_count, cudaStream_t stream, uint64_t *launches,
                               const char **kernel_used);

// merkle.cu ----------------------------------------------------------------
// Root of n leaves.  d_scratch_a / d_scratch_b each hold ceil(n / kMerkleRun)
// digests; d_ticket is one zeroed uint32 per pass (kMerkleMaxPasses of them).
constexpr int kMerkleMaxPasses = 8;
cudaError_t launch_merkle_root(const uint8_t *d_leaves, uint64_t n, uint8_t *d_root,
                               uint8_t *d_scratch_a, uint8_t *d_scratch_b, uint32_t *d_tickets,
                               cudaStream_t stream, uint64_t *launches);

// Roots of `trees` trees of n <= 262,144 leaves each in ONE launch (leaves of tree y at d_leaves + 32 n y):
// d_scratch holds trees * 512 records, d_tickets `trees` zeroed words.
cudaError_t launch_merkle_roots_batch(const uint8_t *d_leaves, uint64_t n, uint32_t trees, uint8_t *d_roots,
                                      uint8_t *d_scratch, uint32_t *d_tickets, cudaStream_t stream, uint64_t *launches);

// `levels` in 1..9 levels of the reduction: d_in[n] -> d_out[ceil(n / 2^levels)] (no aliasing).
cudaError_t launch_merkle_levels(const uint8_t *d_in, uint64_t n, uint32_t levels, uint8_t *d_out,
                                 cudaStream_t stream, uint64_t *launches);

// Several blobs of equal size verified in one pass (batch verification): their chunks as one tensor list.
constexpr uint32_t kMaxBatch = 64;
struct BlobList {
    const uint8_t *ptr[kMaxBatch];
    uint32_t count;
};
cudaError_t launch_batch_ranges(const BlobList &blobs, uint64_t n_chunks, uint64_t nbytes, uint64_t chunk_bytes,
                                uint64_t *d_offsets, uint64_t *d_lengths, cudaStream_t stream, uint64_t *launches);

// Retained tree (all levels in one array, leaves first, the root last).
constexpr int kTreeMaxLevels = 40;
uint64_t tree_records(uint64_t n_leaves);
cudaError_t launch_tree_build(const uint8_t *d_leaves, uint64_t n, uint8_t *d_tree, cudaStream_t stream,
                              uint64_t *launches);
// Offsets and lengths of the column parts of a window's m chunks (entry s * m + i = part s of chunk i): a chunk's
// whole blocks are cut into `parts` pieces of part_bytes (a multiple of 64), the last part takes the rest.
cudaError_t launch_column_ranges(uint64_t m, uint64_t bytes, uint64_t chunk_bytes, uint64_t part_bytes, uint32_t parts,
                                 uint64_t *d_offsets, uint64_t *d_lengths, cudaStream_t stream, uint64_t *launches);
cudaError_t launch_dirty_ranges(const uint64_t *d_dirty, uint64_t n_dirty, uint64_t nbytes, uint64_t chunk_bytes,
                                uint64_t n_leaves, uint64_t *d_offsets, uint64_t *d_lengths, uint32_t *d_status,
                                cudaStream_t stream, uint64_t *launches);
// d_fresh: the new digests of the dirty leaves in dirty-list order.  Writes them into the leaf
// level and recomputes every ancestor of a dirty leaf.
cudaError_t launch_tree_update(uint8_t *d_tree, uint64_t n_leaves, const uint8_t *d_fresh, const uint64_t *d_dirty,
                               uint64_t n_dirty, cudaStream_t stream, uint64_t *launches);

// Compare n computed digests with the manifest's, compact the mismatching
// indices in ascending order, compare the root.  d_words holds ceil(n/32)
// uint32 mask words; d_ticket one zeroed uint32.
struct RootBytes { uint8_t b[32]; };
struct RootBytes384 { uint8_t b[48]; };
struct RootBytes512 { uint8_t b[64]; };
cudaError_t launch_verify_compare_sha512(const uint8_t *d_digests, const uint8_t *d_manifest_digests,
                                         uint64_t n, const uint8_t *d_root, RootBytes512 manifest_root,
                                         iv_verify_result_sha512 *d_result, uint64_t *d_mismatch_idx,
                                         uint64_t idx_cap, uint32_t *d_words, uint32_t *d_ticket,
                                         const uint32_t *d_status, cudaStream_t stream, uint64_t *launches);
cudaError_t launch_verify_compare_sha384(const uint8_t *d_digests, const uint8_t *d_manifest_digests,
                                         uint64_t n, const uint8_t *d_root, RootBytes384 manifest_root,
                                         iv_verify_result_sha384 *d_result, uint64_t *d_mismatch_idx,
                                         uint64_t idx_cap, uint32_t *d_words, uint32_t *d_ticket,
                                         const uint32_t *d_status, cudaStream_t stream, uint64_t *launches);
cudaError_t launch_verify_compare(const uint8_t *d_digests, const uint8_t *d_manifest_digests,
                                  uint64_t n, const uint8_t *d_root, RootBytes manifest_root,
                                  iv_verify_result *d_result, uint64_t *d_mismatch_idx,
                                  uint64_t idx_cap, uint32_t *d_words, uint32_t *d_ticket,
                                  const uint32_t *d_status, cudaStream_t stream, uint64_t *launches);

// hash_chunks_pairs.cu -----------------------------------------------------
// Between few and many chains (2 x SMs < groups of 32 chains < about 3 x SMs): the 2 x SMs producer/consumer
// warp pairs as persistent workers on the slice FIFO.  d_scratch as for launch_hash_chunks_sliced.
bool hash_chunks_wants_pairs(const uint8_t *d_data, uint64_t chunk_bytes, uint64_t n_chunks, int sm_count);
cudaError_t launch_hash_chunks_pairs(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                                     uint8_t *d_digests, uint32_t *d_status, void *d_scratch, const uint32_t *d_one,
                                     int sm_count, cudaStream_t stream, bool zero_prefix = false);

// hash_sha384.cu -----------------------------------------------------------
// SHA-384 / SHA-512 variants (digest_words = 6 / 8): chunk digests of 48 / 64 bytes and the tree whose parents
// are the same hash.  With d_pairs_scratch (sha512_pairs_scratch_bytes(...) bytes, may be NULL) shapes that
// sha512_wants_pairs go through the two-warp kernel of hash_sha512_pairs.cu.
cudaError_t launch_hash_chunks_sha384(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                                      uint8_t *d_digests, int digest_words, int sm_count, uint32_t *d_status,
                                      void *d_pairs_scratch, cudaStream_t stream, uint64_t *launches,
                                      const char **kernel_used, cudaStream_t tail_stream = nullptr);
cudaError_t launch_merkle_root_sha384(const uint8_t *d_leaves, uint64_t n, uint8_t *d_root, uint8_t *d_scratch_a,
                                      uint8_t *d_scratch_b, int digest_words, cudaStream_t stream, uint64_t *launches);

// hash_sha512_pairs.cu ------------------------------------------------------
// 16-byte aligned blobs with at least one whole chunk of 16 KiB or more (a multiple of 16 bytes), at group counts
// where the two-warp kernel is the faster one; sha512_pairs_per_sm is the number of producer/consumer pairs per
// SM it then runs with (2, 4, 6 or 8).
bool sha512_wants_pairs(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, int sm_count);
int sha512_pairs_per_sm(uint64_t groups, uint64_t chunk_bytes, int sm_count);
const char *sha512_pairs_instance_name();     // launch shape of the calling thread's last two-warp launch
uint64_t sha512_pairs_scratch_bytes(uint64_t nbytes, uint64_t chunk_bytes);
// Hashes the blob's whole chunks (*covered of them, from the front; 0 and nothing launched if the blob cannot be
// described to the TMA unit); a short last chunk is left to the caller.
cudaError_t launch_hash_sha512_pairs(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint8_t *d_digests,
                                     int digest_words, uint32_t *d_status, void *d_scratch, int sm_count,
                                     cudaStream_t stream, uint64_t *covered, uint64_t *launches);

// hash_rfc6962.cu ----------------------------------------------------------
// RFC 6962 section 2.1 mode: prefixed leaf hashes and the tree with prefixed nodes.
// With d_slice_scratch (sliced_scratch_bytes(...) bytes) and a launch shape that wants slices
// (hash_chunks_wants_slices) the chains migrate as on the default path; otherwise one chain per lane.
cudaError_t launch_hash_chunks_rfc6962(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                                       uint8_t *d_digests, int sm_count, uint32_t *d_status, const uint32_t *d_one,
                                       void *d_slice_scratch, cudaStream_t stream, uint64_t *launches,
                                       const char **kernel_used, cudaStream_t tail_stream = nullptr);
cudaError_t launch_merkle_root_rfc6962(const uint8_t *d_leaves, uint64_t n, uint8_t *d_root, uint8_t *d_scratch_a,
                                       uint8_t *d_scratch_b, cudaStream_t stream, uint64_t *launches);

// selftest.cu --------------------------------------------------------------
// One warp waits (bounded by limit_cycles SM clocks) on a barrier nobody arrives at, then sets *d_status to
// IVK_DEV_TIMEOUT and returns; *d_waited (may be NULL) receives the clocks it waited.
cudaError_t launch_wait_timeout_selftest(uint64_t limit_cycles, uint32_t *d_status, unsigned long long *d_waited,
                                         cudaStream_t stream, uint64_t *launches);

// probe_alu.cu -------------------------------------------------------------
cudaError_t launch_probe(int kind, unsigned blocks, unsigned threads, uint32_t iters, uint32_t active_lanes,
                         unsigned long long *d_cycles, uint32_t *d_sink, cudaStream_t stream);
uint64_t probe_ops_per_thread(int kind, uint32_t iters);
bool probe_counts_blocks(int kind);   // the kind reports message bytes (one 64-byte block per trip), not instructions

}  // namespace ivk
