/*
 * iv.h -- C ABI of libiv: GPU-resident integrity verification of model-weight
 * bytes on NVIDIA B200 (sm_100a).
 *
 * The library computes, entirely in CUDA kernels, the data-parallel path of the
 * paper "Scalable GPU-Based Integrity Verification for Large Machine Learning
 * Models": FIPS 180-4 SHA-256 digests of fixed-size chunks of a byte blob, a
 * binary Merkle reduction of those digests to a root, and the comparison of
 * digests and root with an expected manifest (Algorithm 1, "Streaming Model
 * Verification", and the section "Memory Scalability Considerations").
 *
 * Conventions
 *  - Pointers named d_* are DEVICE pointers owned by the caller; the library
 *    neither frees nor keeps them beyond the work it enqueues.  Pointers named
 *    h_* are HOST pointers.  Everything else is passed by value.
 *  - A digest is 32 bytes: the eight 32-bit words H0..H7 of FIPS 180-4
 *    section 6.2.2, each stored big-endian.  Digest arrays are contiguous
 *    records in index order.
 *  - Every call enqueues its GPU work on `cuda_stream` (a cudaStream_t passed
 *    as void*, NULL = the legacy default stream) and returns without waiting,
 *    except where stated.  Results in device memory are valid once the stream
 *    has reached that point.
 *  - Return value: IV_OK (0) or a negative iv_status.  Finding a mismatch is
 *    NOT an error: verification calls return IV_OK and report it in the result.
 *  - There is no CPU fallback: without a usable CUDA device iv_create fails.
 *  - A context may be used by one host thread at a time.  Calls on the same
 *    context that overlap on the GPU (different streams) share its scratch
 *    memory and therefore race; serialise them or use one context per stream.
 */
#ifndef IV_H
#define IV_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum iv_status {
    IV_OK = 0,
    IV_ERR_INVALID_ARG = -1, /* null pointer, zero chunk size, capacity too small, inconsistent manifest */
    IV_ERR_NOMEM = -2,       /* a device or host allocation for scratch failed */
    IV_ERR_CUDA = -3,        /* a CUDA runtime call failed; see iv_last_cuda_error */
    IV_ERR_NO_DEVICE = -4,   /* no CUDA device, or not a compute-capability-10.x device */
    IV_ERR_TOO_LARGE = -5    /* the size exceeds a fixed limit of the entry point (iv_merkle_root_noalloc) */
} iv_status;

/* Opaque context.  Owns scratch memory (Merkle level buffers, tickets, the
 * digest array used by verification, streaming windows), sized lazily. */
typedef struct iv_ctx iv_ctx;

/* Creates a context on CUDA device `cuda_device`.  Synchronous.  *out is set
 * to NULL on failure. */
int iv_create(iv_ctx **out, int cuda_device);

/* Waits for the device, frees all scratch, destroys the context.  NULL is allowed. */
int iv_destroy(iv_ctx *ctx);

/* Static, human-readable text for a status code. */
const char *iv_strerror(int code);

/* The cudaError_t (as int) of the last failed CUDA call on this context, 0 if none. */
int iv_last_cuda_error(const iv_ctx *ctx);

/* Device-side status of the kernels this context has run: 0 = all completed,
 * 1 = a kernel gave up on a bounded wait for a bulk copy (its outputs are then
 * invalid), 2 = an index check failed.  Waits for the device (synchronous),
 * writes the word to *h_status and clears it.  Verification calls also copy it
 * into iv_verify_result::status. */
int iv_device_status(iv_ctx *ctx, uint32_t *h_status);

/* Number of kernels this context has launched so far (a host-side counter). */
uint64_t iv_kernel_launches(const iv_ctx *ctx);

/* Name of the leaf-hashing kernel the last hashing or verification call on this context launched
 * (the library picks one of several by chain count, chunk size and alignment); "" before any call.
 * Static text, never freed. */
const char *iv_last_leaf_kernel(const iv_ctx *ctx);

/* Where that kernel has several launch shapes (the many-chain kernel: workers per SM; the SHA-384/512
 * two-warp kernel: pairs per SM), the one the last call ran in; "" otherwise.  Static text. */
const char *iv_last_leaf_instance(const iv_ctx *ctx);

/* Self-test of the bounded waits (a diagnostic; the paper has no counterpart).  Every wait inside the
 * library's kernels -- for a bulk copy, for a hand-over between warps -- gives up after a fixed number of
 * SM clocks (about two seconds), sets the device status to 1 and lets the kernel return, so that a lost
 * copy can never hang the GPU.  This call runs that path on purpose: one warp waits, with the same wait
 * routine and a limit of limit_cycles SM clocks (1 .. 4e9), on a barrier that nobody arrives at, gives
 * up, sets the status word and returns.  Afterwards iv_device_status reports 1 (and clears it), and the
 * context works as before.
 *   h_waited_cycles   optional host pointer; when given, the call waits for the stream and stores the
 *                     SM clocks the warp spent waiting (>= limit_cycles) */
int iv_selftest_wait_timeout(iv_ctx *ctx, uint64_t limit_cycles, uint64_t *h_waited_cycles, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Leaf hashing -- Algorithm 1, "chunk_count <- ceil(|M| / C)" and
 * "H_i = GPU_HASH(M_i)" with GPU_HASH = SHA-256 (FIPS 180-4 section 6.2).
 *
 *   d_data        nbytes bytes of device memory, any alignment
 *   chunk_bytes   C > 0; chunk i covers bytes [i*C, min((i+1)*C, nbytes)); the
 *                 last chunk is hashed at its true length (no zero fill)
 *   d_digests     receives n = ceil(nbytes / C) records of 32 bytes
 *   digests_cap   capacity of d_digests in records; n > digests_cap is an error
 *   h_n_chunks    optional host pointer, receives n (written before returning)
 *
 * nbytes == 0 gives n == 0 and launches nothing.  Streaming (the loop of
 * Algorithm 1) needs no other entry point: call once per resident window,
 * each window a multiple of C except the last, with d_digests advanced by
 * 32 * (chunks before the window).
 */
int iv_hash_chunks(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                   uint8_t *d_digests, uint64_t digests_cap, uint64_t *h_n_chunks,
                   void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Merkle reduction -- Algorithm 1, "Construct Merkle tree from leaf_hashes
 * using GPU".  Binary tree over n_leaves digests in index order; a parent is
 * SHA-256(left || right) of exactly 64 bytes (no domain-separation prefix); an
 * unpaired last node of a level moves up unchanged; one leaf is its own root;
 * zero leaves give SHA-256 of the empty string.
 *
 *   d_leaves   n_leaves * 32 bytes (may be NULL when n_leaves == 0)
 *   d_root     receives 32 bytes
 */
int iv_merkle_root(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root,
                   void *cuda_stream);

/* `levels` levels of the same reduction without going all the way to the root:
 * d_nodes[n] -> d_out[n_out], n_out = n halved (rounding up) `levels` times.  Node j
 * of the result is the root of the aligned run of 2^levels inputs starting at
 * j * 2^levels, which is also a node of the whole tree -- the building block for
 * the paper's multi-GPU scheme (section "Multi-GPU Deployment Architectures",
 * a global tree built from the hashes computed on each device): every GPU
 * reduces its aligned range of leaves to such nodes, the nodes are gathered, and
 * iv_merkle_root over them gives the global root.
 *   d_out, out_cap   receives n_out records; out_cap (in records) must be >= n_out;
 *                    must not overlap d_nodes
 *   h_n_out          optional host pointer, receives n_out
 */
int iv_merkle_levels(iv_ctx *ctx, const uint8_t *d_nodes, uint64_t n, uint32_t levels,
                     uint8_t *d_out, uint64_t out_cap, uint64_t *h_n_out, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Incremental re-verification -- the paper's hierarchical / differential
 * verification (section "Version Management and Incremental Verification": when fine-tuning
 * or an update touches some chunks, only those leaves and their paths to the
 * root are recomputed).
 *
 * A retained tree holds every level of the tree over n leaves in one device
 * array of iv_tree_records(n) records of 32 bytes: the n leaves first, then
 * ceil(n/2) parents, and so on; the LAST record is the root (for n == 0 the
 * single record is SHA-256 of the empty string).  d_tree must be 16-byte aligned.
 *
 * iv_tree_build   fills the array from n leaf digests (d_leaves 16-byte aligned).
 * iv_tree_update  re-hashes the chunks listed in d_dirty (n_dirty uint64 chunk
 *                 indices in DEVICE memory, any order, repeats allowed, each
 *                 < ceil(nbytes / chunk_bytes)) from the current bytes of d_data,
 *                 stores their digests in the leaf level and recomputes only the
 *                 ancestors of those leaves.  Work is n_dirty chunk hashes plus
 *                 n_dirty * ceil(log2 n) node hashes.  An index outside the tree
 *                 is skipped and sets the device status to 2 (iv_device_status).
 */
uint64_t iv_tree_records(uint64_t n_leaves);
int iv_tree_build(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_tree,
                  uint64_t tree_cap, void *cuda_stream);
int iv_tree_update(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                   const uint64_t *d_dirty, uint64_t n_dirty, uint8_t *d_tree, uint64_t tree_cap,
                   void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Verification -- Algorithm 1, "Compare root hash with expected value", plus
 * the per-chunk comparison that locates the damage.
 *
 * The manifest is the publisher's expected value: the blob's size, the chunk
 * size, the chunk digests and their Merkle root.
 */
typedef struct iv_manifest {
    uint64_t total_bytes;     /* must equal nbytes of the call */
    uint64_t chunk_bytes;     /* C */
    uint64_t n_chunks;        /* must equal ceil(total_bytes / chunk_bytes) */
    const uint8_t *d_digests; /* DEVICE: n_chunks * 32 bytes (may be NULL when n_chunks == 0) */
    uint8_t root[32];         /* expected Merkle root (host bytes inside this struct) */
} iv_manifest;

/* Written by the GPU into DEVICE memory supplied by the caller. */
typedef struct iv_verify_result {
    uint32_t status;     /* device-side status: 0 = completed */
    uint32_t root_ok;    /* 1 iff the recomputed root equals manifest root */
    uint64_t n_mismatch; /* exact number of chunks whose digest differs, even if > idx_cap */
    uint8_t root[32];    /* the recomputed root */
} iv_verify_result;

/*   d_data, nbytes    the blob to verify (device)
 *   h_manifest        host struct (read before returning), digests on the device
 *   d_result          device memory for one iv_verify_result
 *   d_mismatch_idx    device array of idx_cap uint64: the indices of mismatching
 *                     chunks in ASCENDING order, the first min(n_mismatch, idx_cap)
 *                     of them; may be NULL when idx_cap == 0
 * The recomputed chunk digests stay in the context (iv_ctx_digests). */
int iv_verify_manifest(iv_ctx *ctx, const void *d_data, uint64_t nbytes,
                       const iv_manifest *h_manifest, iv_verify_result *d_result,
                       uint64_t *d_mismatch_idx, uint64_t idx_cap, void *cuda_stream);

/* Batch verification -- the paper's batch processing (section "Scalability Analysis"): n_blobs blobs of
 * the same size (copies, replicas, variants that share a manifest) are verified against ONE manifest in
 * one pass; all their chunks are independent chains of a single hashing launch, which is what fills the
 * GPU when one blob alone has few chunks.
 *   h_d_blobs        HOST array of n_blobs DEVICE pointers (read before returning), at most 64
 *   d_results        DEVICE array of n_blobs iv_verify_result, one per blob
 *   d_mismatch_idx   DEVICE array of n_blobs * idx_cap uint64: blob b's ascending list starts at b * idx_cap
 * Everything else as for iv_verify_manifest. */
int iv_verify_manifest_batch(iv_ctx *ctx, const void *const *h_d_blobs, uint64_t n_blobs, uint64_t nbytes,
                             const iv_manifest *h_manifest, iv_verify_result *d_results,
                             uint64_t *d_mismatch_idx, uint64_t idx_cap, void *cuda_stream);

/* Device pointer of the digest array the last iv_verify_manifest /
 * iv_verify_streamed on this context wrote (n_chunks * 32 bytes), NULL if none. */
const uint8_t *iv_ctx_digests(const iv_ctx *ctx);

/* ---------------------------------------------------------------------------
 * Two-level leaves -- a SEPARATELY NAMED mode whose digests differ from
 * iv_hash_chunks (the paper's hierarchical verification at several
 * granularities).  The digest of chunk i is the Merkle root (this library's tree
 * rule) over the SHA-256 digests of its sub_bytes-sized pieces:
 *     D_i = root( SHA-256(piece_0), SHA-256(piece_1), ... )   pieces of chunk i.
 * A chunk is then no longer one serial SHA-256 chain but chunk_bytes/sub_bytes
 * independent ones, which is what fills a GPU when a blob has few large chunks.
 * chunk_bytes must be sub_bytes times a power of two (else IV_ERR_INVALID_ARG);
 * with that, the root over the D_i equals the root over all pieces' digests, so
 * a manifest at chunk granularity and one at piece granularity share one root.
 * sub_bytes == chunk_bytes gives iv_hash_chunks / iv_verify_manifest exactly.
 * Other arguments as for iv_hash_chunks / iv_verify_manifest; the manifest's
 * digests and root must have been made in the same mode.
 */
int iv_hash_chunks_two_level(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                             uint64_t sub_bytes, uint8_t *d_digests, uint64_t digests_cap,
                             uint64_t *h_n_chunks, void *cuda_stream);
int iv_verify_manifest_two_level(iv_ctx *ctx, const void *d_data, uint64_t nbytes,
                                 const iv_manifest *h_manifest, uint64_t sub_bytes,
                                 iv_verify_result *d_result, uint64_t *d_mismatch_idx,
                                 uint64_t idx_cap, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Streamed verification -- the whole of Algorithm 1 for a blob that lives in
 * HOST memory ("Load model chunk M_i into GPU memory ... Free GPU memory"):
 * the blob is copied window by window into two device windows owned by the
 * context, the copy of window w+1 overlapping the hashing of window w on a
 * second stream, then the tree is built and compared as in iv_verify_manifest.
 * A window with few large chunks is copied and hashed in column parts (part s of
 * every chunk while part s+1 is in flight), so that its hashing ends shortly
 * after its last byte arrives; the results are the same.
 *
 *   h_windows      host array of n_windows HOST pointers; window w holds bytes
 *                  [w*window_bytes, min((w+1)*window_bytes, nbytes)) of the blob.
 *                  The windows need not be adjacent in memory (file shards,
 *                  mapped pieces) and may repeat.  Page-locked memory is needed
 *                  for the copies to overlap (pageable memory works, slowly).
 *   n_windows      must equal ceil(nbytes / window_bytes)
 *   window_bytes   > 0, a multiple of h_manifest->chunk_bytes
 * The pointer array is read before the call returns; the window contents must
 * stay valid until the enqueued copies have run.  The call returns when all
 * work is ENQUEUED on cuda_stream and the context's copy stream; cuda_stream
 * reaches completion only after both are done.
 */
int iv_verify_streamed(iv_ctx *ctx, const void *const *h_windows, uint64_t n_windows,
                       uint64_t window_bytes, uint64_t nbytes, const iv_manifest *h_manifest,
                       iv_verify_result *d_result, uint64_t *d_mismatch_idx, uint64_t idx_cap,
                       void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Phase timing (the paper's result record carries a verification time).  When
 * switched on, iv_verify_manifest and iv_verify_streamed bracket their three
 * phases -- leaf hashing, tree reduction, comparison -- with CUDA events on
 * cuda_stream.  The context keeps the events of the most recent
 * IV_TIMING_RING verification calls.  Independently of this switch the three
 * phases are NVTX ranges ("iv: leaf hashing", "iv: Merkle reduction",
 * "iv: manifest compare") around the launches of each phase, for profilers.
 *
 * iv_phase_times waits for the events of the call made `calls_back` calls ago
 * (0 = the most recent) and writes the three durations in milliseconds to
 * h_ms[0..2].  Returns IV_ERR_INVALID_ARG if timing was off for that call or
 * calls_back >= IV_TIMING_RING.
 */
#define IV_TIMING_RING 64
int iv_set_timing(iv_ctx *ctx, int enabled);
int iv_phase_times(iv_ctx *ctx, uint32_t calls_back, float *h_ms);

/* ---------------------------------------------------------------------------
 * Per-tensor digests -- the paper's batch verification (section "Scalability
 * Analysis": many payloads per launch, one digest per payload): digest k =
 * SHA-256(d_base[offset_k .. offset_k + length_k)).
 *
 *   d_offsets, d_lengths   n uint64 each, DEVICE memory; any byte alignment of
 *                          offsets, any length including 0
 *   d_digests              receives n * 32 bytes
 * The caller guarantees that every range lies inside the d_base allocation.
 */
int iv_hash_ragged(iv_ctx *ctx, const void *d_base, const uint64_t *d_offsets,
                   const uint64_t *d_lengths, uint64_t n, uint8_t *d_digests,
                   void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Resumable per-tensor digests -- the paper's multi-pass processing (section
 * "Memory Scalability Considerations", the hash state carried from pass to pass): a tensor
 * that is larger than a resident window, or that spans two windows, is hashed
 * part by part.
 *
 * d_states holds one iv_sha_state per tensor in DEVICE memory, zero-filled by
 * the caller before a tensor's first part.  Each call hashes, for every k, the
 * next length_k bytes of tensor k found at d_base + offset_k and advances state
 * k.  With finish == 0 every length must be a multiple of 64 bytes (a remainder
 * is left unhashed and the device status is set to 2); the call with finish != 0
 * takes the last part (any length, 0 allowed), applies the padding for the
 * TOTAL length and writes digest k to d_digests + 32 k (d_digests may be NULL
 * when finish == 0).  At most 32,768 tensors per call (IV_ERR_TOO_LARGE beyond).
 */
typedef struct iv_sha_state {
    uint32_t h[8];     /* chaining value after the bytes hashed so far */
    uint64_t bytes;    /* bytes hashed so far (0 = fresh) */
    uint64_t reserved; /* keeps the record at 48 bytes */
} iv_sha_state;

int iv_hash_ragged_update(iv_ctx *ctx, const void *d_base, const uint64_t *d_offsets,
                          const uint64_t *d_lengths, uint64_t n, iv_sha_state *d_states,
                          int finish, uint8_t *d_digests, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * SHA-384 and SHA-512 variants -- SHA-384 is the digest of the paper's own kernel
 * listings (FIPS 180-4 section 6.5).  Chunking and tree rule as above with 48-byte records: digest i
 * = SHA-384(chunk i); parent = SHA-384(left || right) over exactly 96 bytes, an
 * unpaired last node moves up unchanged, one leaf is its own root, zero leaves
 * give SHA-384 of the empty string.  The SHA-512 entry points (FIPS 180-4 section
 * 6.4, initial value of section 5.3.5, no truncation) are the same with 64-byte
 * records and SHA-512(left || right) over exactly 128 bytes as the parent.
 * 16-byte aligned blobs with up to about 131,000 chunks of 16 KiB or more (a
 * multiple of 16 bytes) run through a kernel in the design of the SHA-256 path
 * (tiled bulk copies, the compression split between two warps, chains migrating
 * between workers); other shapes through a plain one-chain-per-lane kernel,
 * which is the faster one when chains are plentiful.
 */
int iv_hash_chunks_sha384(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                          uint8_t *d_digests, uint64_t digests_cap, uint64_t *h_n_chunks,
                          void *cuda_stream);
int iv_merkle_root_sha384(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root,
                          void *cuda_stream);

int iv_hash_chunks_sha512(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                          uint8_t *d_digests, uint64_t digests_cap, uint64_t *h_n_chunks,
                          void *cuda_stream);
int iv_merkle_root_sha512(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root,
                          void *cuda_stream);

/* iv_verify_manifest for the SHA-384 variant: the same steps over 48-byte records.  The manifest holds the
 * SHA-384 chunk digests (device) and the root of the SHA-384 tree; fields, index list, errors and
 * asynchrony as for iv_manifest / iv_verify_result / iv_verify_manifest. */
typedef struct iv_manifest_sha384 {
    uint64_t total_bytes;
    uint64_t chunk_bytes;
    uint64_t n_chunks;
    const uint8_t *d_digests; /* DEVICE: n_chunks * 48 bytes */
    uint8_t root[48];
} iv_manifest_sha384;
typedef struct iv_verify_result_sha384 {
    uint32_t status;
    uint32_t root_ok;
    uint64_t n_mismatch;
    uint8_t root[48];
} iv_verify_result_sha384;
int iv_verify_manifest_sha384(iv_ctx *ctx, const void *d_data, uint64_t nbytes,
                              const iv_manifest_sha384 *h_manifest, iv_verify_result_sha384 *d_result,
                              uint64_t *d_mismatch_idx, uint64_t idx_cap, void *cuda_stream);

/* The same for SHA-512: 64-byte records. */
typedef struct iv_manifest_sha512 {
    uint64_t total_bytes;
    uint64_t chunk_bytes;
    uint64_t n_chunks;
    const uint8_t *d_digests; /* DEVICE: n_chunks * 64 bytes */
    uint8_t root[64];
} iv_manifest_sha512;
typedef struct iv_verify_result_sha512 {
    uint32_t status;
    uint32_t root_ok;
    uint64_t n_mismatch;
    uint8_t root[64];
} iv_verify_result_sha512;
int iv_verify_manifest_sha512(iv_ctx *ctx, const void *d_data, uint64_t nbytes,
                              const iv_manifest_sha512 *h_manifest, iv_verify_result_sha512 *d_result,
                              uint64_t *d_mismatch_idx, uint64_t idx_cap, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * RFC 6962 section 2.1 mode -- the Merkle Tree Hash the paper cites for its tree,
 * with that RFC's domain separation, over SHA-256 with the chunks as entries:
 * leaf hash i = SHA-256(0x00 || chunk i); node = SHA-256(0x01 || left || right)
 * (65 bytes); the list is split at the largest power of two below n, one entry
 * is its own leaf hash, no entry gives SHA-256 of the empty string.  Digests
 * and root differ from the default (unprefixed) path by construction.
 * Arguments, layout and errors as iv_hash_chunks / iv_merkle_root.
 */
int iv_hash_chunks_rfc6962(iv_ctx *ctx, const void *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                           uint8_t *d_digests, uint64_t digests_cap, uint64_t *h_n_chunks,
                           void *cuda_stream);
int iv_merkle_root_rfc6962(iv_ctx *ctx, const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root,
                           void *cuda_stream);
/* iv_verify_manifest in this mode: the manifest holds the prefixed leaf hashes and the root of the
 * prefixed tree; result record, index list, errors and asynchrony as iv_verify_manifest. */
int iv_verify_manifest_rfc6962(iv_ctx *ctx, const void *d_data, uint64_t nbytes,
                               const iv_manifest *h_manifest, iv_verify_result *d_result,
                               uint64_t *d_mismatch_idx, uint64_t idx_cap, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Merkle root without allocation (the paper has no counterpart; this exists
 * for callers of this library, see below).
 *
 * Same result as iv_merkle_root, for callers that cannot allocate device
 * memory: code running inside a framework whose memory pool already owns the
 * whole GPU, a serving loop that must never block on the allocator, a process
 * that may only use buffers handed to it.  It needs no iv_ctx (creating one
 * allocates) and calls no cudaMalloc, cudaFree or other allocating routine.
 * Its scratch -- 512 intermediate digests and a ticket word -- lives in a
 * fixed 16.25 KiB array inside the library image, which every GPU that loads
 * the library holds until the process exits.
 *
 *   d_leaves, d_root   as for iv_merkle_root; the caller supplies both
 *   n_leaves           at most IV_NOALLOC_MAX_LEAVES (512 * 512); more returns
 *                      IV_ERR_TOO_LARGE and launches nothing
 * Work is enqueued on cuda_stream for the CURRENT device.  The first call on
 * a device looks up the device address of the array (once per device); make
 * that first call before starting any stream capture.  All calls share the
 * one array, which keeps the previous call's contents (the entry point clears
 * the one word that must start at zero): calls that overlap on the GPU --
 * two streams, two threads -- race and give wrong roots; serialise them.
 */
#define IV_NOALLOC_MAX_LEAVES (512ull * 512ull)
int iv_merkle_root_noalloc(const uint8_t *d_leaves, uint64_t n_leaves, uint8_t *d_root,
                           void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Roofline probe (a measurement aid; the paper has no counterpart).  Runs a
 * register-only microbenchmark on every SM and reports, from the SM cycle
 * counter, how many lane-operations of one instruction kind an SM retires per
 * clock -- the denominator of the integer roofline -- or, for the kinds that run
 * SHA-256 (6, 7, 13, 14), how many message bytes per clock per SM that part of the
 * compression function alone sustains.  Synchronous; allocates and frees a few KB of device memory.
 *
 *   warps_per_block, blocks_per_sm   launch shape (blocks = blocks_per_sm * SM count)
 *   active_lanes                     1..32 lanes of each warp that do work
 *   iters                            loop trips (128 operations each; one 64-byte block
 *                                    each for the SHA-256 kinds)
 *   h_out[0]                         lane-ops (or bytes) per clock per SM
 *   h_out[1]                         mean cycles per block
 */
typedef enum iv_probe_kind {
    IV_PROBE_IADD3 = 0,  /* three-input integer add */
    IV_PROBE_LOP3 = 1,   /* three-input logic op */
    IV_PROBE_SHF = 2,    /* funnel shift (rotate) */
    IV_PROBE_PRMT = 3,   /* byte permute */
    IV_PROBE_IMAD = 4,   /* integer multiply-add */
    IV_PROBE_MIXED = 5,  /* LOP3 and IMAD interleaved 1:1 */
    IV_PROBE_SHA256 = 6,     /* full SHA-256 compressions, registers only */
    IV_PROBE_SHA256_SCHED_FMA = 7, /* the same with the message schedule's additions as multiply-adds (FMA pipe) */
    IV_PROBE_LAT_IADD3 = 8,  /* kinds 8..11: ONE dependent chain per thread; with one warp per SM,   */
    IV_PROBE_LAT_LOP3 = 9,   /* 32 / h_out[0] is the dependent-issue latency of the instruction in   */
    IV_PROBE_LAT_SHF = 10,   /* clocks                                                               */
    IV_PROBE_LAT_IMAD = 11,
    IV_PROBE_LAT_CROSS = 12, /* one chain alternating LOP3 (ALU pipe) and IMAD (FMA pipe) */
    IV_PROBE_ROUNDS = 13,    /* the 64 rounds alone, W + K from shared memory: the consumer half of the two-warp kernel */
    IV_PROBE_SCHEDULE = 14   /* the message schedule + round constants alone: its producer half */
} iv_probe_kind;
int iv_probe_alu(iv_ctx *ctx, int kind, uint32_t warps_per_block, uint32_t blocks_per_sm,
                 uint32_t active_lanes, uint32_t iters, double *h_out);

#ifdef __cplusplus
}
#endif
#endif /* IV_H */
