// Leaf hashing when chains are scarce (fewer chunks than the GPU has lanes to spare).
//
// A chunk is one serial compression chain, so with few chunks the time per 64-byte block of
// ONE chain bounds the whole job.  About 40 % of SHA-256's work -- the endian swap, the
// 48-step message schedule and the addition of the round constants -- does not depend on the
// chaining state.  Each CTA therefore runs two warps on two SM schedulers for its 32 chains:
//
//   producer warp: pulls the lanes' streams through a shared-memory ring with bulk copies
//                  (one per lane and segment), forms W[t] + K[t] for t = 0..63 of every block
//                  and writes them to a second ring, lane-interleaved;
//   consumer warp: runs only the 64 rounds, reading W[t] + K[t] with 128-bit shared loads.
//
// The two rings are handed over through mbarriers (full / empty per slot); all waits are bounded.
// The chain's critical path per block drops from the whole compression to the rounds alone.
#include <type_traits>

#include "iv_internal.h"
#include "rfc6962_dev.cuh"
#include "sha256_dev.cuh"
#include "tma_dev.cuh"
#include "sha256_split_dev.cuh"

namespace ivk {
namespace {

__device__ __forceinline__ uint64_t warp_max_u64(uint64_t v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const uint64_t t = __shfl_xor_sync(0xffffffffu, v, o);
        v = t > v ? t : v;
    }
    return v;
}

// RAGGED = false: message i is chunk i of the blob (base and chunk size multiples of 16 bytes).
// RAGGED = true:  message k of the CTA is tensor order[...] at data + offsets[.] with lengths[.] bytes,
//                 any alignment: each bulk copy starts at the 16-byte boundary below the tensor and
//                 carries 16 bytes more than a segment, so that every 64-byte block lies inside one
//                 stage.  A block is read as five aligned 16-byte pieces (conflict-free at this lane stride,
//                 whatever the tensors' alignment; 17 scalar loads at the same stride collided up to
//                 eight ways and cost the CHAIN up to 11 %, because the shared-memory pipe is the
//                 consumer's too); the 0..3 whole words between the 16-byte boundary and the message are
//                 skipped with two levels of selects, the last 0..3 bytes in the endian-swap PRMT.
// PAIR: blocks handed over per W+K slot; the barrier traffic per block falls with it.
// PREFIX (chunks only): message i is 0x00 || chunk i, the RFC 6962 leaf hash.
// MINB, NARROW: the second argument of __launch_bounds__ (0 = none) and 32-bit block counters in the
//                 consumer.  Neither changes what is computed; they change the code the compiler makes of
//                 the consumer's loop, which decides the chain's speed and came out 1,845 to 2,130 cycles
//                 per block over the combinations tried.  The launcher passes the best one measured for
//                 each mode (tensors: 1, true; chunks: 0, false).
template <int SEG, int STAGES, int NSLOT, bool RAGGED, int PAIR = 1, bool PREFIX = false, int MINB = 0, bool NARROW = false>
__global__ void __launch_bounds__(64, MINB)
hash_chunks_split_kernel(const uint8_t *__restrict__ data, uint64_t nbytes, uint64_t chunk_bytes,
                         uint64_t n_chunks, uint8_t *__restrict__ digests, uint32_t *__restrict__ status,
                         const uint32_t *__restrict__ one_ptr, const uint64_t *__restrict__ offsets,
                         const uint64_t *__restrict__ lengths, const uint32_t *__restrict__ order,
                         iv_sha_state *__restrict__ states, int finish) {
    constexpr uint32_t kLaneStride = SEG + 16;            // data ring: bytes per lane per stage (33 or 65 x 16: conflict-free)
    constexpr uint32_t kStageBytes = 32 * kLaneStride;
    constexpr int kBlocksPerSeg = SEG / 64;
    constexpr uint32_t kWkLane = 64 * 4 + 16;             // W+K ring: bytes per lane per slot
    constexpr uint32_t kWkBlock = 32 * kWkLane;           // one block's W+K for the 32 lanes
    constexpr uint32_t kWkSlot = PAIR * kWkBlock;
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ __align__(8) uint64_t bars[STAGES + 2 * NSLOT];

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    const uint32_t data_base = tma::smem_u32(smem) + lane * kLaneStride;
    const uint32_t wk_base = tma::smem_u32(smem) + STAGES * kStageBytes + lane * kWkLane;
    const uint32_t bar_data = tma::smem_u32(&bars[0]);
    const uint32_t bar_full = bar_data + 8 * STAGES;
    const uint32_t bar_empty = bar_full + 8 * NSLOT;
    if (threadIdx.x == 0) {
        // data stages: one arrival (lane 0 announces the bytes of all 32 copies); W+K slots: every lane of the
        // producer (full) or consumer (empty) arrives for itself, which needs no warp barrier and no one-lane branch
        for (int s = 0; s < STAGES; ++s) tma::mbar_init(bar_data + 8 * s, 1);
        for (int s = STAGES; s < STAGES + 2 * NSLOT; ++s) tma::mbar_init(bar_data + 8 * s, 32);
        tma::fence_barrier_init();
    }
    __syncthreads();
    // The multiplier 1 for additions issued as multiply-adds: read from memory, so that neither
    // compiler stage can fold the multiplication away.
    const uint32_t one = __ldg(one_ptr);

    const uint64_t slot_index = (uint64_t)blockIdx.x * 32 + lane;
    const bool valid = slot_index < n_chunks;
    uint64_t i = slot_index, begin = 0, len = 0;
    // Resumable hashing (tensors only): `states` carries each message's chaining value and the bytes
    // hashed so far from call to call; only the finishing call pads and writes digests.  A part that
    // does not finish its message must be a whole number of blocks (the remainder is not hashed and
    // the status word says so).
    uint64_t done_before = 0;
    const bool resumable = RAGGED && states != nullptr;
    const bool finishing = !resumable || finish != 0;
    if (RAGGED) {
        if (valid) {
            i = order ? order[slot_index] : slot_index;
            begin = offsets[i];
            len = lengths[i];
            if (resumable) {
                done_before = states[i].bytes;
                if (!finishing && (len & 63u)) {
                    if (warp == 0) atomicExch(status, (uint32_t)IVK_DEV_BOUNDS);
                    len &= ~63ull;
                }
            }
        }
    } else if (valid) {
        begin = i * chunk_bytes;
        len = (nbytes - begin < chunk_bytes) ? (nbytes - begin) : chunk_bytes;
    }
    // SHA-256 blocks of this lane's message, padding included.  For chunks lane 0 holds the longest
    // message of the warp; for tensors the maximum is taken.
    static_assert(!(PREFIX && RAGGED), "the prefixed leaf hash is for chunks");
    const uint64_t my_total = !valid ? 0 : (finishing ? ((len + (PREFIX ? 1 : 0) + 8) >> 6) + 1 : (len >> 6));
    const uint64_t warp_total = RAGGED ? warp_max_u64(my_total) : __shfl_sync(0xffffffffu, my_total, 0);

    if (NARROW && warp_total > 0xffffffffull) {       // a message of 2^32 blocks (256 GiB) does not fit the device's memory
        if (lane == 0) atomicExch(status, (uint32_t)IVK_DEV_BOUNDS);
        return;                                        // both warps leave: nobody waits for the other
    }

    if (warp == 1) {
        // ------------------------------------------------------------------ producer
        const uint8_t *p = data + begin;
        const uint64_t full_bytes = len & ~63ull;
        const uint64_t my_full = full_bytes >> 6;
        const uint64_t warp_full = RAGGED ? warp_max_u64(my_full) : __shfl_sync(0xffffffffu, my_full, 0);
        const uint64_t nseg = (warp_full * 64 + SEG - 1) / SEG;
        // tensors: misalignment of the message start, the 16-byte aligned copy source and how many
        // aligned bytes cover the whole blocks
        const uint32_t mis = RAGGED ? (uint32_t)(reinterpret_cast<uintptr_t>(p) & 15u) : 0u;
        const uint8_t *p_al = p - mis;
        const uint64_t need = full_bytes ? ((mis + full_bytes + 15) & ~15ull) : 0;
        const bool skip1 = (mis & 4u) != 0, skip2 = (mis & 8u) != 0;   // whole words between the 16-byte boundary and the message
        const uint32_t sel = 0x0123u + 0x1111u * (mis & 3u);       // PRMT: byte shift + big-endian
        // One arrival per stage: lane 0 announces the bytes of all 32 copies, every lane issues its own.
        auto issue = [&](uint64_t seg, int stage) {
            const uint64_t off = seg * SEG;
            const uint32_t bar = bar_data + 8 * stage;
            uint32_t bytes;
            if (RAGGED) bytes = off < need ? (uint32_t)((need - off < SEG + 16) ? (need - off) : SEG + 16) : 0u;
            else bytes = off < full_bytes ? (uint32_t)((full_bytes - off < SEG) ? (full_bytes - off) : SEG) : 0u;
            const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
            if (lane == 0) tma::mbar_arrive_expect_tx(bar, total);
            if (bytes) tma::bulk_g2s(data_base + stage * kStageBytes, p_al + off, bytes, bar);
        };
#pragma unroll
        for (int s = 0; s < STAGES; ++s)
            if ((uint64_t)s < nseg) issue(s, s);

        uint32_t w[16], raw[RAGGED ? 20 : 16], tw[32];
        uint32_t carry = 0u;                          // PREFIX: the data word before the block (byte 3 of 0 = the prefix)
        int stage = 0, in_stage = 0;
        uint32_t dparity = 0;
        bool failed = false, tail_built = false;
        auto fetch = [&](int blk_in_stage) {
            const uint32_t src = data_base + stage * kStageBytes + 64 * blk_in_stage;
#pragma unroll
            for (int q = 0; q < (RAGGED ? 5 : 4); ++q)
                tma::ld_shared_v4(src + 16 * q, raw[4 * q], raw[4 * q + 1], raw[4 * q + 2], raw[4 * q + 3]);
        };
        if (warp_full) {
            failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded(bar_data, 0));
            if (!failed) fetch(0);
        }
        uint64_t next_seg = STAGES;
        int slot = 0;
        uint32_t eparity = 1;                         // first pass over the slots finds them empty
        for (uint64_t blk = 0; blk < warp_total && !failed; ++blk) {
            if (blk < my_full) {
                if constexpr (PREFIX) {
                    w[0] = shifted_word(raw[0], carry);
#pragma unroll
                    for (int k = 1; k < 16; ++k) w[k] = shifted_word(raw[k], raw[k - 1]);
                    carry = raw[15];
                } else if constexpr (RAGGED) {
                    uint32_t a[19], b[17];
#pragma unroll
                    for (int k = 0; k < 19; ++k) a[k] = skip1 ? raw[k + 1] : raw[k];
#pragma unroll
                    for (int k = 0; k < 17; ++k) b[k] = skip2 ? a[k + 2] : a[k];
#pragma unroll
                    for (int k = 0; k < 16; ++k) w[k] = __byte_perm(b[k], b[k + 1], sel);
                } else {
#pragma unroll
                    for (int k = 0; k < 16; ++k) w[k] = bswap32(raw[k]);
                }
            } else if (blk < my_total) {
                if (!tail_built) {
                    if (PREFIX) (void)prefixed_tail(p, 0x00, full_bytes, len + 1, tw);
                    else (void)sha256_build_tail(p + full_bytes, (uint32_t)(len & 63u), done_before + len, tw);
                    tail_built = true;
                }
                const int t = (int)(blk - my_full);
#pragma unroll
                for (int k = 0; k < 16; ++k) w[k] = tw[16 * t + k];
            }
            if (blk + 1 < warp_full) {
                if (++in_stage == kBlocksPerSeg) {
                    in_stage = 0;
                    __syncwarp();
                    if (next_seg < nseg) issue(next_seg, stage);
                    ++next_seg;
                    if (++stage == STAGES) { stage = 0; dparity ^= 1u; }
                    failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded(bar_data + 8 * stage, dparity));
                    if (failed) break;
                }
                fetch(in_stage);
            }
            const uint32_t in_slot = (uint32_t)(blk % PAIR);
            if (in_slot == 0) {
                failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded(bar_empty + 8 * slot, eparity));
                if (failed) break;
            }
            produce_wk(w, wk_base + slot * kWkSlot + in_slot * kWkBlock, one);
            if (in_slot == PAIR - 1 || blk + 1 == warp_total) {
                tma::mbar_arrive(bar_full + 8 * slot);     // every lane arrives after its own stores (release)
                if (++slot == NSLOT) { slot = 0; eparity ^= 1u; }
            }
        }
        if (failed && lane == 0) atomicExch(status, (uint32_t)IVK_DEV_TIMEOUT);
        return;
    }

    // ---------------------------------------------------------------------- consumer
    uint32_t st[8], v[8];
    sha256_init(st);
    if (resumable && valid && done_before != 0) {
#pragma unroll
        for (int k = 0; k < 8; ++k) st[k] = states[i].h[k];
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = st[k];
    int slot = 0;
    uint32_t fparity = 0;
    bool failed = false;
    // block counters of the loop: 64 bits, or 32 where the launcher asks (counts beyond 32 bits were refused above)
    using Count = typename std::conditional<NARROW, uint32_t, uint64_t>::type;
    const Count loop_total = (Count)warp_total, lane_total = (Count)my_total;
    for (Count blk = 0; blk < loop_total; ++blk) {
        const uint32_t in_slot = (uint32_t)(blk % PAIR);
        if (in_slot == 0) {
            // every lane tests the same barrier word, so the outcome is uniform without a vote
            failed = !tma::mbar_wait_bounded(bar_full + 8 * slot, fparity);
            if (failed) break;
        }
        const uint32_t src = wk_base + slot * kWkSlot + in_slot * kWkBlock;
        const bool slot_done = in_slot == PAIR - 1 || blk + 1 == loop_total;
        rounds64(v, src, one);
        if (slot_done) tma::mbar_arrive(bar_empty + 8 * slot);   // every lane arrives once its own values are in registers
        // feed-forward; a lane whose message has ended keeps its state (multiplier 0 instead of 1)
        const uint32_t keep = (blk < lane_total) ? one : 0u;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            st[k] = padd<true>(v[k], st[k], keep);     // v * keep + st
            v[k] = st[k];
        }
        if (slot_done && ++slot == NSLOT) { slot = 0; fparity ^= 1u; }
    }
    if (failed) {
        if (lane == 0) atomicExch(status, (uint32_t)IVK_DEV_TIMEOUT);
        return;
    }
    if (valid && resumable) {
#pragma unroll
        for (int k = 0; k < 8; ++k) states[i].h[k] = st[k];
        states[i].bytes = done_before + len;
    }
    if (valid && finishing) store_digest(digests + 32 * i, st);
}

}  // namespace

namespace {

// Two instances per mode.  Up to one group per SM a CTA may use most of an SM's shared memory: two W+K slots of
// EIGHT blocks each (190 KB; a hand-over every eighth block): 1,860 cycles per block for chunks (three slots of four:
// 1,873, two of four: 1,890, four of four: 1,878).  Up to two groups per SM two CTAs share an SM: three slots of two
// blocks (104 KB): 1,914 cycles per block.  (Fetching the next block's first
// W+K values during the last rounds of the current one, within a slot, was measured and does not pay: 1,890.)
// The 32 bulk copies of a stage leave the producer one after the other and cost it about 2,000 cycles per stage.
// With chunks the consumer is the slower warp either way; with tensors the producer has the selects on top and
// was the slower one (1,970 cycles per block alone against 1,920 for the consumer), so where the CTA has an SM to
// itself its stages are twice as long (two of 1,024 bytes per lane: 1,830 alone).
template <bool RAGGED, bool PREFIX, int PAIR>
cudaError_t launch_split_instance(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n, uint8_t *d_digests,
                                  uint32_t *d_status, const uint32_t *d_one, const uint64_t *d_offsets, const uint64_t *d_lengths,
                                  const uint32_t *d_order, iv_sha_state *d_states, int finish, cudaStream_t stream) {
    constexpr bool ROOMY = PAIR == 8, LONG_STAGES = RAGGED && ROOMY;
    constexpr int SEG = LONG_STAGES ? 1024 : 512, STAGES = LONG_STAGES ? 2 : 3, NSLOT = ROOMY ? 2 : 3;
    constexpr size_t smem = (size_t)STAGES * 32 * (SEG + 16) + (size_t)NSLOT * PAIR * 32 * (64 * 4 + 16);
    auto kernel = hash_chunks_split_kernel<SEG, STAGES, NSLOT, RAGGED, PAIR, PREFIX, RAGGED ? 1 : 0, RAGGED>;
    static bool configured[kMaxDevices] = {};
    if (cudaError_t e0 = ensure_dynamic_smem(kernel, smem, configured); e0 != cudaSuccess) return e0;
    const uint64_t blocks = (n + 31) / 32;
    if (blocks > 0x7fffffffull) return cudaErrorInvalidConfiguration;
    kernel<<<(unsigned)blocks, 64, smem, stream>>>(d_data, nbytes, chunk_bytes, n, d_digests, d_status, d_one, d_offsets,
                                                   d_lengths, d_order, d_states, finish);
    return cudaGetLastError();
}

int sm_count_of_current_device() {
    static int cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    if (!cached[dev]) cudaDeviceGetAttribute(&cached[dev], cudaDevAttrMultiProcessorCount, dev);
    return cached[dev];
}

}  // namespace

cudaError_t launch_hash_chunks_split(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                                     uint64_t n_chunks, uint8_t *d_digests, uint32_t *d_status,
                                     const uint32_t *d_one, cudaStream_t stream, bool zero_prefix) {
    // 512-byte segments, three data stages; the additions that close the two state recurrences stay three-input
    // ALU adds, the others go to the FMA pipe (the fastest placement measured).
    const bool roomy = (n_chunks + 31) / 32 <= (uint64_t)sm_count_of_current_device();
    if (zero_prefix)
        return roomy ? launch_split_instance<false, true, 8>(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, d_one,
                                                             nullptr, nullptr, nullptr, nullptr, 1, stream)
                     : launch_split_instance<false, true, 2>(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, d_one,
                                                             nullptr, nullptr, nullptr, nullptr, 1, stream);
    return roomy ? launch_split_instance<false, false, 8>(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, d_one,
                                                          nullptr, nullptr, nullptr, nullptr, 1, stream)
                 : launch_split_instance<false, false, 2>(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, d_one,
                                                          nullptr, nullptr, nullptr, nullptr, 1, stream);
}

cudaError_t launch_hash_ragged_split(const uint8_t *d_base, const uint64_t *d_offsets, const uint64_t *d_lengths,
                                     const uint32_t *d_order, uint64_t n, uint8_t *d_digests, uint32_t *d_status,
                                     const uint32_t *d_one, iv_sha_state *d_states, int finish, cudaStream_t stream) {
    const bool roomy = (n + 31) / 32 <= (uint64_t)sm_count_of_current_device();
    return roomy ? launch_split_instance<true, false, 8>(d_base, 0, 0, n, d_digests, d_status, d_one, d_offsets, d_lengths,
                                                         d_order, d_states, finish, stream)
                 : launch_split_instance<true, false, 2>(d_base, 0, 0, n, d_digests, d_status, d_one, d_offsets, d_lengths,
                                                         d_order, d_states, finish, stream);
}

}  // namespace ivk
