// Leaf hashing between "few" and "many" chains: more groups of 32 chains than there are pairs of SM
// schedulers (2 x SMs), fewer than about three per SM.
//
// With G groups of 32 chains in that range neither of the other two kernels fits.  The two-warp kernel
// (one producer and one consumer warp per group, each on a scheduler of its own: 1,965 cycles per block
// and chain) has room for 2 x SMs groups at a time, so G groups would run in two waves.  The migrating
// kernel gives every group one whole-compression warp (3,000 cycles per block) and leaves the other
// schedulers idle.  Here the 2 x SMs producer/consumer pairs are persistent workers that take (group,
// slice) tasks from the same FIFO the migrating kernel uses: a group's chaining values are parked in
// global memory between slices, so the groups take turns on the pairs and all of them advance at
// 2 x SMs / G of the two-warp rate -- more than one warp each could give them as long as G < 3.05 x SMs.
//
// Both warps of a pair work on the same task.  The producer, which runs up to six blocks ahead of the
// consumer, takes the tickets: while the consumer finishes a slice the producer already waits for the next
// group, starts its copies and forms its first blocks; it hands the task to the consumer through a small ring
// in shared memory (one mbarrier per entry).  The data ring, the W+K ring and their barrier phases carry over
// from task to task (every task drains what it requested).  All waits are bounded.
#include "iv_internal.h"
#include "rfc6962_dev.cuh"
#include "sha256_dev.cuh"
#include "sha256_split_dev.cuh"
#include "slice_queue_dev.cuh"
#include "tma_dev.cuh"

namespace ivk {
namespace {

constexpr unsigned long long kTaskDone = ~0ull, kTaskFailed = ~0ull - 1;

// PREFIX: every chunk is hashed as 0x00 || chunk (the RFC 6962 leaf hash), as in the migrating kernel.
template <int SEG, int STAGES, int NSLOT, int PAIR, bool PREFIX>
__global__ void __launch_bounds__(64, 1)   // the stated minimum of one CTA per SM changes only the compiler's code: 592 against 585 GB/s
hash_chunks_pairs_kernel(const uint8_t *__restrict__ data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                         uint8_t *__restrict__ digests, uint32_t *__restrict__ status, uint64_t slice_bytes,
                         uint64_t total_tasks, uint32_t *__restrict__ slot, SliceQueue *__restrict__ q,
                         uint32_t *__restrict__ next_slice, uint32_t *__restrict__ mid /* [groups][8][32] */,
                         const uint32_t *__restrict__ one_ptr) {
    constexpr uint32_t kLaneStride = SEG + 16;            // data ring: bytes per lane per stage
    constexpr uint32_t kStageBytes = 32 * kLaneStride;
    constexpr int kBlocksPerSeg = SEG / 64;
    constexpr uint32_t kWkLane = 64 * 4 + 16;             // W+K ring: bytes per lane per block
    constexpr uint32_t kWkBlock = 32 * kWkLane;
    constexpr uint32_t kWkSlot = PAIR * kWkBlock;
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ __align__(8) uint64_t bars[STAGES + 2 * NSLOT];
    constexpr int kTaskRing = 8;                          // more than the producer's largest lead in blocks
    static_assert(NSLOT * PAIR < kTaskRing, "a task has at least one block");
    __shared__ unsigned long long s_task[kTaskRing];
    __shared__ __align__(8) uint64_t task_bars[kTaskRing];
    __shared__ uint32_t s_failed;

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;    // warp 0 consumer, warp 1 producer
    const uint32_t data_base = tma::smem_u32(smem) + lane * kLaneStride;
    const uint32_t wk_base = tma::smem_u32(smem) + STAGES * kStageBytes + lane * kWkLane;
    const uint32_t bar_data = tma::smem_u32(&bars[0]);
    const uint32_t bar_full = bar_data + 8 * STAGES;
    const uint32_t bar_empty = bar_full + 8 * NSLOT;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES + 2 * NSLOT; ++s) tma::mbar_init(bar_data + 8 * s, 1);
        for (int s = 0; s < kTaskRing; ++s) tma::mbar_init(tma::smem_u32(&task_bars[s]), 1);
        tma::fence_barrier_init();
        s_failed = 0u;
    }
    __syncthreads();
    const uint32_t one = __ldg(one_ptr);

    // ring positions, carried from task to task
    int stage = 0;                 // producer: next data stage to read
    uint32_t dparity = 0;
    int wslot = 0;                 // both: next W+K slot (the producer fills it, the consumer drains it)
    uint32_t eparity = 1;          // producer: the first pass over the slots finds them empty
    uint32_t fparity = 0;          // consumer
    bool failed = false;

    for (uint32_t turn = 0;; ++turn) {
        // ---- the producer's lane 0 takes a ticket and waits for the group that is pushed under it
        unsigned long long task = kTaskDone;
        const uint32_t task_bar = tma::smem_u32(&task_bars[turn % kTaskRing]);
        if (warp == 1) {
            if (lane == 0) {
                if (*reinterpret_cast<volatile uint32_t *>(&s_failed)) {
                    task = kTaskFailed;
                } else {
                    const unsigned long long t = atomicAdd(&q->head, 1ull);
                    if (t < total_tasks) {
                        uint32_t entry = ld_acquire_u32(slot + t);
                        if (entry == 0) {
                            const long long t0 = clock64();
                            unsigned ns = 64;
                            while ((entry = ld_acquire_u32(slot + t)) == 0) {
                                if (clock64() - t0 > 8000000000ll) break;       // about four seconds: give up
                                __nanosleep(ns);
                                if (ns < 2048) ns *= 2;
                            }
                        }
                        if (entry == 0) task = kTaskFailed;
                        else task = ((unsigned long long)(entry - 1u) << 32) | __ldcg(next_slice + (entry - 1u));
                    }
                }
                s_task[turn % kTaskRing] = task;
                tma::mbar_arrive(task_bar);        // releases the task (and, through the acquire above, the parked values)
            }
            task = __shfl_sync(0xffffffffu, task, 0);
        } else {
            if (!tma::mbar_wait_bounded(task_bar, (turn / kTaskRing) & 1u)) { failed = true; break; }
            task = *reinterpret_cast<volatile unsigned long long *>(&s_task[turn % kTaskRing]);
        }
        if (task == kTaskDone) break;
        if (task == kTaskFailed) { failed = true; break; }
        const uint64_t g = task >> 32;
        const uint32_t s = (uint32_t)task;

        // ---- this lane's share of the slice
        const uint64_t i = g * 32 + lane;
        const bool valid = i < n_chunks;
        const uint64_t begin = valid ? i * chunk_bytes : 0;
        const uint64_t len = valid ? ((nbytes - begin < chunk_bytes) ? (nbytes - begin) : chunk_bytes) : 0;
        const uint64_t full_bytes = len & ~63ull;
        const uint64_t lo = (uint64_t)s * slice_bytes;
        const uint64_t hi_full = lo + slice_bytes;
        const uint64_t my_lo = lo < full_bytes ? lo : full_bytes;
        const uint64_t my_hi = hi_full < full_bytes ? hi_full : full_bytes;
        // lane 0 holds the longest chunk of its group (only the blob's last chunk can be shorter)
        const uint64_t warp_full_bytes = __shfl_sync(0xffffffffu, full_bytes, 0);
        const bool last_slice = hi_full >= warp_full_bytes;
        const uint32_t my_data = (uint32_t)((my_hi - my_lo) >> 6);            // whole data blocks in this slice
        // blocks after the whole data blocks: the message's remainder and padding (the prefixed message is one
        // byte longer, and its block j ends one byte before data block j does)
        const uint32_t my_tail = !(valid && last_slice) ? 0u
                                 : PREFIX ? ((len + 1 - full_bytes) + 9 <= 64 ? 1u : 2u)
                                          : (uint32_t)((((len + 8) >> 6) + 1) - (full_bytes >> 6));
        const uint32_t my_total = my_data + my_tail;
        const uint32_t warp_total = __shfl_sync(0xffffffffu, my_total, 0);
        const uint32_t warp_data = __shfl_sync(0xffffffffu, my_data, 0);

        if (warp == 1) {
            // -------------------------------------------------------------- producer
            const uint8_t *p = data + begin + my_lo;
            const uint32_t my_bytes = my_data * 64u;
            const uint32_t nseg = (warp_data * 64u + SEG - 1) / SEG;
            auto issue = [&](uint32_t seg, int stg) {
                const uint32_t off = seg * SEG;
                const uint32_t bytes = off < my_bytes ? ((my_bytes - off < (uint32_t)SEG) ? (my_bytes - off) : (uint32_t)SEG) : 0u;
                const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
                if (lane == 0) tma::mbar_arrive_expect_tx(bar_data + 8 * stg, total);
                if (bytes) tma::bulk_g2s(data_base + stg * kStageBytes, p + off, bytes, bar_data + 8 * stg);
            };
            {
                int stg = stage;
#pragma unroll
                for (int k = 0; k < STAGES; ++k) {
                    if ((uint32_t)k < nseg) issue((uint32_t)k, stg);
                    if (++stg == STAGES) stg = 0;
                }
            }
            uint32_t w[16], raw[16], tw[32];
            uint32_t carry = 0u;        // PREFIX: the data word before the block; byte 3 of 0 is the prefix itself
            if (PREFIX && my_lo > 0 && my_data > 0) carry = __ldg(reinterpret_cast<const uint32_t *>(p) - 1);
            int in_stage = 0;
            bool tail_built = false;
            auto fetch = [&](int blk_in_stage) {
                const uint32_t src = data_base + stage * kStageBytes + 64 * blk_in_stage;
#pragma unroll
                for (int qd = 0; qd < 4; ++qd)
                    tma::ld_shared_v4(src + 16 * qd, raw[4 * qd], raw[4 * qd + 1], raw[4 * qd + 2], raw[4 * qd + 3]);
            };
            if (warp_data) {
                failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded(bar_data + 8 * stage, dparity));
                if (!failed) fetch(0);
            }
            uint32_t next_seg = STAGES;
            for (uint32_t blk = 0; blk < warp_total && !failed; ++blk) {
                if (blk < my_data) {
                    if (PREFIX) {
                        w[0] = shifted_word(raw[0], carry);
#pragma unroll
                        for (int k = 1; k < 16; ++k) w[k] = shifted_word(raw[k], raw[k - 1]);
                        carry = raw[15];
                    } else {
#pragma unroll
                        for (int k = 0; k < 16; ++k) w[k] = bswap32(raw[k]);
                    }
                } else if (blk < my_total) {
                    if (!tail_built) {
                        if (PREFIX) (void)prefixed_tail(data + begin, 0x00, full_bytes, len + 1, tw);
                        else (void)sha256_build_tail(data + begin + full_bytes, (uint32_t)(len & 63u), len, tw);
                        tail_built = true;
                    }
                    const int t = (int)(blk - my_data);
#pragma unroll
                    for (int k = 0; k < 16; ++k) w[k] = tw[16 * t + k];
                }
                if (blk + 1 < warp_data) {
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
                } else if (blk + 1 == warp_data) {
                    // the slice's last data block has been taken out: the ring position moves past its stage
                    __syncwarp();
                    if (++stage == STAGES) { stage = 0; dparity ^= 1u; }
                }
                const uint32_t in_slot = blk % PAIR;
                if (in_slot == 0) {
                    failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded(bar_empty + 8 * wslot, eparity));
                    if (failed) break;
                }
                produce_wk(w, wk_base + wslot * kWkSlot + in_slot * kWkBlock, one);
                if (in_slot == PAIR - 1 || blk + 1 == warp_total) {
                    __syncwarp();                          // all 32 lanes' stores are ordered before lane 0's arrival
                    if (lane == 0) tma::mbar_arrive(bar_full + 8 * wslot);
                    if (++wslot == NSLOT) { wslot = 0; eparity ^= 1u; }
                }
            }
            if (failed && lane == 0) atomicExch(&s_failed, 1u);
        } else {
            // -------------------------------------------------------------- consumer
            uint32_t st[8], v[8];
            if (s == 0) {
                sha256_init(st);
            } else {
                const uint32_t *m = mid + g * 256 + lane;
#pragma unroll
                for (int k = 0; k < 8; ++k) st[k] = __ldcg(m + 32 * k);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = st[k];
            for (uint32_t blk = 0; blk < warp_total; ++blk) {
                const uint32_t in_slot = blk % PAIR;
                if (in_slot == 0) {
                    failed = !tma::mbar_wait_bounded(bar_full + 8 * wslot, fparity);     // uniform: one barrier word
                    if (failed) break;
                }
                rounds64(v, wk_base + wslot * kWkSlot + in_slot * kWkBlock, one);
                const bool slot_done = in_slot == PAIR - 1 || blk + 1 == warp_total;
                if (slot_done) {
                    __syncwarp();                          // all 32 lanes have their values in registers
                    if (lane == 0) tma::mbar_arrive(bar_empty + 8 * wslot);
                }
                // feed-forward; a lane whose message has no block here keeps its state (multiplier 0 instead of 1)
                const uint32_t keep = (blk < my_total) ? one : 0u;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    st[k] = padd<true>(v[k], st[k], keep);
                    v[k] = st[k];
                }
                if (slot_done && ++wslot == NSLOT) { wslot = 0; fparity ^= 1u; }
            }
            if (failed) {
                if (lane == 0) atomicExch(&s_failed, 1u);
            } else if (!last_slice) {
                uint32_t *m = mid + g * 256 + lane;
#pragma unroll
                for (int k = 0; k < 8; ++k) __stcg(m + 32 * k, st[k]);
                __syncwarp();
                if (lane == 0) {
                    __stcg(next_slice + g, s + 1u);
                    __threadfence();
                    const unsigned long long pt = atomicAdd(&q->tail, 1ull);
                    st_release_u32(slot + pt, (uint32_t)g + 1u);
                }
            } else if (valid) {
                store_digest(digests + 32 * i, st);
            }
        }
    }
    if (failed && lane == 0) atomicExch(status, (uint32_t)IVK_DEV_TIMEOUT);
}

}  // namespace

bool hash_chunks_wants_pairs(const uint8_t *d_data, uint64_t chunk_bytes, uint64_t n_chunks, int sm_count) {
    // 590 GB/s flat for the pairs against 1.40 GB/s per group for one whole-compression warp per group:
    // measured crossover at 422 groups = 2.85 x SMs, for chunks of 1 MiB and 4 MiB
    return hash_chunks_wants_slices(d_data, chunk_bytes, n_chunks, sm_count) &&
           ((n_chunks + 31) / 32) * 100ull < 285ull * (uint64_t)sm_count;
}

cudaError_t launch_hash_chunks_pairs(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint64_t n_chunks,
                                     uint8_t *d_digests, uint32_t *d_status, void *d_scratch, const uint32_t *d_one,
                                     int sm_count, cudaStream_t stream, bool zero_prefix) {
    constexpr int SEG = 512, STAGES = 3, NSLOT = 3, PAIR = 2;
    constexpr size_t smem = (size_t)STAGES * 32 * (SEG + 16) + (size_t)NSLOT * PAIR * 32 * (64 * 4 + 16);
    auto kernel = zero_prefix ? hash_chunks_pairs_kernel<SEG, STAGES, NSLOT, PAIR, true>
                              : hash_chunks_pairs_kernel<SEG, STAGES, NSLOT, PAIR, false>;
    static bool configured[2][kMaxDevices] = {};
    if (cudaError_t e0 = ensure_dynamic_smem(kernel, smem, configured[zero_prefix ? 1 : 0]); e0 != cudaSuccess) return e0;
    uint64_t slice_bytes = 0, total_tasks = 0;
    (void)sliced_scratch_bytes(n_chunks, chunk_bytes, &slice_bytes, &total_tasks, nbytes);
    const uint64_t groups = (n_chunks + 31) / 32;
    uint8_t *base = static_cast<uint8_t *>(d_scratch);
    SliceQueue *q = reinterpret_cast<SliceQueue *>(base);
    uint32_t *mid = reinterpret_cast<uint32_t *>(base + 64);                       // 1 KiB per group, 16-byte aligned
    uint32_t *slot = reinterpret_cast<uint32_t *>(base + 64 + 1024 * groups);
    uint32_t *next_slice = slot + total_tasks;
    slice_queue_init<<<64, 256, 0, stream>>>(slot, total_tasks, groups, q, next_slice);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // two pairs per SM (104 KB of shared memory each): every warp has a scheduler of its own
    kernel<<<(unsigned)(2 * sm_count), 64, smem, stream>>>(d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status,
                                                           slice_bytes, total_tasks, slot, q, next_slice, mid, d_one);
    return cudaGetLastError();
}

}  // namespace ivk
