// SHA-384 / SHA-512 leaf hashing in the design of the SHA-256 path: tiled bulk copies, chains that migrate
// between workers through the slice FIFO, and the compression split between two warps.
//
// One warp carries 32 chains (a "group"); a chunk is one serial chain of 128-byte blocks (FIPS 180-4
// section 6.4).  The 64-bit additions and rotations are pairs of 32-bit instructions with carry and funnel
// dependencies, so one warp alone issues an instruction every 2.5 cycles, and with few groups the launch is
// bound by what one warp can issue, not by the SM's integer pipes.  As on the SHA-256 path the
// message schedule, the endian swap and the round-constant additions (44 % of the work) do not depend on
// the chaining value, so a group is served by a PAIR of warps:
//
//   producer: takes the (group, slice) task from the FIFO, brings the group's next block with ONE tiled copy
//             (the blob's whole chunks as a 2-D tensor, box = 32 rows x 128 bytes = one block per lane,
//             128-byte swizzle), forms W[t] + K[t] for the 80 rounds and hands them over in units of 16 rounds
//             through a lane-interleaved ring in shared memory (full/empty mbarriers per unit);
//   consumer: runs only the 80 rounds and the feed-forward, parks the chaining values in global memory at the
//             end of a slice and pushes the group back into the FIFO.
//
// The three-input boolean functions and the rotations are written on 32-bit halves (sha512_dev.cuh); left to
// the compiler's 64-bit code the same kernel ran at 78 % instead of 91 % of the integer roofline.  The loops
// over a block's five units stay rolled: the producers and consumers of up to sixteen warps run different code at the
// same time, and unrolled it no longer fits the instruction cache (218 GB/s against 521 at the time).
//
// A CTA holds PAIRS pairs (producer warps 0..PAIRS-1, consumer warps PAIRS..2 PAIRS-1, a pair's two warps on
// different schedulers); the launch picks two, four, six or eight pairs by the groups per SM
// (sha512_pairs_per_sm).  One persistent CTA per SM; pair 0 of every CTA takes tickets as they come, the other
// pairs take a task only when one lies in the FIFO unclaimed, the later ones of a CTA later and less often, so
// that few groups spread one per SM.  All waits are bounded.
#include <cstring>

#include "chunk_tensor_map.h"
#include "iv_internal.h"
#include "sha512_dev.cuh"
#include "slice_queue_dev.cuh"
#include "tma_dev.cuh"

namespace ivk {
namespace {

constexpr unsigned long long kTaskDone = ~0ull, kTaskFailed = ~0ull - 1;
constexpr uint32_t kUnitRounds = 16;                       // rounds handed over at a time
constexpr uint32_t kUnitLane = kUnitRounds * 8 + 16;       // W+K ring: bytes per lane per unit (padded: conflict-free)
constexpr uint32_t kUnitBytes = 32 * kUnitLane;
constexpr uint32_t kBoxBytes = 32 * 128;                   // one block of all 32 chains

// Sixteen schedule steps: w[i] <- W[t+16] from w[] = W[t .. t+15] (FIPS 180-4 section 6.4.2 step 1).
__device__ __forceinline__ void sched16_512(uint64_t (&w)[16]) {
#pragma unroll
    for (int i = 0; i < 16; ++i)
        w[i] += small_s1_512(w[(i + 14) & 15]) + w[(i + 9) & 15] + small_s0_512(w[(i + 1) & 15]);
}

// W[t] + K[t] for the sixteen t of a unit (k points at K[t0]) into this lane's part of a ring unit.
__device__ __forceinline__ void store_wk16_512(const uint64_t (&w)[16], const uint64_t *__restrict__ k, uint32_t dst) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint64_t a = w[2 * j] + k[2 * j], b = w[2 * j + 1] + k[2 * j + 1];
        tma::st_shared_v4(dst + 16 * j, lo32(a), hi32(a), lo32(b), hi32(b));
    }
}

// Sixteen rounds on W + K values already in registers (the variable names rotate back after 8 rounds).
__device__ __forceinline__ void rounds16_512(uint64_t (&v)[8], const uint64_t (&kw)[16]) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        uint64_t &a = v[(8 - i) & 7], &b = v[(9 - i) & 7], &c = v[(10 - i) & 7], &d = v[(11 - i) & 7];
        uint64_t &e = v[(12 - i) & 7], &f = v[(13 - i) & 7], &g = v[(14 - i) & 7], &h = v[(15 - i) & 7];
        const uint64_t t1 = h + big_s1_512(e) + ch64(e, f, g) + kw[i];
        d += t1;
        h = t1 + big_s0_512(a) + maj64(a, b, c);
    }
}

// DIGEST_WORDS = 6: SHA-384 (initial value of section 5.3.4, the leftmost 384 bits); 8: SHA-512 (section 5.3.5).
template <int PAIRS, int STAGES, int NSLOT, int DIGEST_WORDS>
__global__ void __launch_bounds__(64 * PAIRS, 1)
hash_sha512_pairs_kernel(const __grid_constant__ CUtensorMap tmap, const uint8_t *__restrict__ data, uint64_t chunk_bytes,
                         uint64_t n_chunks, uint8_t *__restrict__ digests, uint32_t *__restrict__ status,
                         uint64_t slice_bytes, uint64_t total_tasks, uint32_t *__restrict__ slot,
                         SliceQueue *__restrict__ q, uint32_t *__restrict__ next_slice,
                         uint64_t *__restrict__ mid /* [groups][8][32] */) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int kTaskRing = 8;
    __shared__ __align__(8) uint64_t bars[PAIRS][STAGES + 2 * NSLOT];
    __shared__ __align__(8) uint64_t task_bars[PAIRS][kTaskRing];
    __shared__ unsigned long long s_task[PAIRS][kTaskRing];
    __shared__ uint32_t s_failed[PAIRS];

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    const bool producer = warp < PAIRS;
    // the two warps of a pair sit on different schedulers (warp w runs on scheduler w mod 4)
    const uint32_t pair = producer ? warp : (PAIRS % 4 == 0 ? (warp - PAIRS + PAIRS - 1) % PAIRS : warp - PAIRS);
    // tiled boxes must start on a 1024-byte boundary (the swizzle pattern repeats every 8 rows)
    const uint32_t smem0 = (tma::smem_u32(smem) + 1023u) & ~1023u;
    const uint32_t data_ring = smem0 + pair * (STAGES * kBoxBytes);
    const uint32_t wk_ring = smem0 + PAIRS * (STAGES * kBoxBytes) + pair * (NSLOT * kUnitBytes) + lane * kUnitLane;
    const uint32_t swz = (lane & 7u) * 16u;
    const uint32_t bar_data = tma::smem_u32(&bars[pair][0]);
    const uint32_t bar_full = bar_data + 8 * STAGES;
    const uint32_t bar_empty = bar_full + 8 * NSLOT;
    if (producer && lane == 0) {
        // data stages: one arrival (lane 0 announces the box); W+K units: every lane of the producer (full) or of
        // the consumer (empty) arrives for itself, which needs no warp barrier and no one-lane branch
        for (int s = 0; s < STAGES; ++s) tma::mbar_init(bar_data + 8 * s, 1);
        for (int s = STAGES; s < STAGES + 2 * NSLOT; ++s) tma::mbar_init(bar_data + 8 * s, 32);
        for (int s = 0; s < kTaskRing; ++s) tma::mbar_init(tma::smem_u32(&task_bars[pair][s]), 1);
        s_failed[pair] = 0u;
        tma::fence_barrier_init();
    }
    __syncthreads();

    const uint64_t full_bytes = chunk_bytes & ~127ull;     // every chunk of the launch is a whole chunk
    const uint32_t tail_blocks = ((chunk_bytes & 127u) + 1 + 16 <= 128) ? 1u : 2u;

    // ring positions, carried from task to task
    int stage = 0;                 // producer: next data stage to read
    uint32_t dparity = 0;
    int wslot = 0;                 // both: next W+K unit (the producer fills it, the consumer drains it)
    uint32_t eparity = 1;          // producer: the first pass over the units finds them empty
    uint32_t fparity = 0;          // consumer
    bool failed = false;
    bool first_take = true;

    for (uint32_t turn = 0;; ++turn) {
        // ---- the producer's lane 0 takes a ticket and waits for the group that is pushed under it
        unsigned long long task = kTaskDone;
        const uint32_t task_bar = tma::smem_u32(&task_bars[pair][turn % kTaskRing]);
        if (producer) {
            if (lane == 0) {
                if (*reinterpret_cast<volatile uint32_t *>(&s_failed[pair])) {
                    task = kTaskFailed;
                } else {
                    const unsigned long long t = pair == 0 ? atomicAdd(&q->head, 1ull)
                                                           : take_leftover_ticket(q, total_tasks, first_take, pair - 1u);
                    if (t < total_tasks) {
                        // With few groups a ticket can lie many slices ahead of the pushes; the wait gives up only
                        // when the FIFO has not moved for about four seconds.
                        uint32_t entry = ld_acquire_u32(slot + t);
                        if (entry == 0) {
                            long long t0 = clock64();
                            unsigned long long seen = *reinterpret_cast<volatile unsigned long long *>(&q->tail);
                            unsigned ns = 64;
                            while ((entry = ld_acquire_u32(slot + t)) == 0) {
                                const unsigned long long now = *reinterpret_cast<volatile unsigned long long *>(&q->tail);
                                if (now != seen) { seen = now; t0 = clock64(); }
                                if (clock64() - t0 > 8000000000ll) break;
                                __nanosleep(ns);
                                if (ns < 2048) ns *= 2;
                            }
                        }
                        if (entry == 0) task = kTaskFailed;
                        else task = ((unsigned long long)(entry - 1u) << 32) | __ldcg(next_slice + (entry - 1u));
                    }
                }
                s_task[pair][turn % kTaskRing] = task;
                tma::mbar_arrive(task_bar);        // releases the task (and, through the acquire above, the parked values)
            }
            first_take = false;
            task = __shfl_sync(0xffffffffu, task, 0);
        } else {
            if (!tma::mbar_wait_bounded_sleepy(task_bar, (turn / kTaskRing) & 1u)) { failed = true; break; }
            task = *reinterpret_cast<volatile unsigned long long *>(&s_task[pair][turn % kTaskRing]);
        }
        if (task == kTaskDone) break;
        if (task == kTaskFailed) { failed = true; break; }
        const uint64_t g = task >> 32;
        const uint32_t s = (uint32_t)task;

        // ---- the slice: whole 128-byte blocks [lo, hi) of every chunk of the group, then (last slice) the tail
        const uint64_t i = g * 32 + lane;
        const bool valid = i < n_chunks;
        const uint64_t lo = (uint64_t)s * slice_bytes;
        const uint64_t hi = (lo + slice_bytes < full_bytes) ? lo + slice_bytes : full_bytes;
        const bool last_slice = lo + slice_bytes >= full_bytes;
        const uint32_t n_data = (uint32_t)((hi - lo) >> 7);
        const uint32_t n_total = n_data + (last_slice ? tail_blocks : 0u);

        if (producer) {
            // -------------------------------------------------------------- producer
            auto issue = [&](uint32_t blk, int stg) {
                if (lane == 0) {
                    tma::mbar_arrive_expect_tx(bar_data + 8 * stg, kBoxBytes);
                    tma::tiled_g2s(data_ring + stg * kBoxBytes, &tmap, (uint32_t)(lo + 128ull * blk), (uint32_t)(g * 32),
                                   bar_data + 8 * stg);
                }
            };
            {
                int stg = stage;
#pragma unroll
                for (int k = 0; k < STAGES; ++k) {
                    if ((uint32_t)k < n_data) issue((uint32_t)k, stg);
                    if (++stg == STAGES) stg = 0;
                }
            }
            uint64_t w[16], tw[32];
            bool tail_built = false;
            for (uint32_t blk = 0; blk < n_total && !failed; ++blk) {
                if (blk < n_data) {
                    failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded_sleepy(bar_data + 8 * stage, dparity));
                    if (failed) break;
                    // this lane's row of the box; 16-byte piece c sits at piece c ^ (row mod 8)
                    const uint32_t row = data_ring + stage * kBoxBytes + lane * 128u;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        uint32_t x, y, z, t;
                        tma::ld_shared_v4(row + ((16u * c) ^ swz), x, y, z, t);
                        w[2 * c] = be64(x, y);
                        w[2 * c + 1] = be64(z, t);
                    }
                    __syncwarp();                          // every lane has taken its block out of the stage
                    if (blk + STAGES < n_data) issue(blk + STAGES, stage);
                    if (++stage == STAGES) { stage = 0; dparity ^= 1u; }
                } else {
                    if (!tail_built) {
                        // lanes beyond the blob's last chunk have no bytes: they hash padding only and store nothing
                        (void)sha512_build_tail(data + (valid ? i * chunk_bytes + full_bytes : 0), valid ? (uint32_t)(chunk_bytes & 127u) : 0u,
                                                chunk_bytes, tw);
                        tail_built = true;
                    }
                    const int t = (int)(blk - n_data);
#pragma unroll
                    for (int k = 0; k < 16; ++k) w[k] = tw[16 * t + k];
                }
                // five units of sixteen rounds.  The loop stays rolled: producers and consumers of twelve warps run
                // different code at the same time, and together it has to fit the instruction cache.
#pragma unroll 1
                for (int u = 0; u < 5; ++u) {
                    if (u) sched16_512(w);
                    failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded_sleepy(bar_empty + 8 * wslot, eparity));
                    if (failed) break;
                    store_wk16_512(w, kSha512K + 16 * u, wk_ring + wslot * kUnitBytes);
                    tma::mbar_arrive(bar_full + 8 * wslot);    // every lane arrives after its own stores (release)
                    if (++wslot == NSLOT) { wslot = 0; eparity ^= 1u; }
                }
            }
            if (failed && lane == 0) atomicExch(&s_failed[pair], 1u);
        } else {
            // -------------------------------------------------------------- consumer
            uint64_t st[8], v[8];
            if (s == 0) {
                if (DIGEST_WORDS == 6) sha384_init(st);
                else sha512_init(st);
            } else {
                const uint64_t *m = mid + g * 256 + lane;
#pragma unroll
                for (int k = 0; k < 8; ++k) st[k] = __ldcg(m + 32 * k);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = st[k];
            // Five units of sixteen rounds per block.  A satisfied blocking wait in front of every unit costs about 130
            // cycles (its result decides a branch); a non-blocking test for the NEXT unit, issued before the rounds of
            // the current one, costs nothing when the producer is ahead, which it is after the slice's first units.
            // The fast loop runs while that test succeeds; when it fails the blocking wait outside takes over.
            uint32_t units_left = 5u * n_total;
            int u5 = 0;
            while (units_left != 0) {
                if (!tma::mbar_wait_bounded_sleepy(bar_full + 8 * wslot, fparity)) { failed = true; break; }     // uniform: one barrier word
                bool there;
#pragma unroll 1
                do {
                    const uint32_t src = wk_ring + wslot * kUnitBytes;
                    uint64_t kw[16];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint32_t x, y, z, t;
                        tma::ld_shared_v4(src + 16 * j, x, y, z, t);
                        kw[2 * j] = pack64(x, y);
                        kw[2 * j + 1] = pack64(z, t);
                    }
                    tma::mbar_arrive(bar_empty + 8 * wslot);   // every lane arrives once its own values are in registers
                    if (++wslot == NSLOT) { wslot = 0; fparity ^= 1u; }
                    --units_left;
                    there = units_left != 0 && tma::mbar_test_wait(bar_full + 8 * wslot, fparity);
                    rounds16_512(v, kw);
                    if (++u5 == 5) {
                        u5 = 0;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            st[k] += v[k];
                            v[k] = st[k];
                        }
                    }
                } while (there);
            }
            if (failed) {
                if (lane == 0) atomicExch(&s_failed[pair], 1u);
            } else if (!last_slice) {
                uint64_t *m = mid + g * 256 + lane;
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
                store_digest512<DIGEST_WORDS>(digests + 8 * DIGEST_WORDS * i, st);
            }
        }
    }
    if (failed && lane == 0) atomicExch(status, (uint32_t)IVK_DEV_TIMEOUT);
}

// Slices of at least 16 KiB, at most 256 per chunk, a multiple of 4 KiB, counted over the whole 128-byte blocks.
void sha512_slices(uint64_t chunk_bytes, uint64_t max_slices, uint64_t *slice_bytes, uint64_t *per_group) {
    uint64_t slices = chunk_bytes / 16384;
    if (slices > max_slices) slices = max_slices;
    if (slices < 1) slices = 1;
    uint64_t sb = (chunk_bytes + slices - 1) / slices;
    sb = (sb + 4095) & ~4095ull;
    uint64_t pg = ((chunk_bytes & ~127ull) + sb - 1) / sb;
    if (pg < 1) pg = 1;
    *slice_bytes = sb;
    *per_group = pg;
}

thread_local const char *t_pairs_instance = "";     // which instance the calling thread's last launch used

template <int PAIRS, int STAGES, int NSLOT, int DIGEST_WORDS>
cudaError_t launch_pairs(const CUtensorMap &map, const uint8_t *d_data, uint64_t chunk_bytes, uint64_t whole,
                         uint8_t *d_digests, uint32_t *d_status, void *d_scratch, int sm_count, cudaStream_t stream) {
    constexpr size_t smem = 1024 + (size_t)PAIRS * (STAGES * kBoxBytes + NSLOT * kUnitBytes);
    auto kernel = hash_sha512_pairs_kernel<PAIRS, STAGES, NSLOT, DIGEST_WORDS>;
    static bool configured[kMaxDevices] = {};
    if (cudaError_t e0 = ensure_dynamic_smem(kernel, smem, configured); e0 != cudaSuccess) return e0;
    uint64_t slice_bytes = 0, per_group = 0;
    const uint64_t groups = (whole + 31) / 32;
    // a group per SM or fewer: every group keeps one pair for the whole launch, there is nothing to balance
    sha512_slices(chunk_bytes, groups <= (uint64_t)sm_count ? 1 : 256, &slice_bytes, &per_group);
    const uint64_t total_tasks = groups * per_group;
    uint8_t *base = static_cast<uint8_t *>(d_scratch);
    SliceQueue *q = reinterpret_cast<SliceQueue *>(base);
    uint64_t *mid = reinterpret_cast<uint64_t *>(base + 64);                       // 2 KiB per group
    uint32_t *slot = reinterpret_cast<uint32_t *>(base + 64 + 2048 * groups);
    uint32_t *next_slice = slot + total_tasks;
    slice_queue_init<<<64, 256, 0, stream>>>(slot, total_tasks, groups, q, next_slice);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    kernel<<<(unsigned)sm_count, 64 * PAIRS, smem, stream>>>(map, d_data, chunk_bytes, whole, d_digests, d_status, slice_bytes,
                                                            total_tasks, slot, q, next_slice, mid);
    return cudaGetLastError();
}

}  // namespace

const char *sha512_pairs_instance_name() { return t_pairs_instance; }

// Which launches the two-warp kernel takes and with how many pairs per SM.  Measured on 148 SMs (GB/s of SHA-384, G
// groups of 32 chains, S SMs; "plain" is the one-chain-per-lane kernel of hash_sha384.cu):
//   * pairs a CTA does not need cost the working ones a fifth of their speed (their warps poll and share schedulers
//     in no fixed order), so the pair count follows the groups per SM: two pairs below 3 S groups (1.5 GB/s per
//     group up to 2 S: 256 groups of 256 KiB chunks 375 against 273 with six pairs), four from there (each scheduler
//     one producer and one consumer: 445 to 577 between 3 S and 4 S, where the plain kernel gives 399 to 533, and
//     580 to 590 up to 6 S against 470 to 580 with six), six from 6 S for chunks of 1 MiB and more (612 against 604 on
//     896 groups of 4 MiB), eight from 8 S (two producers and two consumers per scheduler: 620 to 646);
//   * short chunks are short tasks: below 64 KiB the plain kernel is ahead from 3 S groups on (16 KiB chunks: 500
//     against 359 at 592 groups, 548 against 496 at 2,048), below 256 KiB from 4,096 groups on (64 KiB chunks: 635
//     against 610 at 4,000); from 256 KiB the pairs stay ahead at every count (641 against 598 at 4,800 groups).
int sha512_pairs_per_sm(uint64_t groups, uint64_t chunk_bytes, int sm_count) {
    const uint64_t s = (uint64_t)sm_count;
    if (groups < 3 * s) return 2;
    if (groups >= 8 * s && (chunk_bytes >= (128u << 10) || groups >= 14 * s)) return 8;
    if (groups >= 6 * s && chunk_bytes >= (1u << 20)) return 6;
    return 4;
}

bool sha512_wants_pairs(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, int sm_count) {
    if ((reinterpret_cast<uintptr_t>(d_data) & 15u) != 0 || chunk_bytes % 16u != 0 || chunk_bytes < 16384 ||
        chunk_bytes >= (1ull << 31) || nbytes < chunk_bytes)
        return false;
    const uint64_t groups = (nbytes / chunk_bytes + 31) / 32;
    if (chunk_bytes < (64u << 10)) return groups < 3ull * (uint64_t)sm_count;
    if (chunk_bytes < (256u << 10)) return groups < 4096;
    return true;
}

uint64_t sha512_pairs_scratch_bytes(uint64_t nbytes, uint64_t chunk_bytes) {
    uint64_t slice_bytes = 0, per_group = 0;
    sha512_slices(chunk_bytes, 256, &slice_bytes, &per_group);
    const uint64_t groups = (nbytes / chunk_bytes + 31) / 32;
    return 64 + 2048 * groups + 4 * groups * per_group + 4 * groups + 256;
}

// Hashes the blob's whole chunks (*covered of them, from the front; 0 and nothing launched if the blob cannot be
// described to the TMA unit); a short last chunk is left to the caller.
cudaError_t launch_hash_sha512_pairs(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes, uint8_t *d_digests,
                                     int digest_words, uint32_t *d_status, void *d_scratch, int sm_count,
                                     cudaStream_t stream, uint64_t *covered, uint64_t *launches) {
    const uint64_t whole = nbytes / chunk_bytes;
    alignas(64) CUtensorMap map;
    std::memset(&map, 0, sizeof map);
    *covered = 0;
    if (whole == 0 || !make_chunk_tensor_map(&map, d_data, chunk_bytes, whole)) return cudaSuccess;
    *covered = whole;
    if (launches) *launches += 2;
    const int pairs = sha512_pairs_per_sm((whole + 31) / 32, chunk_bytes, sm_count);
    t_pairs_instance = pairs == 8 ? "8 pairs per SM" : pairs == 6 ? "6 pairs per SM" : pairs == 4 ? "4 pairs per SM" : "2 pairs per SM";
#define IV_GO(P, S, N)                                                                                                           \
    (digest_words == 6 ? launch_pairs<P, S, N, 6>(map, d_data, chunk_bytes, whole, d_digests, d_status, d_scratch, sm_count, stream) \
                       : launch_pairs<P, S, N, 8>(map, d_data, chunk_bytes, whole, d_digests, d_status, d_scratch, sm_count, stream))
    switch (pairs) {
        case 8: return IV_GO(8, 2, 4);
        case 6: return IV_GO(6, 3, 5);
        case 4: return IV_GO(4, 3, 5);
        default: return IV_GO(2, 3, 5);
    }
#undef IV_GO
}

}  // namespace ivk
