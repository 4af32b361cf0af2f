// Leaf hashing when chains are plentiful but do not divide evenly over the GPU.
//
// One warp carries 32 chains (a "group").  With G groups on 592 SM schedulers a static
// assignment leaves some schedulers with two warps and others with one for the whole launch
// (28,672 chunks = 896 groups: 304 schedulers get two groups, 288 get one, and the launch lasts as
// long as the doubly loaded ones).  Here the chains migrate instead: every chunk is cut into
// slices, a task is (group, slice), and persistent warps take tasks from a FIFO in global
// memory.  A group re-enters the FIFO when its slice is done, its eight-word chaining values
// parked in global memory, so its next slice can run on any scheduler.  Because a group is in
// the FIFO at most once, its slices run in order; a warp never waits while it holds a task, so
// the scheme needs no co-residency and cannot deadlock.  All waits are bounded.
//
// Worker count.  A scheduler that runs two groups completes about 1.08 groups in the time a
// scheduler with one group completes one, so a second worker per scheduler pays only when it is
// busy: four workers per SM up to six groups per SM, six or seven workers (as many as there are
// whole groups per SM) on two progress-ordered queues up to 7.25, eight from there.
//
// Data movement: the blob is described to the TMA unit as a 2-D tensor [chunk][byte] with the chunk
// size as row pitch, and ONE tiled copy of a 32-row x 128-byte box brings the next two blocks of all
// 32 chains (instead of 32 copies issued one lane after the other).  The box lands row-major, one
// 128-byte row per lane, with the 128-byte swizzle (16-byte piece c of row r sits at piece
// c ^ (r mod 8)), so the lanes' 128-bit loads of the same piece hit eight different bank groups.
// Completion is counted by one mbarrier per stage and the next block is in registers before the
// current block's rounds.
#include <cuda.h>          // CUtensorMap (types only; the encoder is fetched through the runtime)

#include <cstring>

#include "iv_internal.h"
#include "rfc6962_dev.cuh"
#include "sha256_dev.cuh"
#include "slice_queue_dev.cuh"
#include "tma_dev.cuh"
#include "chunk_tensor_map.h"

namespace ivk {
namespace {

// Two FIFOs instead of one, so that groups advance evenly when workers differ in speed.  With five to seven
// workers per SM some schedulers run two workers and some one; a worker that has its scheduler to itself finishes
// a slice in 0.73 M cycles, one that shares it in 1.3 M.  Served from ONE FIFO, a group meets fast and slow workers
// at random, the groups' progress spreads by about ten slices over a launch, and the launch ends with most
// workers waiting for the stragglers (six workers per SM on 896 groups: every worker 5 % idle, 798 GB/s where the
// workers' rates add up to 877).  Here a finished slice pushes its group into queue 0 if the group is at or behind
// the average progress (tasks done so far / groups) and into queue 1 if it is ahead; workers alone on their
// scheduler take from queue 0 first, the others from queue 1 first, each from the other queue when its own is
// empty.  Laggards thus get the fast workers, and all groups finish within a slice or two of one another.
struct LagQueues {
    unsigned long long head[2];     // next ticket of each queue
    unsigned long long tail[2];     // next push position of each queue
    unsigned long long done;        // slices completed so far
};

// slot[k][t] = group + 1 once position t of queue k has been pushed, 0 before.  All groups start in queue 0 at slice 0.
__global__ void lag_queues_init(uint32_t *__restrict__ slot0, uint32_t *__restrict__ slot1, uint64_t total_tasks,
                                uint64_t groups, LagQueues *__restrict__ q, uint32_t *__restrict__ next_slice) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total_tasks; i += stride) {
        slot0[i] = i < groups ? (uint32_t)i + 1u : 0u;
        slot1[i] = 0u;
    }
    for (uint64_t g = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += stride) next_slice[g] = 0u;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        q->head[0] = q->head[1] = 0ull;
        q->tail[0] = groups;
        q->tail[1] = 0ull;
        q->done = 0ull;
    }
}

constexpr uint32_t kNoMoreTasks = 0u, kGaveUp = 0xffffffffu;

// The four counters of the two queues as one lane saw them.
struct QueueCounters {
    unsigned long long head[2], tail[2];
};
__device__ __forceinline__ QueueCounters read_counters(const LagQueues *q) {
    QueueCounters c;
    c.head[0] = *reinterpret_cast<const volatile unsigned long long *>(&q->head[0]);
    c.head[1] = *reinterpret_cast<const volatile unsigned long long *>(&q->head[1]);
    c.tail[0] = *reinterpret_cast<const volatile unsigned long long *>(&q->tail[0]);
    c.tail[1] = *reinterpret_cast<const volatile unsigned long long *>(&q->tail[1]);
    return c;
}

// One lane's call: the next task for a worker that prefers queue `pref`.  Returns group + 1, kNoMoreTasks once every
// slice of the launch is done, or kGaveUp after about four seconds without finding work (some other worker has
// failed); *done_seen receives the number of slices completed when the task was taken (the push that follows the
// task uses it as the average progress: a task's time out of date, which is exact enough).  `seen` holds the
// counters as the caller read them a little earlier (before it parked its finished slice, so that this read overlaps
// that work); they only choose the queue and the position to try, the compare-and-swap decides.  A lost race tries
// the position the swap returned before reading everything again.  Out of line so that the hashing loop's register
// allocation does not depend on it.
__device__ __noinline__ uint32_t take_task(LagQueues *q, const uint32_t *slot0, const uint32_t *slot1, uint32_t pref,
                                           unsigned long long total_tasks, unsigned long long *done_seen, QueueCounters seen) {
    const long long t0 = clock64();
    unsigned ns = 64;
    for (;;) {
        const bool have0 = seen.tail[0] > seen.head[0], have1 = seen.tail[1] > seen.head[1];
        if (have0 || have1) {
            const uint32_t which = (pref == 0u) ? (have0 ? 0u : 1u) : (have1 ? 1u : 0u);
            const unsigned long long h = seen.head[which];
            const unsigned long long was = atomicCAS(&q->head[which], h, h + 1ull);
            if (was != h) {                                    // lost the race (or the counters were stale): try again from
                seen.head[which] = was;                        // where the head stands now, against the tail as last seen
                if (seen.tail[which] <= was) seen = read_counters(q);
                continue;
            }
            // position h is this worker's; its entry may still be on its way (the pusher raises the tail first)
            const unsigned long long d = *reinterpret_cast<volatile unsigned long long *>(&q->done);
            const uint32_t *slot = (which ? slot1 : slot0) + h;
            uint32_t entry;
            while ((entry = ld_acquire_u32(slot)) == 0) {
                if (clock64() - t0 > 8000000000ll) return kGaveUp;
                __nanosleep(32);
            }
            *done_seen = d;
            return entry;
        }
        if (*reinterpret_cast<volatile unsigned long long *>(&q->done) >= total_tasks) return kNoMoreTasks;
        if (clock64() - t0 > 8000000000ll) return kGaveUp;
        __nanosleep(ns);
        if (ns < 1024) ns *= 2;
        seen = read_counters(q);
    }
}

// PREFIX: every chunk is hashed as 0x00 || chunk (the RFC 6962 leaf hash).  Message block j is then the
// byte before data block j followed by its first 63 bytes; the word before the block is carried in a
// register, at the start of a later slice it is read back from the blob.
// ADD: where the additions of the compression go (see sha256_compress).
// MINB: the second argument of __launch_bounds__ (0 = none).  It changes nothing that is computed, only the code the
// compiler makes of the block loop: told that one CTA per SM is enough it spends 91-96 registers instead of 65-71 on
// the instances with up to eight workers and orders the loop better (one group per scheduler: 798 -> 830 GB/s, two:
// 876 -> 891, the 112 GiB launch: 808 -> 826); the twelve-worker instance loses by it (920 -> 904) and keeps 0.
// LAG: tasks come from the two progress-ordered queues (launches whose workers differ in speed: five to seven per
// SM) instead of the single FIFO (workers all alike: four, eight or twelve per SM; the two queues would cost those
// about 1 %: a take and a push are two trips to memory longer).
template <int SEG, int STAGES, int MAX_WARPS, bool PREFIX, int ADD, int MINB, bool LAG>
__global__ void __launch_bounds__(32 * MAX_WARPS, MINB)
hash_chunks_sliced_kernel(const __grid_constant__ CUtensorMap tmap, const uint8_t *__restrict__ data, uint64_t nbytes, uint64_t chunk_bytes,
                          uint64_t n_chunks, uint8_t *__restrict__ digests, uint32_t *__restrict__ status,
                          uint64_t slice_bytes, uint64_t total_tasks, uint64_t groups, uint32_t *__restrict__ slot0,
                          uint32_t *__restrict__ slot1, LagQueues *__restrict__ q, uint32_t *__restrict__ next_slice,
                          uint32_t *__restrict__ mid /* [groups][8][32] */, const uint32_t *__restrict__ one_ptr) {
    // With two warps per scheduler addition placement 0 (left to the compiler) is the fastest; moving the
    // schedule's additions to the FMA pipe (placement 2) lengthens the dependency chains and needs three warps
    // per scheduler to pay (launcher below).
    const uint32_t one = __ldg(one_ptr);
    static_assert(SEG == 256, "a stage is two boxes of 32 rows x 128 bytes");
    constexpr uint32_t kLaneStride = 128;
    constexpr uint32_t kStageBytes = 8192;
    constexpr int kBlocksPerSeg = SEG / 64;
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ __align__(8) uint64_t bars[MAX_WARPS][STAGES];

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    // tiled boxes must start on a 1024-byte boundary (the swizzle pattern repeats every 8 rows)
    const uint32_t ring0 = (tma::smem_u32(ring) + 1023u) & ~1023u;
    const uint32_t ring_warp = ring0 + warp * (STAGES * kStageBytes);
    const uint32_t ring_base = ring_warp + lane * kLaneStride;
    const uint32_t swz = (lane & 7u) * 16u;
    const uint32_t bar_base = tma::smem_u32(&bars[warp][0]);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) tma::mbar_init(bar_base + 8 * s, 1);
        tma::fence_barrier_init();
    }
    __syncwarp();

    // ring position, carried from task to task (every task drains what it requested)
    int stage = 0;
    uint32_t parity = 0;
    bool failed = false;
    // warp w runs on scheduler w mod 4: alone there if no warp w + 4 exists.  Such a worker is the faster kind and
    // takes lagging groups (queue 0) first; a worker that shares its scheduler takes leading groups first -- but only
    // where the CTA has workers of both kinds (five to seven): where all are alike, all take laggards first, which
    // keeps the groups together (leaders first for everybody would let a few groups run away and finish alone).
    const uint32_t n_warps = blockDim.x >> 5;
    const bool mixed = n_warps > 4 && n_warps < 8;
    const uint32_t pref = (mixed && !(warp < 4 && warp + 4 >= n_warps)) ? 1u : 0u;
    QueueCounters seen = {};
    if (LAG && lane == 0) seen = read_counters(q);

    for (;;) {
        uint32_t entry = 0;
        unsigned long long done_seen = 0;
        if constexpr (LAG) {
            // ---- take a task: lagging groups first for a worker alone on its scheduler, leading ones first otherwise
            if (lane == 0) entry = take_task(q, slot0, slot1, pref, total_tasks, &done_seen, seen);
            entry = __shfl_sync(0xffffffffu, entry, 0);
            if (entry == kNoMoreTasks) break;
            if (entry == kGaveUp) { failed = true; break; }
        } else {
            // ---- take a ticket of the single FIFO (queue 0), wait for the group that is pushed under it
            unsigned long long t = 0;
            if (lane == 0) t = atomicAdd(&q->head[0], 1ull);
            t = __shfl_sync(0xffffffffu, t, 0);
            if (t >= total_tasks) break;
            if (lane == 0) {
                entry = ld_acquire_u32(slot0 + t);
                if (entry == 0) {
                    const long long t0 = clock64();
                    unsigned ns = 64;
                    while ((entry = ld_acquire_u32(slot0 + t)) == 0) {
                        if (clock64() - t0 > 8000000000ll) break;       // about four seconds: give up
                        __nanosleep(ns);
                        if (ns < 2048) ns *= 2;
                    }
                }
            }
            entry = __shfl_sync(0xffffffffu, entry, 0);
            if (entry == 0) { failed = true; break; }
        }
        const uint64_t g = entry - 1u;
        // lane 0 made the acquire; it reads the slice number and the warp barrier orders the other
        // lanes' reads of the parked chaining values after it
        uint32_t s = 0;
        if (lane == 0) s = __ldcg(next_slice + g);
        s = __shfl_sync(0xffffffffu, s, 0);
        __syncwarp();

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
        const uint64_t my_bytes = my_hi - my_lo;                       // multiple of 64
        const uint8_t *p = data + begin + my_lo;
        // lane 0 holds the longest chunk of its group (only the blob's last chunk can be shorter)
        const uint64_t warp_bytes = __shfl_sync(0xffffffffu, my_bytes, 0);
        const uint64_t warp_full = __shfl_sync(0xffffffffu, full_bytes, 0);
        const bool last_slice = hi_full >= warp_full;
        const uint64_t nseg = (warp_bytes + SEG - 1) / SEG;

        uint32_t st[8], w[16], raw[16];
        uint32_t carry = 0u;          // PREFIX: the data word before the block; byte 3 of 0 is the prefix itself
        if (PREFIX && my_lo > 0 && my_bytes > 0) carry = __ldg(reinterpret_cast<const uint32_t *>(p) - 1);
        if (s == 0) {
            sha256_init(st);
        } else {
            const uint32_t *m = mid + g * 256 + lane;
#pragma unroll
            for (int k = 0; k < 8; ++k) st[k] = __ldcg(m + 32 * k);
        }

        auto issue = [&](uint64_t seg, int stg) {
            const uint64_t off = seg * SEG;
            const uint32_t bar = bar_base + 8 * stg;
            // one or two boxes of 32 chains x 128 bytes; a box always delivers its 4096 bytes
            // (rows or bytes outside the tensor arrive as zeros and are never hashed)
            if (lane == 0) {
                const uint32_t boxes = (warp_bytes - off > 128) ? 2u : 1u;
                tma::mbar_arrive_expect_tx(bar, boxes * 4096u);
                const uint32_t x = (uint32_t)(lo + off), y = (uint32_t)(g * 32);
                tma::tiled_g2s(ring_warp + stg * kStageBytes, &tmap, x, y, bar);
                if (boxes == 2) tma::tiled_g2s(ring_warp + stg * kStageBytes + 4096u, &tmap, x + 128u, y, bar);
            }
        };
        auto fetch = [&](int stg, int blk_in_stage) {
            // block b of the stage: box b / 2, 16-byte pieces 4 (b mod 2) .. +3 of this lane's row
            const uint32_t row = ring_base + stg * kStageBytes + (uint32_t)(blk_in_stage >> 1) * 4096u;
            const uint32_t c0 = (uint32_t)(blk_in_stage & 1) * 64u;
#pragma unroll
            for (int qd = 0; qd < 4; ++qd)
                tma::ld_shared_v4(row + ((c0 + 16u * qd) ^ swz), raw[4 * qd], raw[4 * qd + 1], raw[4 * qd + 2],
                                  raw[4 * qd + 3]);
        };

        // prologue: request the first STAGES segments into the stages that follow the ring position
        {
            int stg = stage;
#pragma unroll
            for (int k = 0; k < STAGES; ++k) {
                if ((uint64_t)k < nseg) issue(k, stg);
                if (++stg == STAGES) stg = 0;
            }
        }
        // block and segment counts of a slice fit 32 bits (a slice is at most 1/256 of a chunk beyond 4 MiB)
        const uint32_t warp_blocks = (uint32_t)(warp_bytes >> 6);
        const uint32_t nseg32 = (uint32_t)nseg;
        int in_stage = 0;
        if (warp_blocks) {
            failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded(bar_base + 8 * stage, parity));
            if (failed) break;
            fetch(stage, 0);
        }
        uint32_t next_seg = STAGES;
        for (uint32_t blk = 0; blk < warp_blocks; ++blk) {
            if (PREFIX) {
                w[0] = shifted_word(raw[0], carry);
#pragma unroll
                for (int k = 1; k < 16; ++k) w[k] = shifted_word(raw[k], raw[k - 1]);
                carry = raw[15];
            } else {
#pragma unroll
                for (int k = 0; k < 16; ++k) w[k] = bswap32(raw[k]);
            }
            const bool stage_done = (++in_stage == kBlocksPerSeg) || (blk + 1 == warp_blocks);
            if (stage_done) {
                in_stage = 0;
                __syncwarp();                            // every lane has taken its data out of the stage
                if (next_seg < nseg32) issue(next_seg, stage);
                ++next_seg;
                if (++stage == STAGES) { stage = 0; parity ^= 1u; }
                if (blk + 1 < warp_blocks) {
                    failed = !__all_sync(0xffffffffu, tma::mbar_wait_bounded(bar_base + 8 * stage, parity));
                    if (failed) break;
                }
            }
            // Every lane of a group has the same number of blocks (lanes beyond the blob's last chunk hash the
            // zeros their rows were filled with and store nothing), and a fetch past the last block reads ring
            // memory that is never used: neither needs a branch.  Measured: the loop without the two branches
            // and with 32-bit counters is 1.7 % faster on the 112 GiB launch and 3.3 % where every scheduler
            // runs a single group.
            fetch(stage, in_stage);
            sha256_compress<ADD>(st, w, one);
        }
        if (failed) break;

        if (LAG && lane == 0) seen = read_counters(q);          // for the next take; on its way while the slice is parked
        if (!last_slice) {
            uint32_t *m = mid + g * 256 + lane;
#pragma unroll
            for (int k = 0; k < 8; ++k) __stcg(m + 32 * k, st[k]);
            __syncwarp();
            if (lane == 0) {
                __stcg(next_slice + g, s + 1u);
                __threadfence();
                uint32_t which = 0u;
                if constexpr (LAG) {
                    // at or behind the average progress (as of this task's start): queue 0, ahead of it: queue 1
                    atomicAdd(&q->done, 1ull);                                 // result unused: no wait for it
                    which = ((unsigned long long)s * groups <= done_seen) ? 0u : 1u;
                }
                const unsigned long long pt = atomicAdd(&q->tail[which], 1ull);
                st_release_u32((which ? slot1 : slot0) + pt, (uint32_t)g + 1u);
            }
            continue;
        }
        if (LAG && lane == 0) atomicAdd(&q->done, 1ull);
        if (!valid) continue;
        const uint32_t rem = (uint32_t)(len & 63u);
        if (PREFIX) {
            uint32_t tw[32];
            const int nblk = prefixed_tail(data + begin, 0x00, full_bytes, len + 1, tw);
#pragma unroll 1
            for (int tb = 0; tb < nblk; ++tb) {
#pragma unroll
                for (int k = 0; k < 16; ++k) w[k] = tw[16 * tb + k];
                sha256_compress(st, w);
            }
        } else if (rem == 0) {
            sha256_pad_only_block(w, len);
            sha256_compress(st, w);
        } else {
            uint32_t tw[32];
            const int nblk = sha256_build_tail(data + begin + full_bytes, rem, len, tw);
#pragma unroll 1
            for (int tb = 0; tb < nblk; ++tb) {
#pragma unroll
                for (int k = 0; k < 16; ++k) w[k] = tw[16 * tb + k];
                sha256_compress(st, w);
            }
        }
        store_digest(digests + 32 * i, st);
    }
    if (failed && lane == 0) atomicExch(status, (uint32_t)IVK_DEV_TIMEOUT);
}

}  // namespace

uint64_t sliced_scratch_bytes(uint64_t n_chunks, uint64_t chunk_bytes, uint64_t *slice_bytes_out, uint64_t *total_tasks_out,
                              uint64_t nbytes) {
    const uint64_t groups = (n_chunks + 31) / 32;
    // slices of at least 16 KiB, at most 256 per chunk, a multiple of 4 KiB
    uint64_t slices = chunk_bytes / 16384;
    if (slices > 256) slices = 256;
    if (slices < 1) slices = 1;
    uint64_t slice_bytes = (chunk_bytes + slices - 1) / slices;
    slice_bytes = (slice_bytes + 4095) & ~4095ull;
    // slices are counted over the whole 64-byte blocks of a chunk, as the kernel does
    uint64_t per_group = ((chunk_bytes & ~63ull) + slice_bytes - 1) / slice_bytes;
    if (per_group < 1) per_group = 1;
    // the last group's first chunk may be the blob's short last chunk
    const uint64_t first_of_last = (groups - 1) * 32;
    const uint64_t begin = first_of_last * chunk_bytes;
    const uint64_t len = nbytes - begin < chunk_bytes ? nbytes - begin : chunk_bytes;
    const uint64_t full = len & ~63ull;
    uint64_t last_group = (full + slice_bytes - 1) / slice_bytes;
    if (last_group < 1) last_group = 1;
    const uint64_t total = (groups - 1) * per_group + last_group;
    if (slice_bytes_out) *slice_bytes_out = slice_bytes;
    if (total_tasks_out) *total_tasks_out = total;
    // queue header (64) + chaining values + slots of two queues + next_slice
    return 64 + 1024 * groups + 8 * total + 4 * groups + 256;
}

namespace {

// cuTensorMapEncodeTiled, fetched through the runtime so that the library does not link libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult st = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &st) != cudaSuccess ||
            st != cudaDriverEntryPointSuccess)
            p = nullptr;
        (void)cudaGetLastError();
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

}  // namespace

// The blob's whole chunks as a 2-D byte tensor [rows][chunk_bytes], box = 32 rows x 128 bytes, 128-byte swizzle.
bool make_chunk_tensor_map(CUtensorMap *map, const uint8_t *d_data, uint64_t chunk_bytes, uint64_t rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || rows == 0 || chunk_bytes >= (1ull << 31) || rows >= (1ull << 31)) return false;
    const cuuint64_t gdim[2] = {chunk_bytes, rows};
    const cuuint64_t gstride[1] = {chunk_bytes};             // row pitch in bytes (a multiple of 16)
    const cuuint32_t box[2] = {128, 32};
    const cuuint32_t estride[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t *>(d_data), gdim, gstride, box, estride,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

thread_local const char *t_instance = "";

template <bool PREFIX>
cudaError_t launch_sliced(const CUtensorMap &map, const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                          uint64_t n_chunks, uint8_t *d_digests, uint32_t *d_status, void *d_scratch,
                          const uint32_t *d_one, int sm_count, cudaStream_t stream) {
    // Three instances: up to eight workers per SM with three stages each, on the single FIFO or on the two
    // progress-ordered queues, and twelve workers with two stages each for launches that keep all of them busy.
    constexpr int SEG = 256, STAGES = 3, MAX_WARPS = 8, MANY_STAGES = 2, MANY_WARPS = 12;
    constexpr size_t smem_per_warp = (size_t)STAGES * 8192, many_per_warp = (size_t)MANY_STAGES * 8192;
    constexpr size_t smem_pad = 1024;
    auto kernel = hash_chunks_sliced_kernel<SEG, STAGES, MAX_WARPS, PREFIX, 0, 1, false>;
    auto kernel_lag = hash_chunks_sliced_kernel<SEG, STAGES, MAX_WARPS, PREFIX, 0, 1, true>;
    auto kernel_many = hash_chunks_sliced_kernel<SEG, MANY_STAGES, MANY_WARPS, PREFIX, 2, 0, false>;
    static bool configured[kMaxDevices] = {}, configured_lag[kMaxDevices] = {}, configured_many[kMaxDevices] = {};
    if (cudaError_t e0 = ensure_dynamic_smem(kernel, MAX_WARPS * smem_per_warp + smem_pad, configured); e0 != cudaSuccess) return e0;
    if (cudaError_t e0 = ensure_dynamic_smem(kernel_lag, MAX_WARPS * smem_per_warp + smem_pad, configured_lag); e0 != cudaSuccess) return e0;
    if (cudaError_t e0 = ensure_dynamic_smem(kernel_many, MANY_WARPS * many_per_warp + smem_pad, configured_many); e0 != cudaSuccess) return e0;
    uint64_t slice_bytes = 0, total_tasks = 0;
    (void)sliced_scratch_bytes(n_chunks, chunk_bytes, &slice_bytes, &total_tasks, nbytes);
    const uint64_t groups = (n_chunks + 31) / 32;
    uint8_t *base = static_cast<uint8_t *>(d_scratch);
    LagQueues *q = reinterpret_cast<LagQueues *>(base);
    static_assert(sizeof(LagQueues) <= 64, "the queue header has 64 bytes of the scratch");
    uint32_t *mid = reinterpret_cast<uint32_t *>(base + 64);                       // 1 KiB per group, 16-byte aligned
    uint32_t *slot0 = reinterpret_cast<uint32_t *>(base + 64 + 1024 * groups);
    uint32_t *slot1 = slot0 + total_tasks;
    uint32_t *next_slice = slot1 + total_tasks;
    lag_queues_init<<<64, 256, 0, stream>>>(slot0, slot1, total_tasks, groups, q, next_slice);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // One persistent CTA per SM.  Measured (GB/s at G = 600 / 800 / 896 / 1000 / 1100 / 1184 groups of 4 MiB chunks):
    //  * four workers (one per scheduler), single FIFO: 831 / 832 / 833 / 829 / 834 / 834, flat for every G >= 592;
    //  * eight workers (two per scheduler), single FIFO: 745 / 769 / 813 / 852 / 884 / 897 (idle second workers fall
    //    at random, and a scheduler with two groups is only 8 % ahead of one with one);
    //  * as many workers as whole groups per SM, so that all are busy, on the single FIFO: five / six / seven workers
    //    835 / 797 / 795 at 896 and 834 / 849 / 847 at 1000 -- the groups' progress spreads and the launch ends on a
    //    few stragglers; on the two progress-ordered queues: five workers 836 / 843 / 844 at 740 / 800 / 887, six 862 /
    //    863 at 896 / 1000, seven 881 at 1,040.  The queues need slices to work with: with 64 per chunk (1 MiB chunks)
    //    six and seven workers still win (846-850 and 868 against 827 and 858 for four or eight) and five no longer do
    //    (817-831 against 823-829), with 16 per chunk all of them lose.
    const uint64_t slices_per_chunk = ((chunk_bytes & ~63ull) + slice_bytes - 1) / slice_bytes;
    const uint64_t sms = (uint64_t)sm_count;
    uint64_t warps = (100 * groups >= 645 * sms) ? MAX_WARPS : 4;
    if (slices_per_chunk >= 64) {
        if (slices_per_chunk >= 128 && groups >= 5 * sms && groups < 6 * sms) warps = 5;
        if (groups >= 6 * sms && groups < 7 * sms) warps = 6;
        else if (groups >= 7 * sms && 100 * groups < 725 * sms) warps = 7;
    }
    // From twelve groups per SM on, three warps per scheduler hide the longer chains of multiply-add
    // additions, which take a tenth of the ALU pipe's load: 917 GB/s against 884 (32 GiB in 64 KiB chunks).
    if (groups >= (uint64_t)MANY_WARPS * (uint64_t)sm_count) {
        t_instance = "12 workers per SM";
        kernel_many<<<(unsigned)sm_count, 32 * MANY_WARPS, MANY_WARPS * many_per_warp + smem_pad, stream>>>(
            map, d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, slice_bytes, total_tasks, groups, slot0, slot1, q,
            next_slice, mid, d_one);
        return cudaGetLastError();
    }
    static const char *const names[9] = {"", "", "", "", "4 workers per SM", "5 workers per SM", "6 workers per SM",
                                         "7 workers per SM", "8 workers per SM"};
    t_instance = names[warps];
    (warps > 4 && warps < 8 ? kernel_lag : kernel)<<<(unsigned)sm_count, (unsigned)(32 * warps), warps * smem_per_warp + smem_pad, stream>>>(
        map, d_data, nbytes, chunk_bytes, n_chunks, d_digests, d_status, slice_bytes, total_tasks, groups, slot0, slot1, q, next_slice,
        mid, d_one);
    return cudaGetLastError();
}

}  // namespace

const char *sliced_instance_name() { return t_instance; }

// Returns in *covered how many chunks (from the front of the blob) the launch hashes: only whole chunks can be
// described to the TMA unit, so a short last chunk is left to the caller (*covered = n - 1), and so is the
// whole blob (*covered = 0, nothing launched) if the tensor map cannot be made.
cudaError_t launch_hash_chunks_sliced(const uint8_t *d_data, uint64_t nbytes, uint64_t chunk_bytes,
                                      uint64_t n_chunks, uint8_t *d_digests, uint32_t *d_status, void *d_scratch,
                                      const uint32_t *d_one, int sm_count, cudaStream_t stream, uint64_t *covered,
                                      bool zero_prefix) {
    const uint64_t whole = nbytes / chunk_bytes;          // n_chunks or n_chunks - 1
    alignas(64) CUtensorMap map;
    std::memset(&map, 0, sizeof map);
    *covered = 0;
    if (whole == 0 || !make_chunk_tensor_map(&map, d_data, chunk_bytes, whole)) return cudaSuccess;
    *covered = whole;
    const uint64_t bytes = whole * chunk_bytes;
    return zero_prefix ? launch_sliced<true>(map, d_data, bytes, chunk_bytes, whole, d_digests, d_status, d_scratch, d_one,
                                             sm_count, stream)
                       : launch_sliced<false>(map, d_data, bytes, chunk_bytes, whole, d_digests, d_status, d_scratch, d_one,
                                              sm_count, stream);
}

}  // namespace ivk
