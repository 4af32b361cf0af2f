// The FIFO of (group, slice) tasks that the migrating leaf kernels share: a ticket counter for the
// workers, a ticket counter for the pushes, and one slot per ticket that holds the group pushed under
// it.  A group is in the FIFO at most once, so its slices run in order.
#pragma once
#include <cstdint>

namespace ivk {
namespace {

struct SliceQueue {
    unsigned long long head;   // next ticket to hand to a worker
    unsigned long long tail;   // next ticket a finished slice pushes its group under
};

// slot[t] = group + 1 once ticket t has been pushed, 0 before.  The first `groups` tickets are
// pre-filled with the groups in order; every group starts at slice 0.
__global__ void slice_queue_init(uint32_t *__restrict__ slot, uint64_t total_tasks, uint64_t groups,
                                 SliceQueue *__restrict__ q, uint32_t *__restrict__ next_slice) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total_tasks; i += stride)
        slot[i] = i < groups ? (uint32_t)i + 1u : 0u;
    for (uint64_t g = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += stride) next_slice[g] = 0u;
    if (blockIdx.x == 0 && threadIdx.x == 0) { q->head = 0ull; q->tail = groups; }
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t *p, uint32_t v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// A scheduler's second worker takes a task only when one lies in the FIFO unclaimed: the first
// workers (one per scheduler) are served first, so no scheduler idles while another runs two
// groups.  With nothing left over it polls; giving up (the return value total_tasks ends the
// worker) is harmless, the first workers finish the launch.  Kept out of line so that the hashing
// loop's register allocation does not depend on it.
// `rank` orders the leftover workers of a CTA (0 = the first of them): a higher rank starts later and polls less
// often, so that unclaimed work goes to the CTAs with the fewest busy workers first.
__device__ __noinline__ unsigned long long take_leftover_ticket(SliceQueue *q, unsigned long long total_tasks,
                                                                bool first_take, unsigned rank = 0) {
    if (first_take) __nanosleep(20000u + 5000u * rank);      // at launch, let the first workers of every CTA claim their groups
    const unsigned poll_ns = 256u << (rank < 4u ? rank : 4u);
    const long long t0 = clock64();
    for (;;) {
        const unsigned long long h = *reinterpret_cast<volatile unsigned long long *>(&q->head);
        if (h >= total_tasks) return total_tasks;
        const unsigned long long tl = *reinterpret_cast<volatile unsigned long long *>(&q->tail);
        if (tl > h) {
            if (atomicCAS(&q->head, h, h + 1ull) == h) return h;
            continue;
        }
        if (clock64() - t0 > 8000000000ll) return total_tasks;
        __nanosleep(poll_ns);
    }
}

}  // namespace
}  // namespace ivk
