// Grid-wide barrier for kernels launched cooperatively (all blocks co-resident): an arrival
// counter in global memory, release on arrival, acquire on the poll.  The wait is bounded all
// the same: a block that has polled `spin_limit` times without seeing `target` arrivals raises
// QP_DEV_STREAM_TIMEOUT in the status word and reports failure, so the kernel can leave and
// the context stays usable.  The counter must be zero when the launch starts and the kernel
// resets it when its last block leaves; after a time-out qp_get_status clears it.
#pragma once

#include <cuda_runtime.h>

#include "quantpipe.h"                                        // QP_DEV_STREAM_TIMEOUT

namespace qp_grid {

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void arrive_release(unsigned* p)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}

// All blocks arrive, then all leave.  The block's writes are ordered before the arrival by the
// block barrier and the release; the acquire load orders the other blocks' writes before what
// follows.  Returns false (for the whole block) when the wait ran out.  s_ok: one int of
// shared memory.
__device__ __forceinline__ bool barrier(unsigned* bar, unsigned target, unsigned spin_limit, unsigned* status, int* s_ok)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        arrive_release(bar);
        int ok = 1;
        unsigned spins = 0;
        while (ld_acquire(bar) < target) {
            if (++spins > spin_limit) {
                ok = 0;
                atomicOr(status, QP_DEV_STREAM_TIMEOUT);
                break;
            }
            if (spins > 64) __nanosleep(64);
        }
        *s_ok = ok;
    }
    __syncthreads();
    return *s_ok != 0;
}

}  // namespace qp_grid
