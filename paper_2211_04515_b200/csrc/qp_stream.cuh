// Streaming a contiguous, 16-byte aligned global array through shared memory with the
// bulk asynchronous copy engine (cp.async.bulk + mbarrier), for the HBM-bound reduction
// kernels.  One elected thread keeps STAGES tiles in flight per block, so the bytes in
// flight do not depend on how the consumers interleave loads and arithmetic.
//
//   - a persistent block takes tiles  first, first+step, first+2*step, ...
//   - stage s of the ring is filled by one bulk copy that completes on mbarrier full[s]
//   - every thread waits on full[s] (bounded), consumes the tile from shared memory, and a
//     block barrier hands the stage back to the producer
//
// Every wait is bounded: if a tile does not arrive within the wait limit (QP_STREAM_TIMEOUT_CYCLES
// unless the context was given another one) the block raises QP_DEV_STREAM_TIMEOUT in the status
// word, stops issuing copies, gives the copies still in flight a second bounded wait (always
// QP_STREAM_TIMEOUT_CYCLES) and returns, so the context stays usable.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "quantpipe.h"                                        // QP_DEV_STREAM_TIMEOUT

constexpr long long QP_STREAM_TIMEOUT_CYCLES = 4000000000ll;  // about two seconds

namespace qp_stream {

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_inval(uint64_t* bar)
{
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// make the barrier initialisation visible to the asynchronous proxy
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}

// global -> this block's shared memory; src, dst and bytes are multiples of 16
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst)),
                 "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// non-blocking form: has the phase with this parity completed?
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait; false on timeout.  limit = 0 does not wait at all: one non-blocking look
// (try_wait may itself suspend the thread for a while, so it is not used then).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity, long long limit = QP_STREAM_TIMEOUT_CYCLES)
{
    if (limit <= 0) return mbar_test_wait(bar, parity);
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
    }
    return true;
}

// Shared-memory footprint of a ring (bytes, incl. barriers), for the dynamic allocation.
template <int TILE_BYTES, int STAGES>
__host__ __device__ constexpr size_t ring_bytes() { return (size_t)TILE_BYTES * STAGES + 8 * STAGES + 16; }

// Streams tiles [0, ntiles) of TILE_BYTES each, starting at `base` (16-byte aligned), to
// consume(tile_pointer_in_shared_memory, tile_index), called by every thread of the block.
// Block b takes tiles b, b + gridDim.x, ...; with `reverse` the tile order is mirrored
// (tile ntiles-1-t), which lets a pass that follows another one start on the part of the
// array most recently left in L2.  `smem` is the block's dynamic shared memory, 128-byte
// aligned, ring_bytes() long.  Returns false if a wait timed out (status bit raised).
template <int TILE_BYTES, int STAGES, typename F>
__device__ __forceinline__ bool for_each_tile(const unsigned char* __restrict__ base, uint64_t ntiles, bool reverse,
                                              unsigned char* smem, unsigned* status, long long wait_limit, F&& consume)
{
    static_assert(TILE_BYTES % 128 == 0, "tile size");
    unsigned char* buf = smem;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)TILE_BYTES * STAGES);
    __shared__ int timed_out;

    const uint64_t first = blockIdx.x, step = gridDim.x;
    const uint64_t mine = first < ntiles ? (ntiles - first + step - 1) / step : 0;   // tiles of this block
    auto tile_of = [&](uint64_t i) {
        const uint64_t t = first + i * step;
        return reverse ? ntiles - 1 - t : t;
    };
    if (threadIdx.x == 0) {
        timed_out = 0;
        for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (uint64_t i = 0; i < (uint64_t)STAGES && i < mine; ++i) {
            mbar_arrive_expect_tx(&full[i], TILE_BYTES);
            bulk_load(buf + i * TILE_BYTES, base + tile_of(i) * TILE_BYTES, TILE_BYTES, &full[i]);
        }
    }
    uint64_t issued = mine < (uint64_t)STAGES ? mine : (uint64_t)STAGES;   // meaningful in thread 0 only
    uint64_t done = 0;
    bool ok = true;
    for (uint64_t i = 0; i < mine; ++i) {
        const int s = (int)(i % STAGES);
        const unsigned parity = (unsigned)((i / STAGES) & 1);
        if (!mbar_wait(&full[s], parity, wait_limit)) timed_out = 1;   // benign race: every writer writes 1
        __syncthreads();
        if (timed_out) { ok = false; break; }
        consume(buf + (size_t)s * TILE_BYTES, tile_of(i));
        __syncthreads();                                          // stage s is free again
        done = i + 1;
        if (threadIdx.x == 0 && issued < mine) {
            mbar_arrive_expect_tx(&full[s], TILE_BYTES);
            bulk_load(buf + (size_t)s * TILE_BYTES, base + tile_of(issued) * TILE_BYTES, TILE_BYTES, &full[s]);
            ++issued;
        }
    }
    if (!ok) {
        // copies issued but not consumed may still be landing in this block's shared memory:
        // give each a second bounded wait before the block may exit
        if (threadIdx.x == 0) {
            atomicOr(status, QP_DEV_STREAM_TIMEOUT);
            for (uint64_t i = done; i < issued; ++i) mbar_wait(&full[i % STAGES], (unsigned)((i / STAGES) & 1));
        }
        __syncthreads();
    }
    __syncthreads();
    if (threadIdx.x == 0)
        for (int s = 0; s < STAGES; ++s) mbar_inval(&full[s]);
    return ok;
}

// The same ring as an object, for kernels that make more than one pass with it and want the
// tiles of the last pass to stay in shared memory: stage s is filled by issue() (one thread),
// every thread waits for it with wait(), and the caller's block barrier hands a stage back.
// The parity expected at the next wait of each stage is tracked in a bit mask that every
// thread keeps alike.
template <int TILE_BYTES, int STAGES>
struct ring {
    static_assert(TILE_BYTES % 128 == 0 && STAGES <= 32, "ring shape");
    unsigned char* buf;
    uint64_t* full;
    unsigned parity;                                    // bit s: parity of the next completion of stage s

    __device__ __forceinline__ void init(unsigned char* smem)      // all threads; ends with a block barrier
    {
        buf = smem;
        full = reinterpret_cast<uint64_t*>(smem + (size_t)TILE_BYTES * STAGES);
        parity = 0u;
        if (threadIdx.x == 0) {
            for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
            fence_barrier_init();
        }
        __syncthreads();
    }
    __device__ __forceinline__ unsigned char* stage(int s) const { return buf + (size_t)s * TILE_BYTES; }
    __device__ __forceinline__ void issue(int s, const unsigned char* src)          // one thread
    {
        mbar_arrive_expect_tx(&full[s], TILE_BYTES);
        bulk_load(stage(s), src, TILE_BYTES, &full[s]);
    }
    // all threads; false when the wait ran out (the parity bit is then left as it was)
    __device__ __forceinline__ bool wait(int s, long long limit)
    {
        if (!mbar_wait(&full[s], (parity >> s) & 1u, limit)) return false;
        parity ^= 1u << s;
        return true;
    }
    __device__ __forceinline__ void fini()                                          // after a block barrier
    {
        if (threadIdx.x == 0)
            for (int s = 0; s < STAGES; ++s) mbar_inval(&full[s]);
    }
};

// A ring per WARP: every warp of the block streams its own sequence of tiles through its own
// stages and barriers, so the tile loop holds no block barrier at all (a block-wide ring hands a
// stage back through __syncthreads twice per tile, and with a few dozen instructions of work per
// thread and tile the warps spend more time at that barrier than on the data).  Lane 0 issues the
// warp's copies; all lanes wait (the outcome is made uniform with a vote) and __syncwarp hands a
// stage back.  All lanes keep `parity` and `pending` alike.
template <int TILE_BYTES, int STAGES>
struct warp_ring {
    static_assert(TILE_BYTES % 128 == 0 && STAGES <= 32, "ring shape");
    unsigned char* buf;
    uint64_t* full;
    unsigned parity;                                    // bit s: parity of the next completion of stage s
    unsigned pending;                                   // bit s: a copy into stage s is in flight

    static __host__ __device__ constexpr size_t bytes(int warps) { return (size_t)warps * STAGES * (TILE_BYTES + 8); }

    // all threads of the block; smem: 128-byte aligned, bytes(warps) long; ends with a block barrier
    __device__ __forceinline__ void init(unsigned char* smem, int warps)
    {
        const int warp = threadIdx.x >> 5;
        buf = smem + (size_t)warp * STAGES * TILE_BYTES;
        full = reinterpret_cast<uint64_t*>(smem + (size_t)warps * STAGES * TILE_BYTES) + warp * STAGES;
        parity = 0u;
        pending = 0u;
        if ((threadIdx.x & 31) == 0) {
            for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
            fence_barrier_init();
        }
        __syncthreads();
    }
    __device__ __forceinline__ const unsigned char* stage(int s) const { return buf + (size_t)s * TILE_BYTES; }
    // all lanes (lane 0 copies); the stage's earlier contents must have been read (__syncwarp before)
    __device__ __forceinline__ void issue(int s, const unsigned char* src)
    {
        if ((threadIdx.x & 31) == 0) {
            mbar_arrive_expect_tx(&full[s], TILE_BYTES);
            bulk_load(buf + (size_t)s * TILE_BYTES, src, TILE_BYTES, &full[s]);
        }
        pending |= 1u << s;
    }
    // all lanes; false for the whole warp when any lane's wait ran out (the state is then left as it was)
    __device__ __forceinline__ bool wait(int s, long long limit)
    {
        const bool ok = mbar_wait(&full[s], (parity >> s) & 1u, limit);
        if (!__all_sync(0xFFFFFFFFu, ok)) return false;
        parity ^= 1u << s;
        pending &= ~(1u << s);
        return true;
    }
    // all lanes: a second, bounded wait for every copy still in flight (after a failed wait)
    __device__ __forceinline__ void drain()
    {
        if ((threadIdx.x & 31) == 0)
            for (int s = 0; s < STAGES; ++s)
                if (pending & (1u << s)) mbar_wait(&full[s], (parity >> s) & 1u, QP_STREAM_TIMEOUT_CYCLES);
        pending = 0u;
        __syncwarp();
    }
    __device__ __forceinline__ void fini()                                          // after a block barrier
    {
        if ((threadIdx.x & 31) == 0)
            for (int s = 0; s < STAGES; ++s) mbar_inval(&full[s]);
    }
};

}  // namespace qp_stream
