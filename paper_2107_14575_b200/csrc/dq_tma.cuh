// Asynchronous-copy plumbing for sm_100a: mbarriers, bulk copies (TMA) from
// global to shared memory, and the 128-byte swizzle that TMA tensor copies
// apply.  Every copy here is addressed to the issuing CTA alone.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dq.h"

// Host: encodes a tiled tensor map (the driver entry point is looked up at run
// time, so the library does not link against libcuda).  Returns false on failure.
bool dq_encode_tensor_map(CUtensorMap* map, CUtensorMapDataType type, uint32_t rank, const void* base,
                          const uint64_t* dims, const uint64_t* strides_bytes /*rank-1*/, const uint32_t* box,
                          CUtensorMapSwizzle swizzle);

// Limits of the waits for asynchronous copies; every kernel that waits receives them as part of
// its (constant-bank) arguments.  `ns` bounds every wait, in nanoseconds of the global timer (2 s
// unless dq_debug_set_wait_limits changed it).  `lose_first` is the test hook: when set, the FIRST
// wait of every consumer (a warp or a CTA, as the kernel is organised) is declared lost without a
// look at its barrier, while its copy is valid and lands a moment later -- the path taken after a
// time-out then runs with nothing actually lost.  The kernels look at the hook outside their tile
// loops (inside them it cost the quantizers 4 % of their time).  A wait that runs out raises DQ_STAT_WAIT, the
// CTA waits (with `ns`) for every copy it has issued, and leaves.
struct WaitLimits {
    unsigned long long ns;
    uint32_t lose_first;
    uint32_t reserved;
};
WaitLimits dq_wait_limits();     // host: the limits the next launches get

#ifdef __CUDACC__

namespace tma {

__device__ __forceinline__ uint32_t smem_addr(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

// Makes freshly initialised barriers visible to the asynchronous proxy.
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// Orders generic-proxy shared-memory accesses of this thread before later
// asynchronous-proxy accesses (a bulk copy that overwrites or reads them).
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}

// Plain arrival (one of the barrier's expected arrivals), with release semantics for the
// arriving thread's earlier shared-memory accesses.
__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Waits for the phase with the given parity; false if the limit ran out.  The limit is only read
// on the slow path, so that a wait that succeeds at once costs one instruction and no registers.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const WaitLimits& lim)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > lim.ns) return false;
    }
}
// 3-D tiled tensor copy global -> shared, completion counted on `bar`.
__device__ __forceinline__ void load_tile_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_addr(dst)), "l"(map), "r"(smem_addr(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// 2-D tiled tensor copy global -> shared (rows outside the tensor arrive as zeros and still
// count towards the barrier's bytes), completion counted on `bar`.
__device__ __forceinline__ void load_tile_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_addr(dst)), "l"(map), "r"(smem_addr(bar)), "r"(c0), "r"(c1)
        : "memory");
}

// L2 policy for data that is read once and should be the first to leave the cache.
__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// Same copy as load_tile_3d with an L2 cache policy attached to the global reads.
__device__ __forceinline__ void load_tile_3d_hint(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2,
                                                  uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(smem_addr(dst)), "l"(map), "r"(smem_addr(bar)), "r"(c0), "r"(c1), "r"(c2), "l"(policy)
        : "memory");
}

// Linear bulk copy global -> shared; addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void load_bulk(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// 2-D tiled tensor copy shared -> global (rows outside the tensor are clipped), tracked
// by the thread's bulk-async group.
__device__ __forceinline__ void store_tile_2d(const CUtensorMap* map, const void* src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(smem_addr(src)), "r"(c0), "r"(c1)
                 : "memory");
}

__device__ __forceinline__ void store_commit()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// Blocks until every committed bulk store of this thread has finished reading shared memory.
__device__ __forceinline__ void store_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

__device__ __forceinline__ void prefetch_tensor_map(const CUtensorMap* map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// Byte offset inside a tile of 128-byte rows written with the 128-byte swizzle:
// the 16-byte chunk index is xor-ed with the row index modulo 8.  The tile
// must start on a 1024-byte boundary.
__device__ __forceinline__ uint32_t swizzle128(uint32_t row, uint32_t chunk)
{
    return row * 128u + ((chunk ^ (row & 7u)) << 4);
}

}  // namespace tma

#endif  // __CUDACC__
