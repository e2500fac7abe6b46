// Thin inline-PTX layer for the sm_100a kernels: mbarriers with bounded waits, TMA tile loads,
// tensor-memory allocation, tcgen05 MMA issue / commit / accumulator loads, shared-memory matrix
// descriptors.  Nothing here knows about the method; it only names the hardware operations.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace alora {
namespace tc {

// A wait gives up after this many clock cycles (about one second).  The kernel then records
// ALORA_ERR_TIMEOUT, raises its block-wide abort flag and leaves through its normal exit path.
constexpr long long kWaitCycleLimit = 2000000000LL;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Adds to the bytes a barrier phase expects without arriving on it (a later arrive.expect_tx completes the count).
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Programmatic dependent launch.  A kernel launched with the programmatic-stream-serialization attribute may start
// while its predecessor in the stream is still running: grid_dep_wait() returns once the predecessor has completed
// and its writes are visible (it returns at once in a kernel launched the ordinary way), so everything before it
// may only touch this block's own shared and tensor memory.  Every block executes it before it exits.
// grid_dep_launch() lets the successor's blocks start as soon as all blocks of this kernel have called it.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// One lane of a converged warp (the same one every time); all 32 lanes must call it.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  `abort_flag` is a shared-memory word any role may set; once it is set every wait
// returns false at once.  Returns true when the barrier phase completed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          long long limit = kWaitCycleLimit) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            return false;
        }
    }
}

// The same bounded wait for a warp whose reaction time does not matter (a producer several ring slots ahead of
// its consumers): it sleeps between polls, leaving the issue slots of its scheduler to the warps that compute.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        __nanosleep(200);
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycleLimit) {
            *abort_flag = 1;
            return false;
        }
    }
}

// 2-D TMA tile load global -> shared, completion counted on an mbarrier.  c0 is the innermost
// coordinate (elements); c0 * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t smem_dst, const CUtensorMap *map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_dst), "l"((uint64_t)map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)map) : "memory");
}

// ---- tensor memory -----------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols) {  // one full warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {  // same warp that allocated
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor for a K-major bf16 tile written by TMA with 128-byte swizzle:
// rows are 128 bytes (64 elements) apart, groups of 8 rows are 1024 bytes apart (stride byte
// offset), the leading byte offset is unused for swizzled K-major tiles, descriptor version 1,
// layout type 2 (128-byte swizzle).  Advancing K by 16 elements adds 32 bytes to the start address.
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t smem_addr) {
    return (uint64_t)((smem_addr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]; issued by one thread.
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on an mbarrier once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Accumulator load: this warp's 32 lanes (rows) x 32 consecutive fp32 columns.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// A block's work items travel from the one thread that decides their order (its producer) to the block's other
// roles through a small ring in shared memory.  The producer may take items from a global counter: an item that
// waits for the result of another item (a projection item for its row tile's shrink item) is only started once
// every item it can wait for has been claimed, and a claimed item is on a block that is running, so no block ever
// depends on one that has not been scheduled yet, however few blocks are resident.
// Layout at `base` (shared memory): full[kItemSlots], empty[kItemSlots] barriers, then kItemSlots ints.
constexpr int kItemSlots = 4;
constexpr int kItemRingBytes = 16 * kItemSlots + 4 * kItemSlots;
struct ItemRing {
    uint32_t bar0;          // shared-memory address of full[0]
    volatile int *slots;
    uint32_t n = 0;         // items passed through this role so far
    __device__ __forceinline__ uint32_t full(int s) const { return bar0 + 8u * s; }
    __device__ __forceinline__ uint32_t empty(int s) const { return bar0 + 8u * (kItemSlots + s); }
    __device__ __forceinline__ void init(int n_consumers) const {   // one thread, before the block-wide sync
        for (int s = 0; s < kItemSlots; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), n_consumers); }
    }
    // producer (one thread): publish `item` (-1: the list is exhausted); false when a wait expired
    __device__ __forceinline__ bool put(int item, volatile int *abort_flag) {
        const int s = n % kItemSlots;
        if (!mbar_wait(empty(s), ((n / kItemSlots) & 1) ^ 1, abort_flag)) return false;
        slots[s] = item;
        mbar_arrive(full(s));
        ++n;
        return true;
    }
    // consumer (a whole warp): the next item, -1 at the end of the list, -2 when a wait expired
    __device__ __forceinline__ int take(volatile int *abort_flag) {
        const int s = n % kItemSlots;
        const bool got = __all_sync(0xffffffffu, mbar_wait(full(s), (n / kItemSlots) & 1, abort_flag));
        const int item = got ? slots[s] : -2;
        __syncwarp();
        if (got && (threadIdx.x & 31) == 0) mbar_arrive(empty(s));
        ++n;
        return item;
    }
};
// At the end of a kernel that hands items out through a global counter: the last block to get here clears
// the counter for the next launch.  counters[0] = next item, counters[1] = blocks that have finished.
__device__ __forceinline__ void item_counter_release(int32_t *counters) {
    __threadfence();
    if (atomicAdd(counters + 1, 1) == (int)gridDim.x - 1) {
        counters[0] = 0;
        counters[1] = 0;
        __threadfence();
    }
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

}  // namespace tc
}  // namespace alora
