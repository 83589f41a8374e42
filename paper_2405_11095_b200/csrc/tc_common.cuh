// tcgen05 / mbarrier helpers shared by the two tensor-core decoder kernels (sm_100a).
#pragma once
#include "common.cuh"

namespace fosgd {

// shared-memory matrix descriptor, no swizzle: start address, leading and stride byte offsets in
// units of 16 bytes, descriptor version 1.  K-major operand: leading = bytes between core matrices
// (8 rows x 16 bytes) along K, stride = between groups of eight rows; MN-major operand: leading =
// bytes between groups of eight K-rows, stride = between 16-byte column groups.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | ((uint64_t)1 << 46);
}

__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// the barrier completes one arrival when every product this thread has issued so far is done
__device__ __forceinline__ void umma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Bounded wait that also gives up when the block's stop word is raised.  Plain polling: with a suspend-time
// hint of 20 microseconds on the try, the contiguous pass took 0.49 instead of 0.36 ms (sleeping warps wake
// up late).
__device__ __forceinline__ bool mbar_wait_or_stop(uint64_t* bar, uint32_t parity, const volatile int* stop)
{
    for (int it = 0; it < (1 << 22); ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
        if (done) return true;
        if ((it & 255) == 255 && *stop) return false;
    }
    return false;
}

// 32 consecutive accumulator columns of this thread's lane.  The load is asynchronous: it and its wait
// are one statement, so that the compiler never sees the destination registers as live while the load is
// still in flight (a version that started the load earlier, underneath the staging of the next item, had
// them spilled in between and returned stale values).
__device__ __forceinline__ void tmem_load32(uint32_t taddr, uint32_t (&u)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]),
          "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]),
          "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]),
          "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
        : "r"(taddr) : "memory");
}

}  // namespace fosgd
