// Device-side primitives shared by the streaming kernels of libbcq: compile-time loops, mbarrier
// operations with bounded waits, and bulk asynchronous copies into shared memory.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

namespace bcq {

constexpr int kSpinLimit = 1 << 22;   // polls per wait, about 32 ns apart: a wait gives up after roughly 0.2 s

template <int I, int N, class F>
__device__ __forceinline__ void static_for(F &&f)
{
    if constexpr (I < N) {
        f(std::integral_constant<int, I>{});
        static_for<I + 1, N>(f);
    }
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }

// ---- mbarrier / bulk-copy primitives ------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
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
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)   // never blocks
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the block is aborting (this wait or another one ran out); the wait
// that runs out raises the block's abort flag and records its code in the kernel's device status word.
// Polls without blocking and naps in between (a warp suspended inside a blocking try_wait was seen to
// resume only about a microsecond after the phase had completed).  LONG waits -- those that normally
// last microseconds -- lengthen their naps up to 256 ns, so that waiting warps leave the issue slots
// to the working ones; the time limit is about the same either way.
template <bool LONG = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int code, int *status_word)
{
    for (int it = 0; it < (LONG ? kSpinLimit / 4 : kSpinLimit); ++it) {
        if (mbar_test_wait(bar, parity)) return true;
        if (LONG && it >= 8)
            __nanosleep(256);
        else
            __nanosleep(32);
        if ((it & 255) == 255 && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(status_word, code);
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void named_barrier(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

}  // namespace bcq
