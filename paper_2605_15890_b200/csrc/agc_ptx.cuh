// Inline-PTX wrappers shared by the kernels: mbarriers with bounded waits, TMA tensor
// loads and untiled bulk copies into shared memory.
#pragma once
#include <cuda.h>

#include <cstdint>

namespace {

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
// One try. POLL = false: the try may suspend the warp for a while until the barrier's
// state changes (every transaction that lands wakes it); POLL = true: a test that returns at
// once, so that the caller's sleep alone sets how often a waiting warp takes an issue slot.
template <bool POLL = false>
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    if constexpr (POLL) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity), "r"(20000u) : "memory");
    }
    return ok != 0;
}
// Bounded wait. A warp that finds the phase incomplete sleeps between tries (32 ns doubling
// up to MAX_SLEEP_NS) instead of spinning, so that it does not take issue slots from the
// warps still working; a producer warp, whose wake-up delay adds to the refill latency of a
// ring stage, uses a shorter cap. After 2^22 tries (about a second with a cap of 256 ns,
// two with 512 ns) it gives up, records it and lets the caller unwind.
template <uint32_t MAX_SLEEP_NS, bool POLL = false>
__device__ __forceinline__ bool mbar_wait_loop(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    uint32_t ns = 32u;
    for (uint32_t spin = 0; spin < (1u << 22); ++spin) {
        __nanosleep(ns);
        if (mbar_try_wait<POLL>(bar, parity)) return true;
        if (ns < MAX_SLEEP_NS) ns <<= 1;
        else if (*abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
template <uint32_t MAX_SLEEP_NS, bool POLL = false>
__device__ __noinline__ bool mbar_wait_slow(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    return mbar_wait_loop<MAX_SLEEP_NS, POLL>(bar, parity, abort_flag);
}
// OUT_OF_LINE keeps the retry loop out of the caller's instruction stream (measured: better
// for the decoder's consumers, worse for the encoder's). POLL: see mbar_try_wait (measured:
// better for both roles of the encoder, no gain for the decoder).
template <uint32_t MAX_SLEEP_NS = 512u, bool OUT_OF_LINE = true, bool POLL = false>
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try_wait<POLL>(bar, parity)) return true;
    if constexpr (OUT_OF_LINE) return mbar_wait_slow<MAX_SLEEP_NS, POLL>(bar, parity, abort_flag);
    else return mbar_wait_loop<MAX_SLEEP_NS, POLL>(bar, parity, abort_flag);
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_addr(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int x, int y, int z, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_addr(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_addr(bar)) : "memory");
}

// Untiled bulk copy global -> shared; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

}  // namespace
