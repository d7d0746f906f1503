// PTX wrappers shared by the kernels: mbarrier, TMA (bulk tensor and plain bulk copies)
// and the bounded wait every spin in this library goes through.
#pragma once
#include <cuda.h>
#include <stdint.h>

#include "bd_common.cuh"

namespace bd {

// Device status word, read and cleared by bd_poll_status (bits: kStatusNonfinite, kStatusTimeout).
__device__ uint32_t g_status_word = 0;
// Test hooks (bd_debug_fault): a lower poll limit for the bounded waits (0 = the built-in one) and "the code
// producer of the tensor-core product leaves out its very first stage", which makes a wait run out on purpose.
__device__ uint32_t g_debug_spin_limit = 0;
__device__ uint32_t g_debug_skip_first_code_stage = 0;

namespace tc {

constexpr uint32_t kSpinLimit = 1u << 24;   // polls; with the sleeps below roughly a second

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Non-blocking probe of a phase (never suspends the thread).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  `abort_flag` (shared memory) is raised by the first wait that runs out;
// later waits return at once so that the CTA drains quickly.  After a few failed polls the
// warp sleeps between polls (`sleep_ns`), so that a long wait does not take issue slots
// from the warps that are working.  abort_flag[1] is the CTA's "earlier kernels of the stream
// have completed" word: while it is zero the polls are not counted, because the wait then
// includes the rest of the previous kernel, whose length is not this kernel's to bound (the
// warp that waits for that kernel does so in hardware, without a limit, and sets the word).
// abort_flag[2] is the poll limit of this launch (looked at every 1024 polls, like the abort word).
// Returns false when the CTA is aborting (this wait or an earlier one ran out), so that a caller
// in a hot loop need not read the flag again after every wait.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          uint32_t sleep_ns = 32) {
    for (uint32_t spin = 0; spin < kSpinLimit; spin++) {
        if (mbar_try_wait(bar, parity)) return true;
        if (spin >= 8) __nanosleep(sleep_ns);
        if ((spin & 1023u) == 1023u) {
            if (*abort_flag) return false;
            if (!abort_flag[1]) spin = 0;
            else if (spin >= abort_flag[2]) break;
        }
    }
    *abort_flag = 1;
    atomicOr(&g_status_word, kStatusTimeout);
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

}  // namespace tc
}  // namespace bd
