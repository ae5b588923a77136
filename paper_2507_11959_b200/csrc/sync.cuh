// mbarrier / bulk-copy primitives shared by the streaming kernels, and the library's device error words.
//
// Every wait on an mbarrier is bounded: after kSpinLimit unsuccessful polls the waiter gives up, records a
// code in its kernel family's error word and carries on without the data, so a lost copy cannot hang the GPU.
#pragma once
#include "common.cuh"

namespace pot {

constexpr uint32_t kSpinLimit = 1u << 22;

// One device error word per kernel family, defined once in api.cu.  error_ptr() returns this GPU's address of
// the word (nullptr if the runtime cannot tell); error_fetch() reads and clears it (synchronises the device,
// -1 if it cannot be read).
enum ErrorWord { ERR_GEMV = 0, ERR_GEMM = 1, ERR_PREFILL = 2 };
int* error_ptr(int which);
int error_fetch(int which);

#ifdef __CUDACC__
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_inval(uint32_t bar) {
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// bounded wait: false after kSpinLimit unsuccessful polls
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}
// one non-blocking test (1 = the phase with this parity has completed)
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done;
}
// bounded wait that polls with the non-blocking test_wait: a waiter parked inside try_wait can take on the
// order of a microsecond to resume, which is too slow for hand-offs that happen every few hundred cycles
__device__ __forceinline__ bool mbar_wait_spin(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_test(bar, parity)) return true;
    return false;
}
// 1-D bulk copy global -> shared; both addresses 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
#endif

}  // namespace pot
