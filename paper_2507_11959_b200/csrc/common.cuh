// Shared host/device helpers of the PoT library: argument checks, launch bookkeeping,
// canonical-layout field extraction.
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "../../include/pot.h"

namespace pot {

extern std::atomic<uint64_t> g_launches;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline pot_status_t check_shape(int64_t N, int64_t K, int bits, int group) {
    if (bits < 2 || bits > 4) return POT_ERR_UNSUPPORTED;
    if (group != 64 && group != 128) return POT_ERR_UNSUPPORTED;
    if (N <= 0 || K <= 0) return POT_ERR_SHAPE;
    if (K % 128 != 0 || K % group != 0) return POT_ERR_SHAPE;
    if (N > (int64_t(1) << 31) || K > (int64_t(1) << 31)) return POT_ERR_SHAPE;
    return POT_OK;
}

// Call after a kernel launch: counts it and maps a launch error to a status.
inline pot_status_t launched(int n = 1) {
    g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? POT_OK : POT_ERR_CUDA;
}

constexpr int kSmCount = 148;  // B200: 2 dies x 74 SMs

#ifdef __CUDACC__
// Launch with programmatic stream serialization: the kernel may start while the previous kernel
// in the stream is still draining; it must execute griddepcontrol.wait before touching anything
// the previous kernel wrote (and before writing anything the previous kernel may still read).
// Largest dynamic shared memory a CTA may ask for on sm_100a.  Kernels opt in to this maximum rather than to the
// size of the current launch: a launch recorded in a CUDA graph must still fit the function's attribute when the
// graph is replayed, whatever other shapes were launched in between.
constexpr int kMaxDynamicSmem = 227 * 1024;
template <typename K>
inline bool allow_max_dynamic_smem(K kernel) {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kernel) != cudaSuccess) return false;
    const int room = kMaxDynamicSmem - (int)fa.sharedSizeBytes;  // static shared memory counts against the same limit
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess)
        return false;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, room) == cudaSuccess;
}

template <typename... Args>
inline pot_status_t launch_pdl(void (*kernel)(Args...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, args...);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return e == cudaSuccess ? POT_OK : POT_ERR_CUDA;
}
#endif

#ifdef __CUDACC__
__host__ __device__ constexpr int qmax_of(int bits) { return (1 << (bits - 1)) - 1; }

// Read `nbits` (<= 32) bits starting at bit offset `bitoff` of a little-endian bit stream whose
// 32-bit words are `p` (4-byte aligned).  The second word is read only when the field spills.
__device__ __forceinline__ uint32_t read_bits(const uint32_t* __restrict__ p, int64_t bitoff, int nbits) {
    const int64_t w = bitoff >> 5;
    const int sh = (int)(bitoff & 31);
    uint32_t lo = __ldg(p + w);
    uint32_t hi = (sh + nbits > 32) ? __ldg(p + w + 1) : 0u;
    uint32_t v = __funnelshift_r(lo, hi, sh);
    return nbits == 32 ? v : (v & ((1u << nbits) - 1u));
}

// Sec. 4.2, stage 1 on one canonical code c = sign << (n-1) | E:
//   exponent bits by AND mask, sign moved to the top, OR  ->  [S | 0.. E] as a 6-bit word,
//   aligned so that E sits at bit `ebit` (10 for FP16, 7 for BF16) and the sign at bit 15.
template <int BITS>
__device__ __forceinline__ uint32_t signed_exponent(uint32_t c, int ebit) {
    const uint32_t e = (c & (uint32_t)qmax_of(BITS)) << ebit;
    const uint32_t s = (c << (16 - BITS)) & 0x8000u;
    return e | s;
}

// Checked build (-DPOT_CHECKED): device-side index checks in front of stores, atomics and the streaming kernels'
// shared-memory reads.  A failed check records `code` in the kernel family's error word (first failure wins) and the
// access is skipped; nothing traps.  In the normal build the checks compile to nothing.
#ifdef POT_CHECKED
__device__ __forceinline__ bool in_range(bool ok, int* err, int code) {
    if (!ok && err) atomicCAS(err, 0, code);
    return ok;
}
#else
__device__ __forceinline__ bool in_range(bool, int*, int) { return true; }
#endif

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// 16-byte load of data that the previous kernel in the stream may have written (activations, mostly).  Such data is
// NOT read-only for the lifetime of a kernel that was launched early, so it must never go through the non-coherent
// path (__ldg / ld.global.nc): the compiler may move those loads ahead of griddepcontrol.wait, and a load that was
// moved returned the previous content of the buffer.  This one stays where it is written and reads through L2.
__device__ __forceinline__ uint4 ld_dependent16(const void* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

}  // namespace pot
