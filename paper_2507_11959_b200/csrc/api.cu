// Host-only entry points: status strings, size helpers, the launch counter.
#include "common.cuh"
#include "layout.cuh"
#include "sync.cuh"

using namespace pot;

// ---- device error words: one per kernel family, one definition for the whole library --------------------
// In host code the array's name is only a handle for the runtime; its device address is looked up per GPU.
static __device__ int g_error_words[3];

namespace pot {
int* error_ptr(int which) {
    static std::atomic<int*> cache[64];
    int dev = 0;
    if (which < 0 || which > 2 || cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    int* p = cache[dev].load(std::memory_order_acquire);
    if (!p) {
        void* q = nullptr;
        if (cudaGetSymbolAddress(&q, g_error_words) != cudaSuccess) return nullptr;
        p = (int*)q;
        cache[dev].store(p, std::memory_order_release);
    }
    return p + which;
}
int error_fetch(int which) {
    int v = -1, zero = 0;
    if (which < 0 || which > 2) return -1;
    if (cudaMemcpyFromSymbol(&v, g_error_words, sizeof(int), which * sizeof(int)) != cudaSuccess) return -1;
    cudaMemcpyToSymbol(g_error_words, &zero, sizeof(int), which * sizeof(int));
    return v;
}
}  // namespace pot

extern "C" int pot_debug_gemv_error(void) { return error_fetch(ERR_GEMV); }
extern "C" int pot_debug_gemm_error(void) { return error_fetch(ERR_GEMM); }
extern "C" int pot_debug_prefill_error(void) { return error_fetch(ERR_PREFILL); }

extern "C" const char* pot_status_string(pot_status_t s) {
    switch (s) {
        case POT_OK: return "ok";
        case POT_ERR_NULL: return "a required pointer is NULL";
        case POT_ERR_UNSUPPORTED: return "unsupported bits / group size / enum value";
        case POT_ERR_SHAPE: return "invalid shape (N, M > 0; K % 128 == 0; K % group == 0; tiled layout needs N % 16 == 0)";
        case POT_ERR_ALIGN: return "a base pointer is not 16-byte aligned";
        case POT_ERR_WORKSPACE: return "workspace missing or too small";
        case POT_ERR_SCALE_RANGE: return "a scale is outside the legal range";
        case POT_ERR_CUDA: return "CUDA launch failed";
    }
    return "unknown status";
}

extern "C" size_t pot_packed_bytes(int64_t N, int64_t K, int bits) {
    if (N <= 0 || K <= 0 || bits < 2 || bits > 4 || K % 128 != 0) return 0;
    return (size_t)N * (size_t)K * (size_t)bits / 8;
}

extern "C" size_t pot_scales_bytes(int64_t N, int64_t K, int group) {
    if (N <= 0 || K <= 0 || (group != 64 && group != 128) || K % group != 0) return 0;
    return (size_t)N * (size_t)(K / group) * 2;
}

extern "C" uint64_t pot_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

// Host-side view of the tiled layout's bit map (used by tools and tests that want to build or
// inspect tiled buffers without a GPU): where bit b of code q of a 128-code record is stored.
extern "C" pot_status_t pot_layout_bit(int bits, int kind, int q, int b, int* word, int* bit) {
    if (!word || !bit) return POT_ERR_NULL;
    if (bits < 2 || bits > 4 || kind < 0 || kind > 1) return POT_ERR_UNSUPPORTED;
    if (q < 0 || q >= 128 || b < 0 || b >= bits) return POT_ERR_SHAPE;
    const potl::BitPos p = potl::record_bit(bits, kind, q, b);
    *word = p.word;
    *bit = p.bit;
    return POT_OK;
}
