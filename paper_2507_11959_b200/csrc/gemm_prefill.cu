// Prefill GEMM (large M): placeholder until the tcgen05 kernel lands.
#include "common.cuh"

namespace pot {
bool gemm_prefill_supported(int64_t, int64_t, int64_t, int, int) { return false; }
size_t gemm_prefill_workspace(int64_t, int64_t, int64_t, int, int) { return 0; }
pot_status_t gemm_prefill_launch(const void*, const void*, int64_t, int64_t, int, int, const void*, int64_t, void*,
                                 void*, size_t, cudaStream_t) {
    return POT_ERR_UNSUPPORTED;
}
}  // namespace pot
