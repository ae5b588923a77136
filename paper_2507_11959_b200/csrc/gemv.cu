// Batch-1 decode GEMV, y = W~ x, fused with the dequantization (the weights never touch HBM as FP16).
//
//  * tiled layout (the fast path): the streaming kernel of stream.cuh.  Every warp streams its own contiguous
//    range of 16-row x 128-column units through a private shared-memory ring (bulk copies), decodes the codes in
//    registers with the mask / shift / integer-add of Sec. 4.2 and feeds them, as A fragments, to warp-level
//    tensor-core MMAs whose B columns all hold x; row blocks that span warps are combined in a fixed order.
//  * canonical layout (any N): a CUDA-core kernel, one warp per row, 8 codes per lane per step, products
//    accumulated in FP32 with the mixed-precision FMA and reduced across lanes with warp shuffles.
//
// Programmatic dependent launch: weights and scales do not depend on the previous kernel in the stream, x does.
// The kernels request their first weights before they execute griddepcontrol.wait, and touch x, y and the
// workspace only after it.
#include "common.cuh"
#include "layout.cuh"
#include "stream.cuh"

namespace pot {

// two FP16 x FP16 products accumulated in FP32 (mixed-precision FMA: no conversion instructions)
__device__ __forceinline__ void rg_fma2(float& acc0, float& acc1, uint32_t w2, uint32_t x2) {
    asm("{\n\t"
        ".reg .b16 wl, wh, xl, xh;\n\t"
        "mov.b32 {wl, wh}, %2;\n\t"
        "mov.b32 {xl, xh}, %3;\n\t"
        "fma.rn.f32.f16 %0, wl, xl, %0;\n\t"
        "fma.rn.f32.f16 %1, wh, xh, %1;\n\t"
        "}"
        : "+f"(acc0), "+f"(acc1)
        : "r"(w2), "r"(x2));
}


// ------------------------------------------------------------------------------------------
// canonical layout, one warp per row
// ------------------------------------------------------------------------------------------
// BF16 pairs: a BF16 number is the upper half of an FP32 pattern, so the conversions are a shift and a mask
__device__ __forceinline__ void rg_fma2_bf16(float& acc0, float& acc1, uint32_t w2, uint32_t x2) {
    acc0 = fmaf(__uint_as_float(w2 << 16), __uint_as_float(x2 << 16), acc0);
    acc1 = fmaf(__uint_as_float(w2 & 0xFFFF0000u), __uint_as_float(x2 & 0xFFFF0000u), acc1);
}

// DT = 0: FP16 activations / weights / output; DT = 1: BF16 (PoT only: scale rounded once to BF16, E added at bit 7)
template <int BITS, bool UNIFORM, int DT = 0>
__global__ void __launch_bounds__(256) gemv_canonical_kernel(const uint32_t* __restrict__ packed,
                                                             const uint16_t* __restrict__ scales,
                                                             const uint16_t* __restrict__ zeros, int64_t N, int64_t K,
                                                             int G, const uint4* __restrict__ x, uint16_t* __restrict__ y) {
    constexpr int EBIT = DT == 0 ? 10 : 7;
    constexpr uint32_t CM = (1u << BITS) - 1u;
    constexpr uint32_t QM2 = (uint32_t)qmax_of(BITS) * 0x10001u;
    constexpr uint32_t SM2 = (1u << (BITS - 1)) * 0x10001u;
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= N) return;
    const int64_t pieces = K / 8;
    const uint32_t* rowp = packed + row * (K * BITS / 32);
    const uint16_t* srow = scales + row * (K / G);
    const uint16_t* zrow = UNIFORM ? zeros + row * (K / G) : nullptr;
    float acc0 = 0.f, acc1 = 0.f;
    pdl_wait();
    for (int64_t c = lane; c < pieces; c += 32) {
        const uint32_t v = read_bits(rowp, c * (8 * BITS), 8 * BITS);
        uint32_t s16 = __ldg(srow + (c * 8) / G);
        if (DT == 1) s16 = __bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half((uint16_t)s16))));
        const uint4 xv = ld_dependent16(x + c);
        const uint32_t xs[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t t = v >> (2 * j * BITS);
            const uint32_t pr = (t & CM) | ((t << (16 - BITS)) & (CM << 16));
            uint32_t w2;
            if constexpr (!UNIFORM) {
                w2 = s16 * 0x10001u + (((pr & QM2) << EBIT) | ((pr & SM2) << (16 - BITS)));
            } else {
                const __half2 zm2 = __hadd2(__half2half2(__ushort_as_half(__ldg(zrow + (c * 8) / G))), __float2half2_rn(1024.0f));
                const uint32_t h = pr | 0x64006400u;
                const __half2 d = __hsub2(*reinterpret_cast<const __half2*>(&h), zm2);
                const __half2 w = __hmul2(d, __half2half2(__ushort_as_half((uint16_t)s16)));
                w2 = *reinterpret_cast<const uint32_t*>(&w);
            }
            if (DT == 0) rg_fma2(acc0, acc1, w2, xs[j]);
            else rg_fma2_bf16(acc0, acc1, w2, xs[j]);
        }
    }
    float acc = acc0 + acc1;
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) y[row] = sk_out<DT>(acc);
}

// CTAs per SM of the streaming GEMV (16 consumer warps each).  Two: the next launch in the stream becomes resident,
// sets itself up and fills its rings while this one computes, which hides the launch and the prologue (about 2.5 us);
// the price is 64 registers per thread and half the ring, i.e. a slower loop (about 15 %).  Worth it while a CTA's
// share of the matrix is small; one CTA per SM otherwise, and whenever the half-size ring could not hold two slots.
constexpr size_t kTwoCtaMaxShare = 300 * 1024;  // bytes of codes + scales per CTA
static int gemv_occupancy(int64_t N, int64_t K, int bits, int group, int kind) {
    const StreamPlan p2 = plan_stream(N, K, 1, bits, group, kind, 1, 16, 2);
    if (!p2.ok || !p2.x_in_smem || p2.ring_capacity < 2 || p2.grid < kSmCount) return 1;
    const size_t share = (size_t)(N / 16) * (size_t)(K / 128) * (size_t)sk_unit_total_bytes(bits, group, kind) / (size_t)p2.grid;
    return share <= kTwoCtaMaxShare ? 2 : 1;
}

template <int KIND, int DT = 0>
static pot_status_t launch_gemv_stream(const void* packed, const void* scales, const void* zeros, int64_t N, int64_t K,
                                       int bits, int group, const void* x, void* y, void* workspace, cudaStream_t s) {
    int* err = error_ptr(ERR_GEMV);
#define POT_SG(B, O) return launch_stream<B, KIND, 1, 16, O, DT>(packed, scales, zeros, N, K, group, x, 1, y, workspace, err, s)
    if (gemv_occupancy(N, K, bits, group, KIND) == 2) {
        if (bits == 2) POT_SG(2, 2);
        if (bits == 3) POT_SG(3, 2);
        POT_SG(4, 2);
    }
    if (bits == 2) POT_SG(2, 1);
    if (bits == 3) POT_SG(3, 1);
    POT_SG(4, 1);
#undef POT_SG
}

// the tiled FP16 / BF16 GEMV for pot_gemm's single-token case
pot_status_t gemv_stream_launch(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group, const void* x,
                                void* y, void* workspace, cudaStream_t s, int dt) {
    if (dt == 0) return launch_gemv_stream<SK_POT, 0>(packed, scales, nullptr, N, K, bits, group, x, y, workspace, s);
    return launch_gemv_stream<SK_POT, 1>(packed, scales, nullptr, N, K, bits, group, x, y, workspace, s);
}

static size_t gemv_stream_workspace(int64_t N, int64_t K, int bits, int group, int tok) {
    size_t need = 0;
    for (int occ : {1, 2}) {  // the partial-sum layout does not depend on the occupancy, the check is for safety
        const StreamPlan p = plan_stream(N, K, 1, bits, group, SK_UINT, tok, 16, occ);
        if (!p.ok) return 0;
        if (p.ws_bytes > need) need = p.ws_bytes;
    }
    return need;
}

}  // namespace pot

using namespace pot;

// Host arithmetic only: how pot_gemv / uint_gemv would run a tiled shape (tests assert which variants they reach).
extern "C" pot_status_t pot_debug_gemv_plan(int64_t N, int64_t K, int bits, int group, int uniform, int* ctas_per_sm,
                                            int* row_block_split, int* ring_slots, int* units_per_slot, int* x_in_smem) {
    if (!ctas_per_sm || !row_block_split || !ring_slots || !units_per_slot || !x_in_smem) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if (N % 16 != 0) return POT_ERR_SHAPE;
    const int kind = uniform ? SK_UINT : SK_POT;
    const int occ = gemv_occupancy(N, K, bits, group, kind);
    const StreamPlan p = plan_stream(N, K, 1, bits, group, kind, 1, 16, occ);
    if (!p.ok) return POT_ERR_SHAPE;
    *ctas_per_sm = occ;
    *row_block_split = p.aligned ? 1 : 0;
    *ring_slots = p.stages;
    *units_per_slot = p.q;
    *x_in_smem = p.x_in_smem ? 1 : 0;
    return POT_OK;
}

extern "C" size_t pot_gemv_workspace_bytes(int64_t N, int64_t K, int bits, int group) {
    if (check_shape(N, K, bits, group) != POT_OK || N % 16 != 0) return 0;
    return gemv_stream_workspace(N, K, bits, group, 1);  // row-block arrival counters + FP32 partial slots
}

// every argument check of pot_gemv, run before anything is enqueued (also by the wrappers that enqueue copies first)
static pot_status_t check_gemv_args(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                    pot_layout_t layout, const void* x, const void* y, const void* workspace, size_t ws_bytes) {
    if (!packed || !scales || !x || !y) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if (layout != POT_LAYOUT_CANONICAL && layout != POT_LAYOUT_TILED) return POT_ERR_UNSUPPORTED;
    if (!aligned16(packed) || !aligned16(scales) || !aligned16(x) || !aligned16(y) || !aligned16(workspace))
        return POT_ERR_ALIGN;
    if (layout == POT_LAYOUT_TILED) {
        if (N % 16 != 0) return POT_ERR_SHAPE;
        if (!plan_stream(N, K, 1, bits, group, SK_POT, 1, 16).ok) return POT_ERR_SHAPE;
        const size_t need = pot_gemv_workspace_bytes(N, K, bits, group);
        if (need > 0 && (!workspace || ws_bytes < need)) return POT_ERR_WORKSPACE;
    }
    return POT_OK;
}

template <int DT>
static pot_status_t gemv_impl(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                              pot_layout_t layout, const void* x, void* y, void* workspace, size_t ws_bytes, void* stream) {
    const pot_status_t st = check_gemv_args(packed, scales, N, K, bits, group, layout, x, y, workspace, ws_bytes);
    if (st != POT_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    if (layout == POT_LAYOUT_CANONICAL) {
        const dim3 grid((unsigned)((N + 7) / 8)), block(256);
        auto* P = (const uint32_t*)packed;
        auto* S = (const uint16_t*)scales;
        const uint16_t* Z = nullptr;
        if (bits == 2) return launch_pdl(gemv_canonical_kernel<2, false, DT>, grid, block, 0, s, P, S, Z, N, K, group, (const uint4*)x, (uint16_t*)y);
        if (bits == 3) return launch_pdl(gemv_canonical_kernel<3, false, DT>, grid, block, 0, s, P, S, Z, N, K, group, (const uint4*)x, (uint16_t*)y);
        return launch_pdl(gemv_canonical_kernel<4, false, DT>, grid, block, 0, s, P, S, Z, N, K, group, (const uint4*)x, (uint16_t*)y);
    }
    return launch_gemv_stream<SK_POT, DT>(packed, scales, nullptr, N, K, bits, group, x, y, workspace, s);
}

extern "C" pot_status_t pot_gemv(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                 pot_layout_t layout, const void* x, void* y, void* workspace, size_t ws_bytes,
                                 void* stream) {
    return gemv_impl<0>(packed, scales, N, K, bits, group, layout, x, y, workspace, ws_bytes, stream);
}

extern "C" pot_status_t pot_gemv_bf16(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                      pot_layout_t layout, const void* x, void* y, void* workspace, size_t ws_bytes,
                                      void* stream) {
    return gemv_impl<1>(packed, scales, N, K, bits, group, layout, x, y, workspace, ws_bytes, stream);
}

extern "C" pot_status_t pot_gemv_host(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                      pot_layout_t layout, const void* x_host, void* y_host, void* d_x, void* d_y,
                                      void* workspace, size_t ws_bytes, void* stream) {
    if (!x_host || !y_host) return POT_ERR_NULL;
    pot_status_t st = check_gemv_args(packed, scales, N, K, bits, group, layout, d_x, d_y, workspace, ws_bytes);
    if (st != POT_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemcpyAsync(d_x, x_host, (size_t)K * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) return POT_ERR_CUDA;
    st = pot_gemv(packed, scales, N, K, bits, group, layout, d_x, d_y, workspace, ws_bytes, stream);
    if (st != POT_OK) return st;
    if (cudaMemcpyAsync(y_host, d_y, (size_t)N * 2, cudaMemcpyDeviceToHost, s) != cudaSuccess) return POT_ERR_CUDA;
    return POT_OK;
}

extern "C" pot_status_t uint_gemv(const void* packed, const void* scales, const void* zeros, int64_t N, int64_t K,
                                  int bits, int group, pot_layout_t layout, const void* x, void* y, void* workspace,
                                  size_t ws_bytes, void* stream) {
    if (!packed || !scales || !zeros || !x || !y) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if (layout != POT_LAYOUT_CANONICAL && layout != POT_LAYOUT_TILED) return POT_ERR_UNSUPPORTED;
    if (!aligned16(packed) || !aligned16(scales) || !aligned16(zeros) || !aligned16(x) || !aligned16(y) ||
        !aligned16(workspace))
        return POT_ERR_ALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    auto* S = (const uint16_t*)scales;
    auto* Z = (const uint16_t*)zeros;
    if (layout == POT_LAYOUT_CANONICAL) {
        const dim3 grid((unsigned)((N + 7) / 8)), block(256);
        auto* P = (const uint32_t*)packed;
        if (bits == 2) return launch_pdl(gemv_canonical_kernel<2, true>, grid, block, 0, s, P, S, Z, N, K, group, (const uint4*)x, (uint16_t*)y);
        if (bits == 3) return launch_pdl(gemv_canonical_kernel<3, true>, grid, block, 0, s, P, S, Z, N, K, group, (const uint4*)x, (uint16_t*)y);
        return launch_pdl(gemv_canonical_kernel<4, true>, grid, block, 0, s, P, S, Z, N, K, group, (const uint4*)x, (uint16_t*)y);
    }
    if (N % 16 != 0) return POT_ERR_SHAPE;
    const size_t need = pot_gemv_workspace_bytes(N, K, bits, group);
    if (need > 0 && (!workspace || ws_bytes < need)) return POT_ERR_WORKSPACE;
    // same kernel as pot_gemv (tensor-core path); only the decode differs
    return launch_gemv_stream<SK_UINT>(packed, scales, zeros, N, K, bits, group, x, y, workspace, s);
}

// ------------------------------------------------------------------------------------------
// pot_gemv_noalloc: the split-K GEMV for callers that are not allowed to allocate device memory.
// ------------------------------------------------------------------------------------------
// Some hosts of this library own all device memory themselves and hand their plug-ins a fixed
// budget: an inference server whose serving loop must never hit the implicit device-wide
// synchronisation of cudaMalloc/cudaFree, or an embedding application whose allocator the
// library cannot reach.  Such a caller cannot provide the split-K workspace that pot_gemv asks
// for.  For them the scratch lives in the library image itself: a fixed-size array in device
// memory that every GPU which loads the library carries until the process exits.
namespace {
constexpr size_t kNoAllocScratchBytes = size_t(1) << 20;  // 1 MiB per GPU
constexpr int kNoAllocMaxDevices = 64;
}  // namespace

// In host code this name is only a handle for the runtime (it is NOT a device address); the
// device address is looked up per GPU with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

namespace {
std::atomic<void*> g_noalloc_ptr[kNoAllocMaxDevices];
}

extern "C" size_t pot_gemv_noalloc_max_scratch_bytes(void) { return kNoAllocScratchBytes; }

extern "C" pot_status_t pot_gemv_noalloc(const void* packed_tiled, const void* scales, int64_t N, int64_t K, int bits,
                                         int group, const void* x, void* y, void* stream) {
    if (!packed_tiled || !scales || !x || !y) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if (N % 16 != 0) return POT_ERR_SHAPE;
    const size_t need = pot_gemv_workspace_bytes(N, K, bits, group);
    if (need > kNoAllocScratchBytes) return POT_ERR_WORKSPACE;  // shape needs more scratch than the built-in array holds
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return POT_ERR_CUDA;
    if (dev < 0 || dev >= kNoAllocMaxDevices) return POT_ERR_UNSUPPORTED;
    // Set-up, once per device, with that device current: ask the runtime where this GPU's copy of the
    // array lives.  (Racing first calls both get the same answer, so a plain atomic store is enough.)
    void* scratch = g_noalloc_ptr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return POT_ERR_CUDA;
        g_noalloc_ptr[dev].store(p, std::memory_order_release);
        scratch = p;
    }
    st = check_gemv_args(packed_tiled, scales, N, K, bits, group, POT_LAYOUT_TILED, x, y, scratch, kNoAllocScratchBytes);
    if (st != POT_OK) return st;  // nothing has been enqueued yet
    if (need == 0) return pot_gemv(packed_tiled, scales, N, K, bits, group, POT_LAYOUT_TILED, x, y, nullptr, 0, stream);
    // The array keeps whatever the previous call left in it.  Only the arrival counters have to start
    // at zero (the partial sums are fully overwritten before they are read), so clear just those.
    const size_t counters_bytes = plan_stream(N, K, 1, bits, group, SK_POT, 1, 16).ws_counters;
    if (cudaMemsetAsync(scratch, 0, counters_bytes, (cudaStream_t)stream) != cudaSuccess) return POT_ERR_CUDA;
    return pot_gemv(packed_tiled, scales, N, K, bits, group, POT_LAYOUT_TILED, x, y, scratch, need, stream);
}

#ifdef SK_TRACE
extern "C" void pot_debug_set_trace(void* p) { pot::g_sk_trace = (unsigned long long*)p; }
#endif
