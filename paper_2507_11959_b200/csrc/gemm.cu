// pot_gemm: Y[M,N] = X[M,K] W~^T with the dequantization fused in.
//
//  * M = 1, tiled layout: the GEMV kernel (gemv.cu).
//  * 2 <= M <= 8, tiled layout: the streaming tensor-core kernel of stream.cuh.  The weights are the MMA's
//    M-side operand (16 rows per warp-step), the tokens its 8-wide N side, so no padding of M
//    to 16 is needed and a warp decodes each record exactly once, straight into the A
//    fragment registers -- the FP16 weights never exist in shared or global memory.
//    Because a reduction may visit K in any order, the MMA's k-slots are mapped to the four
//    lanes' column blocks: lane (gid, tig) feeds codes 4j..4j+3 of its record (rows gid and
//    gid+8, column block 4*chunk + tig) into k-slots {2tig, 2tig+1, 2tig+8, 2tig+9} of step j,
//    and the B fragment reads x at the same columns.
//  * any M, canonical layout: a plain shared-memory tiled mma.sync kernel (the fallback).
//  * otherwise, tiled layout: the tcgen05 kernel in gemm_prefill.cu.
#include "common.cuh"
#include "layout.cuh"
#include "stream.cuh"

namespace pot {

// ------------------------------------------------------------------------------------------
// fallback: canonical layout, any M.  64 tokens x 64 rows x 128 columns per CTA step.
// ------------------------------------------------------------------------------------------
constexpr int FB_LD = 136;  // padded leading dimension (halves) -> conflict-free fragment loads

template <int BITS, int DT = 0>  // DT = 1: BF16 activations, weights (scale rounded once to BF16) and output
__global__ void __launch_bounds__(128) pot_gemm_fallback_kernel(const uint32_t* __restrict__ packed,
                                                                const uint16_t* __restrict__ scales, int64_t N, int64_t K,
                                                                int G, const __half* __restrict__ X, int64_t M,
                                                                uint16_t* __restrict__ Y) {
    constexpr int EBIT = DT == 0 ? 10 : 7;
    constexpr uint32_t CM = (1u << BITS) - 1u;
    constexpr uint32_t QM2 = (uint32_t)qmax_of(BITS) * 0x10001u;
    constexpr uint32_t SM2 = (1u << (BITS - 1)) * 0x10001u;
    __shared__ __align__(16) __half Xs[64 * FB_LD];
    __shared__ __align__(16) __half Ws[64 * FB_LD];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    const int wm = (warp & 1) * 32, wn = (warp >> 1) * 32;
    const int64_t n0 = (int64_t)blockIdx.x * 64, m0 = (int64_t)blockIdx.y * 64;
    float acc[2][4][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[a][b][i] = 0.f;

    pdl_wait();
    for (int64_t kb = 0; kb < K / 128; ++kb) {
        __syncthreads();
        for (int idx = threadIdx.x; idx < 64 * 16; idx += 128) {
            const int r = idx >> 4, pc = idx & 15;
            uint4 xv = make_uint4(0, 0, 0, 0);
            if (m0 + r < M) xv = ld_dependent16(reinterpret_cast<const uint4*>(X + (m0 + r) * K + kb * 128) + pc);
            *reinterpret_cast<uint4*>(&Xs[r * FB_LD + pc * 8]) = xv;
            uint4 wv = make_uint4(0, 0, 0, 0);
            const int64_t row = n0 + r;
            if (row < N) {
                const int64_t k = kb * 128 + pc * 8;
                const uint32_t v = read_bits(packed + row * (K * BITS / 32), k * BITS, 8 * BITS);
                uint32_t s16 = __ldg(scales + row * (K / G) + k / G);
                if (DT == 1) s16 = __bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half((uint16_t)s16))));
                const uint32_t sc2 = s16 * 0x10001u;
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t t = v >> (2 * j * BITS);
                    const uint32_t pr = (t & CM) | ((t << (16 - BITS)) & (CM << 16));
                    o[j] = sc2 + (((pr & QM2) << EBIT) | ((pr & SM2) << (16 - BITS)));
                }
                wv = make_uint4(o[0], o[1], o[2], o[3]);
            }
            *reinterpret_cast<uint4*>(&Ws[r * FB_LD + pc * 8]) = wv;
        }
        __syncthreads();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const int k0 = ks * 16 + 2 * tig;
            uint32_t a[2][4], b[4][2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int r = wm + 16 * i + gid;
                a[i][0] = *reinterpret_cast<const uint32_t*>(&Xs[r * FB_LD + k0]);
                a[i][1] = *reinterpret_cast<const uint32_t*>(&Xs[(r + 8) * FB_LD + k0]);
                a[i][2] = *reinterpret_cast<const uint32_t*>(&Xs[r * FB_LD + k0 + 8]);
                a[i][3] = *reinterpret_cast<const uint32_t*>(&Xs[(r + 8) * FB_LD + k0 + 8]);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = wn + 8 * j + gid;
                b[j][0] = *reinterpret_cast<const uint32_t*>(&Ws[r * FB_LD + k0]);
                b[j][1] = *reinterpret_cast<const uint32_t*>(&Ws[r * FB_LD + k0 + 8]);
            }
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (DT == 0) sk_mma(acc[i][j], a[i][0], a[i][1], a[i][2], a[i][3], b[j][0], b[j][1]);
                    else sk_mma_bf16(acc[i][j], a[i][0], a[i][1], a[i][2], a[i][3], b[j][0], b[j][1]);
                }
        }
    }
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int64_t token = m0 + wm + 16 * i + gid + 8 * hh;
                const int64_t row = n0 + wn + 8 * j + 2 * tig;
                if (token < M) {
                    if (row < N) Y[token * N + row] = sk_out<DT>(acc[i][j][2 * hh]);
                    if (row + 1 < N) Y[token * N + row + 1] = sk_out<DT>(acc[i][j][2 * hh + 1]);
                }
            }
}

pot_status_t gemm_prefill_launch(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                 const void* X, int64_t M, void* Y, void* workspace, size_t ws_bytes, cudaStream_t s, int dt);
size_t gemm_prefill_workspace(int64_t M, int64_t N, int64_t K, int bits, int group);
bool gemm_prefill_supported(int64_t M, int64_t N, int64_t K, int bits, int group);
pot_status_t gemv_stream_launch(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group, const void* x,
                                void* y, void* workspace, cudaStream_t s, int dt);

}  // namespace pot

using namespace pot;

// The streaming kernel (weights decoded straight into MMA fragments, one token per MMA column) serves up to 8 tokens;
// the tcgen05 kernel's time is flat in the batch but its floor is higher.  Measured on the 13B shapes: 13 - 23 us for
// 1 - 8 tokens on the streaming kernel, 25 - 26 us for 8 - 32 tokens on the tcgen05 kernel.
constexpr int64_t kSmallBatchMax = 8;
// ... and, above four tokens, only while the eight-token activation block fits in shared memory beside the rings
// (K <= 8192 or so): read through L2 for every unit instead, the streaming kernel loses to the tcgen05 kernel at 8
// tokens (27.7 against 26.1 us at 13824 -> 5120) and still wins at 4 (20.3 against 25.8 us).  One token always takes
// the GEMV kernel.
static bool use_small(int64_t M, int64_t N, int64_t K, pot_layout_t layout, int bits = 3, int group = 128) {
    if (layout != POT_LAYOUT_TILED || M > kSmallBatchMax || N % 16 != 0) return false;
    if (M == 1) return true;
    const StreamPlan p = plan_stream(N, K, M, bits, group, SK_POT, 8, 16);
    return p.ok && (p.x_in_smem || M <= 4 || !gemm_prefill_supported(M, N, K, bits, group));
}

extern "C" size_t pot_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int bits, int group) {
    if (check_shape(N, K, bits, group) != POT_OK || M <= 0) return 0;
    if (use_small(M, N, K, POT_LAYOUT_TILED, bits, group)) {
        const size_t tok8 = plan_stream(N, K, M, bits, group, SK_POT, 8, 16).ws_bytes;
        const size_t tok1 = M == 1 ? pot_gemv_workspace_bytes(N, K, bits, group) : 0;  // one token runs the GEMV kernel
        return tok8 > tok1 ? tok8 : tok1;
    }
    return gemm_prefill_workspace(M, N, K, bits, group);
}

template <int DT>
static pot_status_t gemm_impl(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                              pot_layout_t layout, const void* X, int64_t M, void* Y, void* workspace, size_t ws_bytes,
                              void* stream) {
    if (!packed || !scales || !X || !Y) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if (M <= 0 || M > (int64_t(1) << 24)) return POT_ERR_SHAPE;
    if (layout != POT_LAYOUT_CANONICAL && layout != POT_LAYOUT_TILED) return POT_ERR_UNSUPPORTED;
    if (layout == POT_LAYOUT_TILED && N % 16 != 0) return POT_ERR_SHAPE;
    if (!aligned16(packed) || !aligned16(scales) || !aligned16(X) || !aligned16(Y) || !aligned16(workspace))
        return POT_ERR_ALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    if (use_small(M, N, K, layout, bits, group)) {
        const size_t need = pot_gemm_workspace_bytes(M, N, K, bits, group);
        if (need > 0 && (!workspace || ws_bytes < need)) return POT_ERR_WORKSPACE;
        // one token: the GEMV kernel (x in every MMA column, two CTAs per SM where the share per CTA is small)
        if (M == 1) return gemv_stream_launch(packed, scales, N, K, bits, group, X, Y, workspace, s, DT);
        const int Mi = (int)M;
#define POT_GS(B) return launch_stream<B, SK_POT, 8, 16, 1, DT>(packed, scales, nullptr, N, K, group, X, Mi, Y, workspace, error_ptr(ERR_GEMM), s)
        if (bits == 2) POT_GS(2);
        if (bits == 3) POT_GS(3);
        POT_GS(4);
#undef POT_GS
    }
    if (layout == POT_LAYOUT_TILED) {
        if (!gemm_prefill_supported(M, N, K, bits, group)) return POT_ERR_UNSUPPORTED;
        return gemm_prefill_launch(packed, scales, N, K, bits, group, X, M, Y, workspace, ws_bytes, s, DT);
    }
    if ((M + 63) / 64 > 65535) return POT_ERR_SHAPE;  // the fallback kernel's token tiles ride on gridDim.y
    const dim3 grid((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64)), block(128);
    auto* P = (const uint32_t*)packed;
    auto* S = (const uint16_t*)scales;
    if (bits == 2) return launch_pdl(pot_gemm_fallback_kernel<2, DT>, grid, block, 0, s, P, S, N, K, group, (const __half*)X, M, (uint16_t*)Y);
    if (bits == 3) return launch_pdl(pot_gemm_fallback_kernel<3, DT>, grid, block, 0, s, P, S, N, K, group, (const __half*)X, M, (uint16_t*)Y);
    return launch_pdl(pot_gemm_fallback_kernel<4, DT>, grid, block, 0, s, P, S, N, K, group, (const __half*)X, M, (uint16_t*)Y);
}

extern "C" pot_status_t pot_gemm(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                 pot_layout_t layout, const void* X, int64_t M, void* Y, void* workspace,
                                 size_t ws_bytes, void* stream) {
    return gemm_impl<0>(packed, scales, N, K, bits, group, layout, X, M, Y, workspace, ws_bytes, stream);
}

extern "C" pot_status_t pot_gemm_bf16(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                      pot_layout_t layout, const void* X, int64_t M, void* Y, void* workspace,
                                      size_t ws_bytes, void* stream) {
    return gemm_impl<1>(packed, scales, N, K, bits, group, layout, X, M, Y, workspace, ws_bytes, stream);
}

// Diagnostic: reads and clears the device error word of the gemm kernels in this library (0 = every bounded
// wait completed; 1 = a producer gave up waiting for a free ring slot; 2 = a consumer gave up waiting for
// data).  Synchronises the device.
