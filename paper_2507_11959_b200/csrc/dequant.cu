// Standalone dequantization kernels: PoT (Sec. 4.2 of the paper) and the uniform-INT twin
// (first equation of Sec. 4.1).  Both stream canonical codes + per-group FP16 parameters from
// HBM and write [N,K] 16-bit weights; they are bound by HBM bandwidth (mostly the 2-byte
// write per weight), so the work is laid out for full-width coalesced stores: consecutive
// lanes produce consecutive 16-byte pieces of a row, and every thread has several independent
// pieces in flight.
#include "common.cuh"

namespace pot {

constexpr int DQ_THREADS = 256;
constexpr int DQ_UNROLL = 4;  // 8-code pieces per thread

// 8 canonical codes (8*BITS bits in v) -> 4 words with the code pairs spread 16 bits apart:
// out[j] = code(2j) | code(2j+1) << 16
template <int BITS>
__device__ __forceinline__ void spread_pairs(uint32_t v, uint32_t (&out)[4]) {
    constexpr uint32_t CM = (1u << BITS) - 1u;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t t = v >> (2 * j * BITS);
        out[j] = (t & CM) | ((t << (16 - BITS)) & (CM << 16));
    }
}

// Piece c = 8 codes = 8*BITS bits starting at bit 8*BITS*c of the stream.  The pieces of one thread are
// DQ_THREADS apart, i.e. a whole number of words (64*BITS), so word offset and bit phase are computed once.
template <int BITS>
__device__ __forceinline__ uint32_t read_piece(const uint32_t* __restrict__ w0, int sh) {
    const uint32_t lo = __ldg(w0);
    const uint32_t hi = (sh + 8 * BITS > 32) ? __ldg(w0 + 1) : 0u;
    const uint32_t v = __funnelshift_r(lo, hi, sh);
    return (8 * BITS == 32) ? v : (v & ((1u << (8 * BITS % 32)) - 1u));
}

// PoT: FP16 (EBIT = 10) or BF16 (EBIT = 7) output.
template <int BITS, int EBIT>
__global__ void __launch_bounds__(DQ_THREADS) pot_dequant_kernel(const uint32_t* __restrict__ packed,
                                                                 const uint16_t* __restrict__ scales, int64_t n_pieces,
                                                                 int ppg_shift, uint4* __restrict__ out) {
    // programmatic dependent launch: this grid may have been scheduled while its predecessor in the stream was still
    // running; nothing is read or written before the predecessor has completed
    pdl_wait();
    pdl_launch_dependents();
    constexpr uint32_t QM2 = (uint32_t)qmax_of(BITS) * 0x10001u;   // exponent mask, both halves
    constexpr uint32_t SM2 = (1u << (BITS - 1)) * 0x10001u;        // sign mask, both halves
    const int64_t base = ((int64_t)blockIdx.x * DQ_UNROLL) * DQ_THREADS + threadIdx.x;
    const int64_t bit0 = base * (8 * BITS);
    const uint32_t* w0 = packed + (bit0 >> 5);
    const int sh = (int)(bit0 & 31);
    uint32_t v[DQ_UNROLL];
    uint32_t sc[DQ_UNROLL];
#pragma unroll
    for (int u = 0; u < DQ_UNROLL; ++u) {
        const int64_t c = base + (int64_t)u * DQ_THREADS;
        if (c < n_pieces) {
            v[u] = read_piece<BITS>(w0 + u * (DQ_THREADS * BITS / 4), sh);
            sc[u] = __ldg(scales + (c >> ppg_shift));
        }
    }
#pragma unroll
    for (int u = 0; u < DQ_UNROLL; ++u) {
        const int64_t c = base + (int64_t)u * DQ_THREADS;
        if (c >= n_pieces) continue;
        uint32_t s16 = sc[u];
        if (EBIT == 7) {  // BF16 output: round the FP16 scale once to BF16
            s16 = __bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half((uint16_t)s16))));
        }
        const uint32_t sc2 = s16 * 0x10001u;
        uint32_t pr[4];
        spread_pairs<BITS>(v[u], pr);
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // stage 1 (bit manipulation): exponent by AND mask, sign moved up, OR;
            // stage 2 (fixed-point add): align with the exponent field and add to the scale's bits.
            // (the power-of-two multiplies are the alignment shifts, fused with the adds into IMADs)
            const uint32_t e = (pr[j] & QM2) * (1u << EBIT) + sc2;
            o[j] = (pr[j] & SM2) * (1u << (16 - BITS)) + e;
        }
        out[c] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// PoT, n = 3: the 24-bit pieces of the canonical stream straddle 32-bit words, so the generic kernel needs two
// loads per piece.  Here a thread takes four consecutive pieces = exactly three words (one coalesced 12-byte
// read) and the block transposes the decoded pieces through shared memory, so that the stores stay coalesced.
template <int EBIT>
__global__ void __launch_bounds__(DQ_THREADS) pot_dequant3_kernel(const uint32_t* __restrict__ packed,
                                                                  const uint16_t* __restrict__ scales, int64_t n_pieces,
                                                                  int ppg_shift, uint4* __restrict__ out) {
    // programmatic dependent launch: this grid may have been scheduled while its predecessor in the stream was still
    // running; nothing is read or written before the predecessor has completed
    pdl_wait();
    pdl_launch_dependents();
    constexpr uint32_t QM2 = (uint32_t)qmax_of(3) * 0x10001u, SM2 = 4u * 0x10001u;
    __shared__ uint4 tile[4 * DQ_THREADS];
    const int t = threadIdx.x;
    const int64_t base = (int64_t)blockIdx.x * (4 * DQ_THREADS);  // first piece of the block
    const int64_t c0 = base + 4 * t;                              // this thread's four pieces (one scale group)
    if (c0 < n_pieces) {
        const uint32_t* w = packed + (int64_t)blockIdx.x * (3 * DQ_THREADS) + 3 * t;
        const uint32_t w0 = __ldg(w), w1 = __ldg(w + 1), w2 = __ldg(w + 2);
        uint32_t s16 = __ldg(scales + (c0 >> ppg_shift));
        if (EBIT == 7) s16 = __bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half((uint16_t)s16))));
        const uint32_t sc2 = s16 * 0x10001u;
        const uint32_t v[4] = {w0 & 0xFFFFFFu, __funnelshift_r(w0, w1, 24) & 0xFFFFFFu, __funnelshift_r(w1, w2, 16) & 0xFFFFFFu,
                               w2 >> 8};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t pr[4], o[4];
            spread_pairs<3>(v[j], pr);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t e = (pr[i] & QM2) * (1u << EBIT) + sc2;
                o[i] = (pr[i] & SM2) * (1u << 13) + e;
            }
            tile[j * DQ_THREADS + ((t + 2 * j) & (DQ_THREADS - 1))] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int o = i * DQ_THREADS + t;  // piece of the block, written by consecutive threads
        const int tt = o >> 2, j = o & 3;
        if (base + o < n_pieces) out[base + o] = tile[j * DQ_THREADS + ((tt + 2 * j) & (DQ_THREADS - 1))];
    }
}

// uniform twin, packed-half arithmetic: q -> FP16 by splicing it under the exponent of 1024,
// (1024 + q) - (1024 + z) is exact, one HMUL2 by the scale rounds once.
template <int BITS>
__global__ void __launch_bounds__(DQ_THREADS) uint_dequant_fast_kernel(const uint32_t* __restrict__ packed,
                                                                       const uint16_t* __restrict__ scales,
                                                                       const uint16_t* __restrict__ zeros,
                                                                       int64_t n_pieces, int ppg_shift,
                                                                       uint4* __restrict__ out) {
    // programmatic dependent launch: this grid may have been scheduled while its predecessor in the stream was still
    // running; nothing is read or written before the predecessor has completed
    pdl_wait();
    pdl_launch_dependents();
    const int64_t base = ((int64_t)blockIdx.x * DQ_UNROLL) * DQ_THREADS + threadIdx.x;
    const int64_t bit0 = base * (8 * BITS);
    const uint32_t* w0 = packed + (bit0 >> 5);
    const int sh = (int)(bit0 & 31);
    uint32_t v[DQ_UNROLL];
    uint32_t sc[DQ_UNROLL], zp[DQ_UNROLL];
#pragma unroll
    for (int u = 0; u < DQ_UNROLL; ++u) {
        const int64_t c = base + (int64_t)u * DQ_THREADS;
        if (c < n_pieces) {
            v[u] = read_piece<BITS>(w0 + u * (DQ_THREADS * BITS / 4), sh);
            sc[u] = __ldg(scales + (c >> ppg_shift));
            zp[u] = __ldg(zeros + (c >> ppg_shift));
        }
    }
#pragma unroll
    for (int u = 0; u < DQ_UNROLL; ++u) {
        const int64_t c = base + (int64_t)u * DQ_THREADS;
        if (c >= n_pieces) continue;
        const __half2 s2 = __half2half2(__ushort_as_half((uint16_t)sc[u]));
        const __half2 zm2 = __hadd2(__half2half2(__ushort_as_half((uint16_t)zp[u])), __float2half2_rn(1024.0f));
        uint32_t pr[4];
        spread_pairs<BITS>(v[u], pr);
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t h = pr[j] | 0x64006400u;  // half2{1024 + q0, 1024 + q1}
            const __half2 d = __hsub2(*reinterpret_cast<const __half2*>(&h), zm2);
            const __half2 w = __hmul2(d, s2);
            o[j] = *reinterpret_cast<const uint32_t*>(&w);
        }
        out[c] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// uniform twin, n = 3, same access pattern as pot_dequant3_kernel (three aligned words per thread, transposition
// through shared memory): only the arithmetic differs
__global__ void __launch_bounds__(DQ_THREADS) uint_dequant3_fast_kernel(const uint32_t* __restrict__ packed,
                                                                        const uint16_t* __restrict__ scales,
                                                                        const uint16_t* __restrict__ zeros, int64_t n_pieces,
                                                                        int ppg_shift, uint4* __restrict__ out) {
    // programmatic dependent launch: this grid may have been scheduled while its predecessor in the stream was still
    // running; nothing is read or written before the predecessor has completed
    pdl_wait();
    pdl_launch_dependents();
    __shared__ uint4 tile[4 * DQ_THREADS];
    const int t = threadIdx.x;
    const int64_t base = (int64_t)blockIdx.x * (4 * DQ_THREADS);
    const int64_t c0 = base + 4 * t;
    if (c0 < n_pieces) {
        const uint32_t* w = packed + (int64_t)blockIdx.x * (3 * DQ_THREADS) + 3 * t;
        const uint32_t w0 = __ldg(w), w1 = __ldg(w + 1), w2 = __ldg(w + 2);
        const __half2 s2 = __half2half2(__ushort_as_half(__ldg(scales + (c0 >> ppg_shift))));
        const __half2 zm2 = __hadd2(__half2half2(__ushort_as_half(__ldg(zeros + (c0 >> ppg_shift)))), __float2half2_rn(1024.0f));
        const uint32_t v[4] = {w0 & 0xFFFFFFu, __funnelshift_r(w0, w1, 24) & 0xFFFFFFu, __funnelshift_r(w1, w2, 16) & 0xFFFFFFu,
                               w2 >> 8};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t pr[4], o[4];
            spread_pairs<3>(v[j], pr);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t h = pr[i] | 0x64006400u;  // half2{1024 + q0, 1024 + q1}
                const __half2 wv = __hmul2(__hsub2(*reinterpret_cast<const __half2*>(&h), zm2), s2);
                o[i] = *reinterpret_cast<const uint32_t*>(&wv);
            }
            tile[j * DQ_THREADS + ((t + 2 * j) & (DQ_THREADS - 1))] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int o = i * DQ_THREADS + t;
        const int tt = o >> 2, j = o & 3;
        if (base + o < n_pieces) out[base + o] = tile[j * DQ_THREADS + ((tt + 2 * j) & (DQ_THREADS - 1))];
    }
}

// uniform twin, the textbook form: integer -> float, subtract the zero-point, multiply by the scale.
template <int BITS>
__global__ void __launch_bounds__(DQ_THREADS) uint_dequant_naive_kernel(const uint32_t* __restrict__ packed,
                                                                        const uint16_t* __restrict__ scales,
                                                                        const uint16_t* __restrict__ zeros,
                                                                        int64_t n_pieces, int ppg_shift,
                                                                        uint4* __restrict__ out) {
    // programmatic dependent launch: this grid may have been scheduled while its predecessor in the stream was still
    // running; nothing is read or written before the predecessor has completed
    pdl_wait();
    pdl_launch_dependents();
    constexpr uint32_t CM = (1u << BITS) - 1u;
    const int64_t base = ((int64_t)blockIdx.x * DQ_UNROLL) * DQ_THREADS + threadIdx.x;
#pragma unroll
    for (int u = 0; u < DQ_UNROLL; ++u) {
        const int64_t c = base + (int64_t)u * DQ_THREADS;
        if (c >= n_pieces) continue;
        const uint32_t v = read_bits(packed, c * (8 * BITS), 8 * BITS);
        const float s = __half2float(__ushort_as_half(__ldg(scales + (c >> ppg_shift))));
        const float z = __half2float(__ushort_as_half(__ldg(zeros + (c >> ppg_shift))));
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float q0 = (float)((v >> (2 * j * BITS)) & CM);
            const float q1 = (float)((v >> ((2 * j + 1) * BITS)) & CM);
            const __half2 w = __floats2half2_rn((q0 - z) * s, (q1 - z) * s);
            o[j] = *reinterpret_cast<const uint32_t*>(&w);
        }
        out[c] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

}  // namespace pot

using namespace pot;

extern "C" pot_status_t pot_dequant(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                    pot_dtype_t out_dtype, void* W_out, void* stream) {
    if (!packed || !scales || !W_out) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if (out_dtype != POT_F16 && out_dtype != POT_BF16) return POT_ERR_UNSUPPORTED;
    if (!aligned16(packed) || !aligned16(scales) || !aligned16(W_out)) return POT_ERR_ALIGN;
    const int64_t n_pieces = N * K / 8;
    const unsigned grid = (unsigned)((n_pieces + DQ_THREADS * DQ_UNROLL - 1) / (DQ_THREADS * DQ_UNROLL));
    cudaStream_t s = (cudaStream_t)stream;
    auto* P = (const uint32_t*)packed;
    auto* S = (const uint16_t*)scales;
    auto* O = (uint4*)W_out;
    const int ppg = group == 64 ? 3 : 4;  // log2(pieces per group): a 64-bit division per piece would dominate the kernel
    pot_status_t rc = POT_OK;
#define POT_DQ(B)                                                                                     \
    if (out_dtype == POT_F16) rc = launch_pdl(pot_dequant_kernel<B, 10>, dim3(grid), dim3(DQ_THREADS), 0, s, P, S, n_pieces, ppg, O); \
    else rc = launch_pdl(pot_dequant_kernel<B, 7>, dim3(grid), dim3(DQ_THREADS), 0, s, P, S, n_pieces, ppg, O);
    if (bits == 2) {
        POT_DQ(2)
    } else if (bits == 3) {
        if (out_dtype == POT_F16) rc = launch_pdl(pot_dequant3_kernel<10>, dim3(grid), dim3(DQ_THREADS), 0, s, P, S, n_pieces, ppg, O);
        else rc = launch_pdl(pot_dequant3_kernel<7>, dim3(grid), dim3(DQ_THREADS), 0, s, P, S, n_pieces, ppg, O);
    } else {
        POT_DQ(4)
    }
#undef POT_DQ
    return rc;
}

extern "C" pot_status_t uint_dequant(const void* packed, const void* scales, const void* zeros, int64_t N, int64_t K,
                                     int bits, int group, uint_kernel_t kernel, void* W_out, void* stream) {
    if (!packed || !scales || !zeros || !W_out) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if (kernel != UINT_KERNEL_FAST && kernel != UINT_KERNEL_NAIVE) return POT_ERR_UNSUPPORTED;
    if (!aligned16(packed) || !aligned16(scales) || !aligned16(zeros) || !aligned16(W_out)) return POT_ERR_ALIGN;
    const int64_t n_pieces = N * K / 8;
    const unsigned grid = (unsigned)((n_pieces + DQ_THREADS * DQ_UNROLL - 1) / (DQ_THREADS * DQ_UNROLL));
    cudaStream_t s = (cudaStream_t)stream;
    auto* P = (const uint32_t*)packed;
    auto* S = (const uint16_t*)scales;
    auto* Z = (const uint16_t*)zeros;
    auto* O = (uint4*)W_out;
    const int ppg = group == 64 ? 3 : 4;  // log2(pieces per group): a 64-bit division per piece would dominate the kernel
    pot_status_t rc = POT_OK;
#define UINT_DQ(B)                                                                                              \
    if (kernel == UINT_KERNEL_FAST) rc = launch_pdl(uint_dequant_fast_kernel<B>, dim3(grid), dim3(DQ_THREADS), 0, s, P, S, Z, n_pieces, ppg, O); \
    else rc = launch_pdl(uint_dequant_naive_kernel<B>, dim3(grid), dim3(DQ_THREADS), 0, s, P, S, Z, n_pieces, ppg, O);
    if (bits == 2) {
        UINT_DQ(2)
    } else if (bits == 3) {
        if (kernel == UINT_KERNEL_FAST) rc = launch_pdl(uint_dequant3_fast_kernel, dim3(grid), dim3(DQ_THREADS), 0, s, P, S, Z, n_pieces, ppg, O);
        else rc = launch_pdl(uint_dequant_naive_kernel<3>, dim3(grid), dim3(DQ_THREADS), 0, s, P, S, Z, n_pieces, ppg, O);
    } else {
        UINT_DQ(4)
    }
#undef UINT_DQ
    return rc;
}
