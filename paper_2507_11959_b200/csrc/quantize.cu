// Set-up kernels: reference quantizers (Eq. 2 and the uniform twin), scale validation and the
// canonical <-> tiled repack.  None of these is on the timed path; they are written for
// exactness (FP64 threshold tests, correctly rounded conversions), not speed.
#include "common.cuh"
#include "layout.cuh"

namespace pot {

std::atomic<uint64_t> g_launches{0};

__device__ __forceinline__ uint16_t clamp_scale_bits(uint16_t sb, int bits) {
    const uint16_t lo = 0x0400;
    const uint16_t hi = (uint16_t)(((30 - qmax_of(bits)) << 10) | 0x3FF);
    return sb < lo ? lo : (sb > hi ? hi : sb);
}

// One warp per group.  codes are staged in shared memory, then packed 32 bits at a time.
// rule 0: top level on max|w|; 1: Algorithm 1's s0; 2: given; 3: Algorithm 1's grid search.
template <int BITS, bool UNIFORM>
__global__ void __launch_bounds__(256) quantize_kernel(const __half* __restrict__ W, int64_t N, int64_t K, int G,
                                                       int rule, __half* __restrict__ S, __half* __restrict__ Z,
                                                       uint32_t* __restrict__ packed) {
    __shared__ uint8_t codes_s[8][128];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t ngroups = N * (K / G);
    const int64_t gi = (int64_t)blockIdx.x * 8 + warp;
    if (gi >= ngroups) return;
    const __half* wg = W + gi * G;
    const int per = G / 32;  // 2 or 4 elements per lane
    double w[4];
    double amax = 0.0, mn = 1e300, mx = -1e300;
    for (int i = 0; i < per; ++i) {
        w[i] = (double)__half2float(wg[lane * per + i]);
        amax = fmax(amax, fabs(w[i]));
        mn = fmin(mn, w[i]);
        mx = fmax(mx, w[i]);
    }
    for (int o = 16; o; o >>= 1) {
        amax = fmax(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        mn = fmin(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    constexpr int QMAX = qmax_of(BITS);
    if constexpr (!UNIFORM) {
        uint16_t sb;
        if (rule == POT_SCALE_GIVEN) {
            sb = __half_as_ushort(S[gi]);
        } else if (rule == POT_SCALE_SEARCH) {
            // Algorithm 1: s0 = max|w| / (2^q_max - 1); b = 0.01 i, i = 1..200; keep the first minimiser of
            // Q1(b) = sum_k (w_k - s0 b sign(w_k) 2^E_k(b))^2.  The 200 candidates are spread over the lanes
            // (lane l takes i = l + 1, l + 33, ...), every lane adds the G terms of its candidates in the order
            // k = 0 .. G-1 with separately rounded multiply and add -- the order and rounding of a plain sequential
            // loop -- and the warp takes the smallest (Q1, i) pair.  The weights travel by shuffle.
            const double s0 = amax / (double)((1 << QMAX) - 1);
            constexpr int NC = 7;  // ceil(200 / 32)
            double sc[NC], q1[NC];
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                sc[c] = __dmul_rn(s0, __dmul_rn(0.01, (double)(lane + 1 + 32 * c)));
                q1[c] = 0.0;
            }
            for (int src = 0; src < 32; ++src) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (j < per) {
                        const double wk = __shfl_sync(0xffffffffu, w[j], src);
                        const double w2 = __dmul_rn(wk, wk);
#pragma unroll
                        for (int c = 0; c < NC; ++c) {
                            const double s2 = __dmul_rn(sc[c], sc[c]);
                            int E = 0;
#pragma unroll
                            for (int k = 0; k < QMAX; ++k) E += (w2 > __dmul_rn(s2, (double)(1 << (2 * k + 1)))) ? 1 : 0;
                            double rec = __dmul_rn(sc[c], (double)(1 << E));
                            if (wk < 0.0) rec = -rec;
                            const double d = (sc[c] > 0.0) ? __dsub_rn(wk, rec) : wk;
                            q1[c] = __dadd_rn(q1[c], __dmul_rn(d, d));
                        }
                    }
                }
            }
            double qmin = 1e300;
            int best = 1;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                const int i = lane + 1 + 32 * c;
                if (i <= 200 && q1[c] < qmin) { qmin = q1[c]; best = i; }
            }
            for (int o = 16; o; o >>= 1) {  // smallest Q1, ties to the smaller i
                const double qo = __shfl_xor_sync(0xffffffffu, qmin, o);
                const int bo = __shfl_xor_sync(0xffffffffu, best, o);
                if (qo < qmin || (qo == qmin && bo < best)) { qmin = qo; best = bo; }
            }
            sb = clamp_scale_bits(__half_as_ushort(__double2half(__dmul_rn(s0, __dmul_rn(0.01, (double)best)))), BITS);
            if (lane == 0) S[gi] = __ushort_as_half(sb);
        } else {
            const double s = (rule == POT_SCALE_TOP) ? ldexp(amax, -QMAX) : amax / (double)((1 << QMAX) - 1);
            sb = clamp_scale_bits(__half_as_ushort(__double2half(s)), BITS);
            if (lane == 0) S[gi] = __ushort_as_half(sb);
        }
        const double Sd = (double)__half2float(__ushort_as_half(sb));
        for (int i = 0; i < per; ++i) {
            int E = 0;
            // E >= k+1  <=>  |w|/S > 2^(k+1/2)  <=>  w^2 > 2^(2k+1) S^2   (exact in FP64 for FP16 inputs)
            for (int k = 0; k < QMAX; ++k) E += (w[i] * w[i] > ldexp(Sd * Sd, 2 * k + 1)) ? 1 : 0;
            const int sign = w[i] < 0.0 ? 1 : 0;
            codes_s[warp][lane * per + i] = (uint8_t)((sign << (BITS - 1)) | E);
        }
    } else {
        const double levels = (double)((1 << BITS) - 1);
        uint16_t sb = __half_as_ushort(__double2half((mx - mn) / levels));
        if (sb < 0x0400) sb = 0x0400;
        const double s = (double)__half2float(__ushort_as_half(sb));
        double z = rint(-mn / s);
        z = fmin(fmax(z, 0.0), levels);
        if (lane == 0) {
            S[gi] = __ushort_as_half(sb);
            Z[gi] = __double2half(z);
        }
        for (int i = 0; i < per; ++i) {
            double q = rint(w[i] / s) + z;
            q = fmin(fmax(q, 0.0), levels);
            codes_s[warp][lane * per + i] = (uint8_t)q;
        }
    }
    __syncwarp();
    const int words = G * BITS / 32;
    uint32_t* out = packed + gi * words;
    for (int wi = lane; wi < words; wi += 32) {
        uint32_t v = 0;
        for (int bit = 0; bit < 32; ++bit) {
            const int B = wi * 32 + bit;
            v |= (uint32_t)((codes_s[warp][B / BITS] >> (B % BITS)) & 1u) << bit;
        }
        out[wi] = v;
    }
}

__global__ void validate_scales_kernel(const uint16_t* __restrict__ S, int64_t count, int bits, int32_t* bad) {
    int local = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
        const uint16_t s = S[i];
        local += (s != clamp_scale_bits(s, bits)) ? 1 : 0;
    }
    for (int o = 16; o; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
    if ((threadIdx.x & 31) == 0 && local) atomicAdd(bad, local);
}

// canonical bit (row stream) helpers
__device__ __forceinline__ uint32_t canon_bit(const uint8_t* row, int64_t idx) { return (row[idx >> 3] >> (idx & 7)) & 1u; }

// word index (in 32-bit words) of record word `wi` of row r (0..15) inside unit (rb, cb)
__device__ __forceinline__ int64_t tiled_word_index(int64_t rb, int64_t cb, int64_t ncb, int bits, int r, int wi) {
    const int64_t unit_words = 16 * 4 * bits;
    return (rb * ncb + cb) * unit_words + (wi >> 2) * 64 + r * 4 + (wi & 3);
}

// direction 0: canonical -> tiled.  One thread per destination word.
__global__ void repack_forward_kernel(const uint8_t* __restrict__ src, uint32_t* __restrict__ dst, int64_t N, int64_t K,
                                      int bits, int kind) {
    const int64_t ncb = K / 128, nw = 4 * bits;
    const int64_t total = N * ncb * nw;
    const int64_t row_bytes = K * bits / 8;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int wi = (int)(t % nw);
        const int64_t cb = (t / nw) % ncb;
        const int64_t i = t / (nw * ncb);
        const uint8_t* row = src + i * row_bytes;
        uint32_t v = 0;
        for (int q = 0; q < 128; ++q)
            for (int b = 0; b < bits; ++b) {
                const potl::BitPos pos = potl::record_bit(bits, kind, q, b);
                if (pos.word == wi) v |= canon_bit(row, (cb * 128 + q) * bits + b) << pos.bit;
            }
        dst[tiled_word_index(i >> 4, cb, ncb, bits, (int)(i & 15), wi)] = v;
    }
}

// direction 1: tiled -> canonical.  One thread per canonical 32-bit word.
__global__ void repack_backward_kernel(const uint32_t* __restrict__ src, uint32_t* __restrict__ dst, int64_t N, int64_t K,
                                       int bits, int kind) {
    const int64_t ncb = K / 128, nw = 4 * bits;
    const int64_t total = N * ncb * nw;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int j = (int)(t % nw);
        const int64_t cb = (t / nw) % ncb;
        const int64_t i = t / (nw * ncb);
        uint32_t v = 0;
        for (int bit = 0; bit < 32; ++bit) {
            const int B = j * 32 + bit;
            const potl::BitPos pos = potl::record_bit(bits, kind, B / bits, B % bits);
            const uint32_t w = src[tiled_word_index(i >> 4, cb, ncb, bits, (int)(i & 15), pos.word)];
            v |= ((w >> pos.bit) & 1u) << bit;
        }
        dst[i * (K * bits / 32) + cb * nw + j] = v;
    }
}

// per-group parameters: row-major [N, K/G] <-> tiled (see scale_tiled_index); one thread per value
__global__ void repack_scales_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int64_t N, int64_t K,
                                     int G, int direction) {
    const int64_t gpr = K / G, total = N * gpr;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t ti = potl::scale_tiled_index(t / gpr, t % gpr, K, G);
        if (direction == 0) dst[ti] = src[t];
        else dst[t] = src[ti];
    }
}

}  // namespace pot

using namespace pot;

extern "C" pot_status_t pot_repack_scales(const void* src, void* dst, int64_t N, int64_t K, int group, int direction,
                                          void* stream) {
    if (!src || !dst) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, 2, group);
    if (st != POT_OK) return st;
    if (N % 16 != 0) return POT_ERR_SHAPE;
    if (direction != 0 && direction != 1) return POT_ERR_UNSUPPORTED;
    if (!aligned16(src) || !aligned16(dst)) return POT_ERR_ALIGN;
    const int64_t total = N * (K / group);
    const unsigned grid = (unsigned)((total + 255) / 256 < 65535 ? (total + 255) / 256 : 65535);
    repack_scales_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((const uint16_t*)src, (uint16_t*)dst, N, K, group, direction);
    return launched();
}

extern "C" pot_status_t pot_layout_scale_index(int64_t N, int64_t K, int group, int64_t row, int64_t g, int64_t* index) {
    if (!index) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, 2, group);
    if (st != POT_OK) return st;
    if (N % 16 != 0 || row < 0 || row >= N || g < 0 || g >= K / group) return POT_ERR_SHAPE;
    *index = potl::scale_tiled_index(row, g, K, group);
    return POT_OK;
}

extern "C" pot_status_t pot_quantize_ref(const void* W, int64_t N, int64_t K, int bits, int group,
                                         pot_scale_rule_t rule, void* scales, void* packed, void* stream) {
    if (!W || !scales || !packed) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if ((int)rule < 0 || (int)rule > 3) return POT_ERR_UNSUPPORTED;
    if (!aligned16(W) || !aligned16(scales) || !aligned16(packed)) return POT_ERR_ALIGN;
    const int64_t ngroups = N * (K / group);
    const unsigned grid = (unsigned)((ngroups + 7) / 8);
    cudaStream_t s = (cudaStream_t)stream;
    auto* Wp = (const __half*)W;
    auto* Sp = (__half*)scales;
    auto* Pp = (uint32_t*)packed;
    if (bits == 2) quantize_kernel<2, false><<<grid, 256, 0, s>>>(Wp, N, K, group, (int)rule, Sp, nullptr, Pp);
    else if (bits == 3) quantize_kernel<3, false><<<grid, 256, 0, s>>>(Wp, N, K, group, (int)rule, Sp, nullptr, Pp);
    else quantize_kernel<4, false><<<grid, 256, 0, s>>>(Wp, N, K, group, (int)rule, Sp, nullptr, Pp);
    return launched();
}

extern "C" pot_status_t uint_quantize_ref(const void* W, int64_t N, int64_t K, int bits, int group, void* scales,
                                          void* zeros, void* packed, void* stream) {
    if (!W || !scales || !zeros || !packed) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if (!aligned16(W) || !aligned16(scales) || !aligned16(zeros) || !aligned16(packed)) return POT_ERR_ALIGN;
    const int64_t ngroups = N * (K / group);
    const unsigned grid = (unsigned)((ngroups + 7) / 8);
    cudaStream_t s = (cudaStream_t)stream;
    auto* Wp = (const __half*)W;
    auto* Sp = (__half*)scales;
    auto* Zp = (__half*)zeros;
    auto* Pp = (uint32_t*)packed;
    if (bits == 2) quantize_kernel<2, true><<<grid, 256, 0, s>>>(Wp, N, K, group, 0, Sp, Zp, Pp);
    else if (bits == 3) quantize_kernel<3, true><<<grid, 256, 0, s>>>(Wp, N, K, group, 0, Sp, Zp, Pp);
    else quantize_kernel<4, true><<<grid, 256, 0, s>>>(Wp, N, K, group, 0, Sp, Zp, Pp);
    return launched();
}

extern "C" pot_status_t pot_validate_scales(const void* scales, int64_t count, int bits, int32_t* d_bad, void* stream) {
    if (!scales || !d_bad) return POT_ERR_NULL;
    if (bits < 2 || bits > 4) return POT_ERR_UNSUPPORTED;
    if (count <= 0) return POT_ERR_SHAPE;
    const unsigned grid = (unsigned)((count + 255) / 256 > 1184 ? 1184 : (count + 255) / 256);
    validate_scales_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((const uint16_t*)scales, count, bits, d_bad);
    return launched();
}

// kind: 0 = PoT sign/exponent codes, 1 = uniform integer codes
static pot_status_t repack_impl(const void* src, void* dst, int64_t N, int64_t K, int bits, int kind,
                                        int direction, void* stream) {
    if (!src || !dst) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, 128);
    if (st != POT_OK) return st;
    if (N % 16 != 0) return POT_ERR_SHAPE;
    if (kind < 0 || kind > 1 || direction < 0 || direction > 1) return POT_ERR_UNSUPPORTED;
    if (!aligned16(src) || !aligned16(dst)) return POT_ERR_ALIGN;
    const int64_t total = N * (K / 128) * 4 * bits;
    const unsigned grid = (unsigned)((total + 255) / 256 > 148 * 64 ? 148 * 64 : (total + 255) / 256);
    if (direction == 0)
        repack_forward_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((const uint8_t*)src, (uint32_t*)dst, N, K, bits, kind);
    else
        repack_backward_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((const uint32_t*)src, (uint32_t*)dst, N, K, bits, kind);
    return launched();
}

extern "C" pot_status_t pot_repack(const void* src, void* dst, int64_t N, int64_t K, int bits, int direction,
                                   void* stream) {
    return repack_impl(src, dst, N, K, bits, 0, direction, stream);
}

extern "C" pot_status_t uint_repack(const void* src, void* dst, int64_t N, int64_t K, int bits, int direction,
                                    void* stream) {
    return repack_impl(src, dst, N, K, bits, 1, direction, stream);
}
