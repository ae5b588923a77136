// pot_gemm: Y[M,N] = X[M,K] W~^T with the dequantization fused in.
//
//  * M <= 32, tiled layout: bandwidth-bound tensor-core kernel.  The weights are the MMA's
//    M-side operand (16 rows per warp-step), the tokens its 8-wide N side, so no padding of M
//    to 16 is needed and a warp decodes each record exactly once, straight into the A
//    fragment registers -- the FP16 weights never exist in shared or global memory.
//    Because a reduction may visit K in any order, the MMA's k-slots are mapped to the four
//    lanes' column blocks: lane (gid, tig) feeds codes 4j..4j+3 of its record (rows gid and
//    gid+8, column block 4*chunk + tig) into k-slots {2tig, 2tig+1, 2tig+8, 2tig+9} of step j,
//    and the B fragment reads x at the same columns.
//  * any M, canonical layout: a plain shared-memory tiled mma.sync kernel (the fallback).
//  * large M, tiled layout: the tcgen05 kernel in gemm_prefill.cu.
#include "common.cuh"
#include "layout.cuh"

namespace pot {

__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int GS_WARPS = 4;

struct GemmSmallPlan {
    int splits;
    int chunks_per_split;
};

inline GemmSmallPlan plan_gemm_small(int64_t N, int64_t K) {
    const int64_t rbs = N / 16;
    const int chunks = (int)((K + 511) / 512);
    int splits = 1;
    while (rbs * splits < 4 * kSmCount && chunks / (splits * 2) >= GS_WARPS && splits < 16) splits *= 2;
    GemmSmallPlan p;
    p.chunks_per_split = (chunks + splits - 1) / splits;
    p.splits = (chunks + p.chunks_per_split - 1) / p.chunks_per_split;
    return p;
}

// MT = number of 8-token tiles (M <= 8*MT)
template <int BITS, int MT>
__global__ void __launch_bounds__(GS_WARPS * 32) pot_gemm_small_kernel(const uint4* __restrict__ packed,
                                                                        const uint16_t* __restrict__ scales, int64_t N,
                                                                        int64_t K, int G, int chunks_per_split,
                                                                        const __half* __restrict__ X, int M,
                                                                        __half* __restrict__ Y, float* __restrict__ partial,
                                                                        unsigned* __restrict__ counters) {
    constexpr int NW = 4 * BITS;
    __shared__ float red[GS_WARPS][MT][16][8];
    __shared__ int is_last;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    const int64_t rb = blockIdx.x;
    const int split = blockIdx.y, nsplit = gridDim.y;
    const int64_t ncb = K / 128;
    const int gpr = (int)(K / G);
    const int spr = 128 / G;
    const int chunk_begin = split * chunks_per_split;
    const int chunk_end = min(chunk_begin + chunks_per_split, (int)((K + 511) / 512));

    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;

    // Lanes whose column block lies beyond K (partial last chunk) keep all-zero records with scale 1.0
    // and read x as zero: every lane of the warp must still execute the (warp-wide) MMA instructions.
    uint32_t rec[2][NW];
    uint32_t sc[2][2];
    auto load = [&](int chunk) {
        const int64_t cb = 4 * (int64_t)chunk + tig;
        if (cb < ncb) {
            const uint4* unit = packed + (rb * ncb + cb) * (16 * BITS);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int t = 0; t < BITS; ++t) {
                    const uint4 q = __ldg(unit + t * 16 + gid + 8 * h);
                    rec[h][4 * t + 0] = q.x; rec[h][4 * t + 1] = q.y; rec[h][4 * t + 2] = q.z; rec[h][4 * t + 3] = q.w;
                }
                const uint16_t* sp = scales + (rb * 16 + gid + 8 * h) * gpr + cb * spr;
                sc[h][0] = (uint32_t)__ldg(sp) * 0x10001u;
                sc[h][1] = (uint32_t)__ldg(sp + spr - 1) * 0x10001u;
            }
        } else {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int i = 0; i < NW; ++i) rec[h][i] = 0u;
                sc[h][0] = sc[h][1] = 0x3C003C00u;
            }
        }
    };
    int c = chunk_begin + warp;
    if (c < chunk_end) load(c);
    pdl_launch_dependents();
    pdl_wait();
    for (; c < chunk_end; c += GS_WARPS) {
        const int64_t cb = 4 * (int64_t)c + tig;
        const bool valid = cb < ncb;
#pragma unroll
        for (int blk = 0; blk < 8; ++blk) {
            uint32_t w0[8], w1[8];
            potl::pot_decode_pairs16<BITS>(rec[0], blk, sc[0][blk >> 2], w0);
            potl::pot_decode_pairs16<BITS>(rec[1], blk, sc[1][blk >> 2], w1);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const int token = 8 * mt + gid;
                uint4 xa = make_uint4(0, 0, 0, 0), xb = make_uint4(0, 0, 0, 0);
                if (valid && token < M) {
                    const uint4* xp = reinterpret_cast<const uint4*>(X + (int64_t)token * K + cb * 128) + 2 * blk;
                    xa = __ldg(xp);
                    xb = __ldg(xp + 1);
                }
                mma_16816(acc[mt], w0[0], w1[0], w0[1], w1[1], xa.x, xa.y);
                mma_16816(acc[mt], w0[2], w1[2], w0[3], w1[3], xa.z, xa.w);
                mma_16816(acc[mt], w0[4], w1[4], w0[5], w1[5], xb.x, xb.y);
                mma_16816(acc[mt], w0[6], w1[6], w0[7], w1[7], xb.z, xb.w);
            }
        }
        if (c + GS_WARPS < chunk_end) load(c + GS_WARPS);
    }
    // accumulator (row gid / gid+8, token 2tig / 2tig+1) -> shared, then sum the warps
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        red[warp][mt][gid][2 * tig] = acc[mt][0];
        red[warp][mt][gid][2 * tig + 1] = acc[mt][1];
        red[warp][mt][gid + 8][2 * tig] = acc[mt][2];
        red[warp][mt][gid + 8][2 * tig + 1] = acc[mt][3];
    }
    __syncthreads();
    // thread -> (token, row): consecutive threads take consecutive rows, so stores to Y[token][rows] coalesce
    for (int e = threadIdx.x; e < MT * 8 * 16; e += GS_WARPS * 32) {
        const int r = e & 15, token = e >> 4;
        if (token >= M) continue;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < GS_WARPS; ++w) s += red[w][token >> 3][r][token & 7];
        const int64_t row = rb * 16 + r;
        if (nsplit == 1) Y[(int64_t)token * N + row] = __float2half_rn(s);
        else partial[((int64_t)split * M + token) * N + row] = s;
    }
    if (nsplit == 1) return;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned prev = atomicAdd(&counters[rb], 1u);
        is_last = (prev == (unsigned)nsplit - 1u);
        if (is_last) counters[rb] = 0u;
    }
    __syncthreads();
    if (is_last) {
        __threadfence();
        for (int e = threadIdx.x; e < MT * 8 * 16; e += GS_WARPS * 32) {
            const int r = e & 15, token = e >> 4;
            if (token >= M) continue;
            const int64_t row = rb * 16 + r;
            float s = 0.f;
            for (int sp = 0; sp < nsplit; ++sp) s += __ldcg(partial + ((int64_t)sp * M + token) * N + row);
            Y[(int64_t)token * N + row] = __float2half_rn(s);
        }
    }
}

// ------------------------------------------------------------------------------------------
// fallback: canonical layout, any M.  64 tokens x 64 rows x 128 columns per CTA step.
// ------------------------------------------------------------------------------------------
constexpr int FB_LD = 136;  // padded leading dimension (halves) -> conflict-free fragment loads

template <int BITS>
__global__ void __launch_bounds__(128) pot_gemm_fallback_kernel(const uint32_t* __restrict__ packed,
                                                                const uint16_t* __restrict__ scales, int64_t N, int64_t K,
                                                                int G, const __half* __restrict__ X, int64_t M,
                                                                __half* __restrict__ Y) {
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
            if (m0 + r < M) xv = __ldg(reinterpret_cast<const uint4*>(X + (m0 + r) * K + kb * 128) + pc);
            *reinterpret_cast<uint4*>(&Xs[r * FB_LD + pc * 8]) = xv;
            uint4 wv = make_uint4(0, 0, 0, 0);
            const int64_t row = n0 + r;
            if (row < N) {
                const int64_t k = kb * 128 + pc * 8;
                const uint32_t v = read_bits(packed + row * (K * BITS / 32), k * BITS, 8 * BITS);
                const uint32_t sc2 = (uint32_t)__ldg(scales + row * (K / G) + k / G) * 0x10001u;
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t t = v >> (2 * j * BITS);
                    const uint32_t pr = (t & CM) | ((t << (16 - BITS)) & (CM << 16));
                    o[j] = sc2 + (((pr & QM2) << 10) | ((pr & SM2) << (16 - BITS)));
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
                for (int j = 0; j < 4; ++j) mma_16816(acc[i][j], a[i][0], a[i][1], a[i][2], a[i][3], b[j][0], b[j][1]);
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
                    if (row < N) Y[token * N + row] = __float2half_rn(acc[i][j][2 * hh]);
                    if (row + 1 < N) Y[token * N + row + 1] = __float2half_rn(acc[i][j][2 * hh + 1]);
                }
            }
}

pot_status_t gemm_prefill_launch(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                 const void* X, int64_t M, void* Y, void* workspace, size_t ws_bytes, cudaStream_t s);
size_t gemm_prefill_workspace(int64_t M, int64_t N, int64_t K, int bits, int group);
bool gemm_prefill_supported(int64_t M, int64_t N, int64_t K, int bits, int group);

}  // namespace pot

using namespace pot;

static bool use_small(int64_t M, int64_t N, pot_layout_t layout) {
    return layout == POT_LAYOUT_TILED && M <= 32 && N % 16 == 0;
}

extern "C" size_t pot_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int bits, int group) {
    if (check_shape(N, K, bits, group) != POT_OK || M <= 0) return 0;
    if (M <= 32 && N % 16 == 0) {
        const GemmSmallPlan p = plan_gemm_small(N, K);
        if (p.splits == 1) return 0;
        const size_t counters = ((size_t)(N / 16) * 4 + 255) / 256 * 256;
        return counters + (size_t)p.splits * (size_t)M * (size_t)N * 4;
    }
    return gemm_prefill_workspace(M, N, K, bits, group);
}

extern "C" pot_status_t pot_gemm(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                 pot_layout_t layout, const void* X, int64_t M, void* Y, void* workspace,
                                 size_t ws_bytes, void* stream) {
    if (!packed || !scales || !X || !Y) return POT_ERR_NULL;
    pot_status_t st = check_shape(N, K, bits, group);
    if (st != POT_OK) return st;
    if (M <= 0 || M > (int64_t(1) << 24)) return POT_ERR_SHAPE;
    if (layout != POT_LAYOUT_CANONICAL && layout != POT_LAYOUT_TILED) return POT_ERR_UNSUPPORTED;
    if (layout == POT_LAYOUT_TILED && N % 16 != 0) return POT_ERR_SHAPE;
    if (!aligned16(packed) || !aligned16(scales) || !aligned16(X) || !aligned16(Y) || !aligned16(workspace))
        return POT_ERR_ALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    if (use_small(M, N, layout)) {
        const GemmSmallPlan p = plan_gemm_small(N, K);
        const size_t need = pot_gemm_workspace_bytes(M, N, K, bits, group);
        if (need > 0 && (!workspace || ws_bytes < need)) return POT_ERR_WORKSPACE;
        const size_t counters_bytes = ((size_t)(N / 16) * 4 + 255) / 256 * 256;
        unsigned* counters = (unsigned*)workspace;
        float* partial = need ? (float*)((char*)workspace + counters_bytes) : nullptr;
        const dim3 grid((unsigned)(N / 16), (unsigned)p.splits), block(GS_WARPS * 32);
        auto* P = (const uint4*)packed;
        auto* S = (const uint16_t*)scales;
        auto* Xp = (const __half*)X;
        auto* Yp = (__half*)Y;
        const int Mi = (int)M;
#define POT_GS(B, T) return launch_pdl(pot_gemm_small_kernel<B, T>, grid, block, 0, s, P, S, N, K, group, p.chunks_per_split, Xp, Mi, Yp, partial, counters)
#define POT_GS_B(B)                  \
    if (M <= 8) POT_GS(B, 1);        \
    else if (M <= 16) POT_GS(B, 2);  \
    else POT_GS(B, 4);
        if (bits == 2) { POT_GS_B(2) } else if (bits == 3) { POT_GS_B(3) } else { POT_GS_B(4) }
#undef POT_GS_B
#undef POT_GS
    }
    if (layout == POT_LAYOUT_TILED) {
        if (!gemm_prefill_supported(M, N, K, bits, group)) return POT_ERR_UNSUPPORTED;
        return gemm_prefill_launch(packed, scales, N, K, bits, group, X, M, Y, workspace, ws_bytes, s);
    }
    const dim3 grid((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64)), block(128);
    auto* P = (const uint32_t*)packed;
    auto* S = (const uint16_t*)scales;
    if (bits == 2) return launch_pdl(pot_gemm_fallback_kernel<2>, grid, block, 0, s, P, S, N, K, group, (const __half*)X, M, (__half*)Y);
    if (bits == 3) return launch_pdl(pot_gemm_fallback_kernel<3>, grid, block, 0, s, P, S, N, K, group, (const __half*)X, M, (__half*)Y);
    return launch_pdl(pot_gemm_fallback_kernel<4>, grid, block, 0, s, P, S, N, K, group, (const __half*)X, M, (__half*)Y);
}
