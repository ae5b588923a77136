// Streaming kernel for the decode GEMV (PoT and the uniform twin) and the small-batch GEMM on the tiled layout.
//
// Work decomposition.  The matrix is a sequence of units (16 rows x 128 columns, stored contiguously in
// [row block][column block] order, codes and per-group parameters alike).  The U units are cut into grid * W equal,
// contiguous ranges, one per consumer warp of the grid (W warps per CTA), so a CTA -- and every warp in it -- streams one
// contiguous byte range and all SMs move the same number of bytes (+- one unit per warp).
//
// Every warp is its own streaming engine: it owns a private ring of S slots of Q units in shared memory; lane 0 requests
// a slot's codes and scales with 1-D bulk copies (cp.async.bulk + mbarrier transaction bytes), the warp waits for the
// slot, works through its units and, when all lanes are done with it, lane 0 requests the chunk that reuses the slot.
// There is no producer warp, no empty barrier and no synchronisation between warps on the data path; the first S chunks
// are requested before the kernel waits for its predecessor in the stream (the weights are constants).
//
// Arithmetic.  Lane (gid, tig) of a warp owns quarter tig (32 columns) of rows gid and gid + 8 of a unit: exactly its
// share of the A fragments of eight m16n8k16 MMAs.  It decodes its 2 x 32 codes in registers (mask, shift and integer add
// into the group scale's bit pattern, Sec. 4.2 of the paper) and issues the MMAs against B fragments that hold the
// activation vector in every column (GEMV) or one token per column (small batch).  The FP32 accumulators stay in
// registers for as long as the warp stays inside one row block.
//
// Delivery.  A warp that covered a whole row block writes Y.  Otherwise its sums go to slot (row block, position of the
// warp among the row block's contributors) of the workspace; a per-row-block arrival counter tells the last contributor,
// which adds the slots in ascending order -- the result does not depend on timing, and no warp ever waits for another.
#pragma once
#include "common.cuh"
#include "layout.cuh"
#include "sync.cuh"

namespace pot {

enum StreamKind { SK_POT = 0, SK_UINT = 1 };

constexpr int SK_QMAX = 4;  // units per chunk (one ring slot, one set of bulk copies): 4; 2 where 4 would leave one slot; 8 for long ranges

__host__ __device__ constexpr int sk_unit_bytes(int bits) { return 256 * bits; }
// bytes of one ring slot: Q units of codes, then their scales (then their zero-points)
__host__ __device__ constexpr int sk_param_bytes(int group) { return 16 * (128 / group) * 2; }
__host__ __device__ constexpr int sk_unit_total_bytes(int bits, int group, int kind) {
    return sk_unit_bytes(bits) + (kind == SK_UINT ? 2 : 1) * sk_param_bytes(group);
}
__host__ __device__ constexpr int sk_slot_bytes(int bits, int group, int kind, int q) { return q * sk_unit_total_bytes(bits, group, kind); }

// shared-memory header of a CTA: W x 8 full barriers, W x 8 words of per-warp state, W local arrival counters, W x 2 local
// partial-sum slots
__host__ __device__ constexpr int sk_header_bytes(int warps, int tok) {
    return (warps * 64 + warps * 32 + warps * 4 + warps * 2 * 16 * tok * 4 + 127) / 128 * 128;
}

struct StreamPlan {
    int grid, warps;      // CTAs; consumer warps per CTA
    int ncb;              // column blocks (units per row block)
    uint32_t units;       // U
    uint32_t gw_total;    // GW: warps that own a range (grid * W, or U when there are fewer units than that)
    int q;                // Q: units per slot
    int stages;           // S: slots per warp ring
    int ring_capacity;    // slots per warp that would fit
    int tok;              // B columns in use: 1 (GEMV) or 8 (small batch)
    bool x_in_smem;
    int token_shift;      // log2 of the token slots of the staged activations (0 for the GEMV)
    size_t x_bytes, smem_bytes;
    int max_slots;        // partial-sum slots per row block
    size_t ws_counters, ws_bytes;
    bool aligned;         // CTA ranges end on row-block boundaries (no partial sums cross CTAs)
    int nrb;
    bool ok;              // false: the shape cannot run on this kernel (too many units)
};

inline StreamPlan plan_stream(int64_t N, int64_t K, int64_t M, int bits, int group, int kind, int tok, int warps, int occ = 1) {
    StreamPlan p = {};
    const int64_t nrb = N / 16, ncb = K / 128, U = nrb * ncb;
    p.ok = U > 0 && U < (int64_t(1) << 31) && ncb < (1 << 24);
    if (!p.ok) return p;
    p.warps = warps;
    p.ncb = (int)ncb;
    p.units = (uint32_t)U;
    p.tok = tok;
    // every range must be non-empty (the contributors of a row block are counted as consecutive warps): GW <= U
    int64_t grid = U / warps;
    if (grid < 1) grid = 1;
    p.grid = (int)(grid < kSmCount ? grid : kSmCount);
    p.gw_total = (uint32_t)((int64_t)p.grid * warps < U ? (int64_t)p.grid * warps : U);
    const int64_t GW = (int64_t)p.gw_total;
    // Row-block split: no sums cross CTAs, at the price of CTAs that differ by one row block.  Taken when that costs at
    // most a fifth more than the even split and every warp of a CTA still gets a unit.
    p.nrb = (int)nrb;
    const int64_t rb_min = nrb / p.grid, rb_max = (nrb + p.grid - 1) / p.grid;
    p.aligned = nrb >= p.grid && p.grid == kSmCount && rb_min * ncb >= warps && (double)rb_max * p.grid <= 1.2 * (double)nrb;
    const int64_t per_warp = p.aligned ? (rb_max * ncb + warps - 1) / warps : (U + GW - 1) / GW;
    // shared memory: header, the staged activations, W rings
    const size_t budget = (occ == 2 ? 113 : 224) * 1024;  // two CTAs per SM: 228 KB less 1 KB reserve each
    const size_t hdr = (size_t)sk_header_bytes(warps, tok);
    // multi-token kernel: the staged block has 2, 4 or 8 token slots per 16-byte chunk position (the smallest that holds M)
    p.token_shift = tok > 1 ? (M <= 2 ? 1 : (M <= 4 ? 2 : 3)) : 0;
    const size_t xb = ((size_t)K * 2) << p.token_shift;
    // slots of 4 units unless the ring could then hold only one of them next to the staged activations
    int q = SK_QMAX;
    if (hdr + xb + (size_t)warps * 2 * (size_t)sk_slot_bytes(bits, group, kind, q) > budget) q = 2;
    // long ranges (large matrices, one CTA per SM): slots of 8 units halve the per-slot hand-off work, if two of them fit
    else if (occ == 1 && tok == 1 && per_warp >= 32 && hdr + xb + (size_t)warps * 2 * (size_t)sk_slot_bytes(bits, group, kind, 8) <= budget) q = 8;
    p.q = q;
    const size_t slot = (size_t)sk_slot_bytes(bits, group, kind, q);
    const size_t ring2 = (size_t)warps * 2 * slot;  // at least two slots per warp
    p.x_in_smem = hdr + xb + ring2 <= budget;
    p.x_bytes = p.x_in_smem ? (xb + 127) / 128 * 128 : 0;
    int64_t st = (int64_t)((budget - hdr - p.x_bytes) / ((size_t)warps * slot));
    p.ring_capacity = (int)(st > 8 ? 8 : st);
    const int64_t need = (per_warp + q - 1) / q;
    if (st > need) st = need;
    if (st > 8) st = 8;
    if (st < 1) st = 1;
    p.stages = (int)st;
    p.smem_bytes = hdr + p.x_bytes + (size_t)warps * (size_t)p.stages * slot;
    const int64_t m = U / GW;  // shortest warp range
    int64_t slots = m >= 1 ? (ncb + m - 1) / m + 1 : ncb;
    if (slots > ncb) slots = ncb;
    p.max_slots = (int)slots;
    p.ws_counters = ((size_t)nrb * 4 + 255) / 256 * 256;
    p.ws_bytes = ncb > 1 ? p.ws_counters + (size_t)nrb * (size_t)slots * 16 * (size_t)tok * 4 : 0;
    return p;
}

struct StreamArgs {
    const unsigned char* packed;   // tiled codes
    const unsigned char* scales;   // tiled scales
    const unsigned char* zeros;    // tiled zero-points (uniform twin)
    const uint16_t* X;             // FP16 or BF16 bit patterns
    uint16_t* Y;
    float* partial;
    unsigned* counters;
    int64_t N, K;
    uint32_t units, gw_total;      // U, grid * W
    int ncb, group, stages, x_bytes, max_slots, M;
    int token_shift;               // log2 of the token slots of the staged activations
    int fits32;                    // U * gw_total < 2^32: 32-bit range arithmetic
    int aligned, nrb;              // row-block split (see the kernel), number of row blocks
#ifdef SK_TRACE
    unsigned long long* trace;     // [launch slot][cta][8] globaltimer stamps
#endif
};

#ifdef __CUDACC__
__device__ __forceinline__ void sk_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void sk_mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                            uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// FP32 sum -> 16-bit output pattern (DT = 0: FP16, 1: BF16), round to nearest even
template <int DT>
__device__ __forceinline__ uint16_t sk_out(float v) {
    if (DT == 0) return __half_as_ushort(__float2half_rn(v));
    return __bfloat16_as_ushort(__float2bfloat16_rn(v));
}
__device__ __forceinline__ uint32_t sk_lds32(const unsigned char* p) { return *reinterpret_cast<const uint32_t*>(p); }
__device__ __forceinline__ uint4 sk_lds128(const unsigned char* p) { return *reinterpret_cast<const uint4*>(p); }
// floor(a * b / c) for a * b that may need 64 bits
__device__ __forceinline__ uint32_t sk_muldiv(uint32_t a, uint32_t b, uint32_t c, bool fits32) {
    if (fits32) return (a * b) / c;
    return (uint32_t)(((uint64_t)a * (uint64_t)b) / (uint64_t)c);
}

// DT = 0: FP16 activations, weights and output; DT = 1: BF16 (PoT codes only: the scale is rounded once to BF16 and the
// exponent is added at bit 7).
// KIND: SK_POT / SK_UINT.  TOK = 1: GEMV (x in every B column).  TOK = 8: up to 8 tokens, one per B column.
// XSMEM: the activations are staged in shared memory in fragment order (else they are read through L1 from global).
// W consumer warps per CTA; OCC = 2 leaves room for a second CTA on the SM (64 registers per thread, half the shared
// memory), so that the next launch in the stream can become resident and fill its rings while this one still computes.
template <int BITS, int KIND, int TOK, bool XSMEM, int W, int OCC, int SK_Q, int DT>
__device__ __forceinline__ void stream_body(const StreamArgs& sa, int* __restrict__ err) {
    constexpr int UB = sk_unit_bytes(BITS);
    constexpr bool UNIFORM = (KIND == SK_UINT);
    constexpr int NPARAM = UNIFORM ? 2 : 1;
    extern __shared__ __align__(128) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;  // MMA fragment coordinates: rows gid and gid + 8, quarter tig
#ifdef SK_TRACE
    auto stamp = [&](int i) {
        if (sa.trace && lane == 0 && (warp == 0 || warp == W - 1)) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
            sa.trace[((size_t)blockIdx.x * 2 + (warp ? 1 : 0)) * 8 + i] = t;
        }
    };
    stamp(0);
#else
    auto stamp = [&](int) {};
#endif
    const int S = sa.stages;
    const int spg = 128 / sa.group;
    const uint32_t PB = 32u * (uint32_t)spg;                 // parameter bytes of one unit
    const uint32_t slot_bytes = SK_Q * (UB + NPARAM * PB);
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t bars = smem0 + (uint32_t)warp * 64u;      // this warp's full barriers (S <= 8)
    constexpr int HDR = sk_header_bytes(W, TOK);
    // Values a warp needs only when it requests a chunk or delivers sums live in shared memory, not in registers (the
    // two-CTAs-per-SM build has 64 registers per thread): [0] a, [1] n, [2] first row block, [3] last row block,
    // [4] slot of the first segment, [5] contributors of the first segment, [6] of the last, [7] bit 0 / 1: the first / last
    // segment is combined inside the CTA
    uint32_t* wst = reinterpret_cast<uint32_t*>(smem + W * 64) + warp * 8;
    unsigned* lcnt = reinterpret_cast<unsigned*>(smem + W * 96);               // local arrival counters
    float* lslots = reinterpret_cast<float*>(smem + W * 96 + W * 4);           // [warp][first, last][16 TOK]
    const unsigned char* xs = smem + HDR;
    const unsigned char* ringp = xs + sa.x_bytes + (uint32_t)warp * (uint32_t)S * slot_bytes;  // this warp's ring
    const uint32_t ring = smem0 + (uint32_t)HDR + (uint32_t)sa.x_bytes + (uint32_t)warp * (uint32_t)S * slot_bytes;

    // ---- this warp's range of units [a, b) ---------------------------------------------------------------
    // Unit split (sa.aligned == 0): the U units are cut into GW equal ranges, warp gw = blockIdx * W + warp takes range gw.
    // Row-block split (sa.aligned == 1): CTA c takes the row blocks [c nrb / grid, (c + 1) nrb / grid) and its W warps
    // cut that range of units into W equal ranges -- no row block is shared between CTAs.
    const bool f32 = sa.fits32 != 0;
    uint32_t base = 0, U = sa.units, GW = sa.gw_total, gw = blockIdx.x * W + warp;
    if (sa.aligned) {
        const uint32_t r0 = sk_muldiv(blockIdx.x, (uint32_t)sa.nrb, gridDim.x, f32), r1 = sk_muldiv(blockIdx.x + 1, (uint32_t)sa.nrb, gridDim.x, f32);
        base = r0 * (uint32_t)sa.ncb;
        U = (r1 - r0) * (uint32_t)sa.ncb;
        GW = W;
        gw = (uint32_t)warp;
    }
    const uint32_t a = base + (gw < GW ? sk_muldiv(gw, U, GW, f32) : 0u), b = base + (gw < GW ? sk_muldiv(gw + 1, U, GW, f32) : 0u);
    const uint32_t n = b - a;
    const uint32_t nchunks = (n + SK_Q - 1) / SK_Q;

    // chunk j of the range holds units [a + Q j, a + Q j + Q) (fewer at the end) and lives in slot j % S
    auto issue = [&](uint32_t a_, uint32_t n_, uint32_t j, uint32_t s) {  // one lane: request chunk j into slot s
        const uint32_t left_j = n_ - j * SK_Q;
        const uint32_t cnt = left_j < (uint32_t)SK_Q ? left_j : (uint32_t)SK_Q;
        const uint32_t bar = bars + s * 8u, dst = ring + s * slot_bytes;
        const size_t u0 = (size_t)a_ + (size_t)j * SK_Q;
        if (!in_range(s < (uint32_t)S && u0 + cnt <= sa.units && cnt >= 1 && cnt <= (uint32_t)SK_Q, err, 0x110)) return;
        mbar_expect_tx(bar, cnt * (UB + NPARAM * PB));
        bulk_g2s(dst, sa.packed + u0 * UB, cnt * UB, bar);
        bulk_g2s(dst + SK_Q * UB, sa.scales + u0 * PB, cnt * PB, bar);
        if constexpr (UNIFORM) bulk_g2s(dst + SK_Q * (UB + PB), sa.zeros + u0 * PB, cnt * PB, bar);
    };
    if (lane < S) {  // lane s sets up slot s and requests chunk s: the weights do not depend on the predecessor
        mbar_init(bars + (uint32_t)lane * 8u, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if ((uint32_t)lane < nchunks) issue(a, n, (uint32_t)lane, (uint32_t)lane);
    }
    __syncwarp();
    stamp(7);
    pdl_launch_dependents();

    // ---- row blocks of the range; which of its segments are partial, and their place among the contributors
    const uint32_t ncb = (uint32_t)sa.ncb;
    uint32_t rb = a / ncb, cb = a - rb * ncb;
    const uint32_t rb0 = rb, rbL = n ? (b - 1) / ncb : rb;
    uint32_t slot0 = 0, exp0 = 0, expL = 0;  // exp == 0: the segment covers its whole row block
    auto owner = [&](uint32_t u) {  // the warp (numbered like gw) whose range holds unit u
        u -= base;
        return f32 ? ((u + 1) * GW - 1) / U : (uint32_t)((((uint64_t)u + 1) * GW - 1) / U);
    };
    if (n) {
        if (cb != 0 || b < (rb0 + 1) * ncb) {
            const uint32_t lo = owner(rb0 * ncb), hi = owner((rb0 + 1) * ncb - 1);
            slot0 = gw - lo;
            exp0 = hi - lo + 1;
        }
        if (rbL != rb0 && b != (rbL + 1) * ncb) expL = owner((rbL + 1) * ncb - 1) - gw + 1;  // this warp is its first contributor
    }
    // a row block whose contributors all sit in this CTA is combined in shared memory
    const uint32_t cta_lo = sa.aligned ? 0u : blockIdx.x * W;
    const bool loc0 = exp0 && gw - slot0 >= cta_lo && gw - slot0 + exp0 <= cta_lo + W;
    const bool locL = expL && gw + expL <= cta_lo + W;
    if (lane == 0) {
        wst[0] = a; wst[1] = n; wst[2] = rb0; wst[3] = rbL;
        wst[4] = slot0; wst[5] = exp0; wst[6] = expL; wst[7] = (loc0 ? 1u : 0u) | (locL ? 2u : 0u);
    }
    if (threadIdx.x < W) lcnt[threadIdx.x] = 0u;

    stamp(1);
    pdl_wait();  // x, Y and the workspace may belong to the previous kernel in the stream
    stamp(2);
    if constexpr (XSMEM) {
        uint4* dst = reinterpret_cast<uint4*>(smem + HDR);
        const uint4* src = reinterpret_cast<const uint4*>(sa.X);
        const int kc = (int)(sa.K / 8);  // 16-byte chunks per token
        if constexpr (TOK == 1) {
            // chunk (quarter t, part j) of a unit goes to position j * 4 + t: lanes tig = 0..3 read 64 contiguous bytes
            // (four loads in flight per thread before the first store: one round trip for K <= 32 * 32 W)
            for (int i0 = threadIdx.x; i0 < kc; i0 += 4 * W * 32) {
                uint4 v[4];
#pragma unroll
                for (int p = 0; p < 4; ++p)
                    if (i0 + p * W * 32 < kc) v[p] = ld_dependent16(src + i0 + p * W * 32);
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    const int i = i0 + p * W * 32;
                    if (i < kc) dst[(i & ~15) | ((i & 3) << 2) | ((i >> 2) & 3)] = v[p];
                }
            }
        } else {
            // T = 2, 4 or 8 token slots (the smallest that holds M).  Chunk (token, unit, quarter t, part j) goes to
            // 16-byte slot (unit * 4 + j) * 4 T + (token / 2) * 8 + (token % 2) * 4 + t: the eight lanes of a quarter-warp
            // of the MMA loop (tokens 2q and 2q + 1, quarters 0..3) read one 128-byte line, a warp 4 lines -- no bank
            // conflict (token-major slots cost four-way conflicts: 11 against 8 us in the loop at 5+ tokens).  With fewer
            // than 8 slots the MMA columns beyond T repeat the first T tokens; they are never delivered, like the
            // tokens >= M.  The threads are numbered so that a quarter-warp also STORES one line: t fastest, then the
            // token's parity, then j -- a warp loads the 256 contiguous bytes of a unit for two tokens.
            const int ts = sa.token_shift;
            const int total = kc << ts;
            for (int e0 = threadIdx.x; e0 < total; e0 += 8 * W * 32) {  // eight loads in flight per thread
                uint4 v[8];
#pragma unroll
                for (int p = 0; p < 8; ++p) {
                    const int e = e0 + p * W * 32;
                    const int t = e & 3, par = (e >> 2) & 1, j = (e >> 3) & 3, hi = (e >> 5) & ((1 << (ts - 1)) - 1), unit_ = e >> (4 + ts);
                    const int token = (hi << 1) | par;
                    if (e < total && token < sa.M) v[p] = ld_dependent16(src + (int64_t)token * kc + unit_ * 16 + t * 4 + j);
                }
#pragma unroll
                for (int p = 0; p < 8; ++p) {
                    const int e = e0 + p * W * 32;
                    const int t = e & 3, par = (e >> 2) & 1, j = (e >> 3) & 3, hi = (e >> 5) & ((1 << (ts - 1)) - 1), unit_ = e >> (4 + ts);
                    const int token = (hi << 1) | par;
                    if (e < total && token < sa.M) dst[(((unit_ << 2) + j) << (2 + ts)) + (hi << 3) + (par << 2) + t] = v[p];
                }
            }
        }
    }
    __syncthreads();
    stamp(3);

    float acc[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;

    // ---- delivery of the sums of rows [16 rb, 16 rb + 16) accumulated so far ---------------------------------
    auto deliver = [&](uint32_t rbd) {
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            v[e] = acc[0][e] + acc[1][e];
            acc[0][e] = 0.f;
            acc[1][e] = 0.f;
        }
        const bool first = rbd == wst[2];
        const uint32_t expect = first ? wst[5] : (rbd == wst[3] ? wst[6] : 0u);
        const uint32_t slot = first ? wst[4] : 0u;
        const int64_t row0 = (int64_t)rbd * 16;
        if (expect == 0) {
            if constexpr (TOK == 1) {
                if (tig == 0 && in_range(row0 + gid + 8 < sa.N, err, 0x120)) {
                    sa.Y[row0 + gid] = sk_out<DT>(v[0]);
                    sa.Y[row0 + gid + 8] = sk_out<DT>(v[2]);
                }
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int token = 2 * tig + (e & 1);
                    if (token < sa.M && in_range(row0 + gid + 8 * (e >> 1) < sa.N, err, 0x121))
                        sa.Y[(int64_t)token * sa.N + row0 + gid + 8 * (e >> 1)] = sk_out<DT>(v[e]);
                }
            }
            return;
        }
        if ((wst[7] >> (first ? 0 : 1)) & 1u) {
            // slot of warp w: [w][1] if w is the row block's first contributor, else [w][0]
            const uint32_t wl = (uint32_t)warp - slot;  // first contributor (local warp index)
            if (!in_range(slot <= (uint32_t)warp && wl + expect <= (uint32_t)W && row0 + 16 <= sa.N, err, 0x130)) return;
            float* mine = lslots + ((size_t)warp * 2 + (slot == 0 ? 1 : 0)) * (16 * TOK);
            if constexpr (TOK == 1) {
                if (tig == 0) {
                    mine[gid] = v[0];
                    mine[gid + 8] = v[2];
                }
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) mine[(2 * tig + (e & 1)) * 16 + gid + 8 * (e >> 1)] = v[e];
            }
            __threadfence_block();
            __syncwarp();
            unsigned prev = 0;
            if (lane == 0) prev = atomicAdd(&lcnt[wl], 1u);
            prev = __shfl_sync(0xffffffffu, prev, 0);
            if (prev == expect - 1u) {
                __threadfence_block();
                for (int e = lane; e < 16 * (TOK == 1 ? 1 : sa.M); e += 32) {
                    float sum = 0.f;
                    for (uint32_t q = 0; q < expect; ++q) sum += lslots[((size_t)(wl + q) * 2 + (q == 0 ? 1 : 0)) * (16 * TOK) + e];
                    sa.Y[(int64_t)(e >> 4) * sa.N + row0 + (e & 15)] = sk_out<DT>(sum);
                }
            }
            return;
        }
        if (!in_range(rbd < (uint32_t)sa.nrb && slot < (uint32_t)sa.max_slots && expect <= (uint32_t)sa.max_slots && sa.partial != nullptr,
                      err, 0x140))
            return;
        float* base = sa.partial + ((size_t)rbd * (size_t)sa.max_slots) * (16 * TOK);
        float* mine = base + (size_t)slot * (16 * TOK);
        if constexpr (TOK == 1) {
            if (tig == 0) {
                mine[gid] = v[0];
                mine[gid + 8] = v[2];
            }
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int token = 2 * tig + (e & 1);
                if (token < sa.M) mine[token * 16 + gid + 8 * (e >> 1)] = v[e];
            }
        }
        __threadfence();
        __syncwarp();
        unsigned prev = 0;
        if (lane == 0) prev = atomicAdd(&sa.counters[rbd], 1u);
        prev = __shfl_sync(0xffffffffu, prev, 0);
        if (prev == expect - 1u) {  // this warp delivered the last slot of the row block: add them in ascending order
            __threadfence();
            for (int e = lane; e < 16 * (TOK == 1 ? 1 : sa.M); e += 32) {
                float sum = 0.f;
                for (uint32_t q = 0; q < expect; ++q) sum += __ldcg(base + (size_t)q * (16 * TOK) + e);
                sa.Y[(int64_t)(e >> 4) * sa.N + row0 + (e & 15)] = sk_out<DT>(sum);
            }
            if (lane == 0) sa.counters[rbd] = 0u;  // leave the workspace ready for the next call
        }
    };

    // ---- one unit: 2 x 32 codes of this lane -> 32 half2 (decode: needs no activations) -> eight MMAs (multiply) ----
    auto unit_ok = [&](const unsigned char* code, const unsigned char* param, uint32_t cbu) {
        return in_range(code >= ringp && code + UB <= ringp + (size_t)S * slot_bytes && param + NPARAM * PB <= ringp + (size_t)S * slot_bytes &&
                            cbu < ncb && (!XSMEM || ((size_t)(cbu + 1) * 256u << sa.token_shift) <= (size_t)sa.x_bytes),
                        err, 0x150);
    };
    auto decode = [&](const unsigned char* code, const unsigned char* param, uint32_t (&lo)[16], uint32_t (&hi)[16]) {
        // the scale words {row gid, row gid + 8} of this lane's group
        const uint32_t poff = ((spg == 2 ? (uint32_t)(tig >> 1) * 8u : 0u) + (uint32_t)gid) * 4u;
        if constexpr (!UNIFORM) {
            // plane k of a unit holds word k of every (row, quarter): this lane's word sits at byte 4 * lane
            uint32_t w[2][BITS];
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int k = 0; k < BITS; ++k) w[h][k] = sk_lds32(code + (uint32_t)(k * 256 + h * 128) + (uint32_t)lane * 4u);
            const uint32_t scw = sk_lds32(param + poff);  // {row gid, row gid + 8}
            if constexpr (DT == 0) {
                potl::pot_decode32<BITS, 1>(w[0], 0, __byte_perm(scw, 0, 0x1010), lo);
                potl::pot_decode32<BITS, 1>(w[1], 0, __byte_perm(scw, 0, 0x3232), hi);
            } else {  // the FP16 scale rounded once to BF16
                const uint32_t s0 = __bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half((uint16_t)(scw & 0xFFFFu)))));
                const uint32_t s1 = __bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half((uint16_t)(scw >> 16)))));
                potl::pot_decode32_bf16<BITS, 1>(w[0], 0, s0 * 0x10001u, lo);
                potl::pot_decode32_bf16<BITS, 1>(w[1], 0, s1 * 0x10001u, hi);
            }
        } else {
            // the quarter's words sit at record words 2 tig, 2 tig + 1 (n = 2), 2 tig, 2 tig + 1, 8 + tig (n = 3) or
            // 4 tig .. 4 tig + 3 (n = 4); record word w is byte (w / 4) * 256 + row * 16 + (w % 4) * 4
            const uint32_t scw = sk_lds32(param + poff);
            const uint32_t zw = sk_lds32(param + SK_Q * PB + poff);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t q[BITS == 3 ? 9 : BITS];
#pragma unroll
                for (int k = 0; k < BITS; ++k) {
                    const int wi = BITS == 4 ? 4 * tig + k : (k < 2 ? 2 * tig + k : 8 + tig);
                    q[(BITS == 3 && k == 2) ? 8 : k] =
                        sk_lds32(code + (uint32_t)((wi >> 2) * 256 + (wi & 3) * 4 + h * 128) + (uint32_t)gid * 16u);
                }
                potl::UintParams pr;
                pr.s2 = potl::bits_h2(__byte_perm(scw, 0, h ? 0x3232 : 0x1010));
                pr.z = potl::bits_h2(__byte_perm(zw, 0, h ? 0x3232 : 0x1010));
                uint32_t a8[8], b8[8];
                potl::uint_decode_pairs16<BITS>(q, 0, pr, a8);
                potl::uint_decode_pairs16<BITS>(q, 1, pr, b8);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    (h ? hi : lo)[i] = a8[i];
                    (h ? hi : lo)[8 + i] = b8[i];
                }
            }
        }
    };
    auto multiply = [&](const uint32_t (&lo)[16], const uint32_t (&hi)[16], uint32_t cbu) {
        // activations of quarter tig (of token gid): the B fragments of the eight MMAs
        uint32_t xq[16];
        if constexpr (XSMEM) {
            const unsigned char* xa = TOK == 1 ? xs + cbu * 256u + (uint32_t)tig * 16u
                                               : xs + ((((cbu * 16u) << sa.token_shift) + ((((uint32_t)gid & ((1u << sa.token_shift) - 1u)) >> 1) << 3) +
                                                        (((uint32_t)gid & 1u) << 2) + (uint32_t)tig) << 4);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 v = sk_lds128(xa + (TOK == 1 ? 64u : (64u << sa.token_shift)) * i);
                xq[4 * i + 0] = v.x; xq[4 * i + 1] = v.y; xq[4 * i + 2] = v.z; xq[4 * i + 3] = v.w;
            }
        } else {
            const bool live = TOK == 1 || gid < sa.M;
            const uint4* xp = reinterpret_cast<const uint4*>(sa.X) + (TOK == 1 || !live ? 0 : (int64_t)gid * (sa.K / 8)) +
                              (int64_t)cbu * 16 + tig * 4;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 v = make_uint4(0, 0, 0, 0);
                if (live) v = ld_dependent16(xp + i);
                xq[4 * i + 0] = v.x; xq[4 * i + 1] = v.y; xq[4 * i + 2] = v.z; xq[4 * i + 3] = v.w;
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)  // two accumulators: half the length of the dependent chain
            if constexpr (DT == 0) sk_mma(acc[j & 1], lo[2 * j], hi[2 * j], lo[2 * j + 1], hi[2 * j + 1], xq[2 * j], xq[2 * j + 1]);
            else sk_mma_bf16(acc[j & 1], lo[2 * j], hi[2 * j], lo[2 * j + 1], hi[2 * j + 1], xq[2 * j], xq[2 * j + 1]);
    };
    auto unit = [&](const unsigned char* code, const unsigned char* param, uint32_t cbu) {
        if (!unit_ok(code, param, cbu)) return;
        uint32_t lo[16], hi[16];
        decode(code, param, lo, hi);
        multiply(lo, hi, cbu);
    };

    // ---- main loop over this warp's chunks --------------------------------------------------------------------
    uint32_t s = 0, phase = 0, left = n;
    for (uint32_t j = 0; left > 0; ++j) {
        const unsigned char* code = ringp + s * slot_bytes;
        const unsigned char* param = code + SK_Q * UB;
        const uint32_t bar = bars + s * 8u;
        if (!mbar_test(bar, phase) && !mbar_wait(bar, phase)) {
            // A copy never arrived.  Record it, request nothing more, deliver nothing more (the rows this warp still owed
            // stay unwritten: the error word says so), wait -- bounded again -- for the chunks already requested, leave.
            if (err && lane == 0) atomicCAS(err, 0, 2 | (int)(j << 8) | (warp << 24));
            uint32_t s2 = s, ph2 = phase;
            for (uint32_t k = 1; k < (uint32_t)S && (j + k) * SK_Q < wst[1]; ++k) {
                if (++s2 == (uint32_t)S) {
                    s2 = 0;
                    ph2 ^= 1u;
                }
                mbar_wait(bars + s2 * 8u, ph2);
            }
            return;
        }
        if (j == 0) stamp(4);
        if (left >= (uint32_t)SK_Q && cb + (uint32_t)SK_Q <= ncb) {
            // the common case: a full chunk inside one row block, straight-line code
#pragma unroll
            for (int i = 0; i < SK_Q; ++i) unit(code + i * UB, param + (uint32_t)i * PB, cb + (uint32_t)i);
            cb += SK_Q;
            left -= SK_Q;
            if (cb == ncb) {
                deliver(rb);
                cb = 0;
                ++rb;
            }
        } else {
            const uint32_t cnt = left < (uint32_t)SK_Q ? left : (uint32_t)SK_Q;
            for (uint32_t i = 0; i < cnt; ++i) {
                unit(code, param, cb);
                code += UB;
                param += PB;
                if (++cb == ncb) {
                    deliver(rb);
                    cb = 0;
                    ++rb;
                }
            }
            left -= cnt;
        }
        __syncwarp();  // every lane has read the slot: it may be refilled
        if (lane == 0 && (j + (uint32_t)S) * SK_Q < wst[1]) issue(wst[0], wst[1], j + (uint32_t)S, s);
        if (++s == (uint32_t)S) {
            s = 0;
            phase ^= 1u;
        }
    }
    stamp(5);
    if (n && cb != 0) deliver(rb);
    stamp(6);
}

template <int BITS, int KIND, int TOK, bool XSMEM, int W, int OCC = 1, int SK_Q = SK_QMAX, int DT = 0>
__global__ void __launch_bounds__(W * 32, OCC) stream_kernel(const StreamArgs sa, int* __restrict__ err) {
    stream_body<BITS, KIND, TOK, XSMEM, W, OCC, SK_Q, DT>(sa, err);
}
#endif  // __CUDACC__

#ifdef SK_TRACE
inline unsigned long long* g_sk_trace = nullptr;   // next launch's trace block (advanced per launch)
#endif
// ---- host side --------------------------------------------------------------------------------------------
inline StreamArgs stream_args(const StreamPlan& p, const void* packed, const void* scales, const void* zeros, int64_t N,
                              int64_t K, int group, const void* X, int M, void* Y, void* workspace) {
    StreamArgs sa;
    sa.packed = (const unsigned char*)packed;
    sa.scales = (const unsigned char*)scales;
    sa.zeros = (const unsigned char*)zeros;
    sa.X = (const uint16_t*)X;
    sa.Y = (uint16_t*)Y;
    sa.counters = (unsigned*)workspace;
    sa.partial = workspace ? (float*)((char*)workspace + p.ws_counters) : nullptr;
    sa.N = N;
    sa.K = K;
    sa.units = p.units;
    sa.gw_total = p.gw_total;
    sa.aligned = p.aligned ? 1 : 0;
    sa.nrb = p.nrb;
    sa.ncb = p.ncb;
    sa.group = group;
    sa.stages = p.stages;
    sa.x_bytes = (int)p.x_bytes;
    sa.max_slots = p.max_slots;
    sa.M = M;
    sa.token_shift = p.token_shift;
#ifdef SK_TRACE
    sa.trace = g_sk_trace;
    if (g_sk_trace) g_sk_trace += 148 * 2 * 8;
#endif
    sa.fits32 = ((uint64_t)p.units + 1) * ((uint64_t)sa.gw_total + 1) < (uint64_t(1) << 32) ? 1 : 0;
    return sa;
}

#ifdef __CUDACC__
template <int BITS, int KIND, int TOK, int W, int OCC = 1, int DT = 0>
pot_status_t launch_stream(const void* packed, const void* scales, const void* zeros, int64_t N, int64_t K, int group,
                           const void* X, int M, void* Y, void* workspace, int* err, cudaStream_t s) {
    const StreamPlan p = plan_stream(N, K, M, BITS, group, KIND, TOK, W, OCC);
    if (!p.ok) return POT_ERR_SHAPE;
    const StreamArgs sa = stream_args(p, packed, scales, zeros, N, K, group, X, M, Y, workspace);
    auto run = [&](auto kernel) -> pot_status_t {
        if (!allow_max_dynamic_smem(kernel)) return POT_ERR_CUDA;
        return launch_pdl(kernel, dim3((unsigned)p.grid), dim3(W * 32), p.smem_bytes, s, sa, err);
    };
    if (p.q == 2) {
        if (p.x_in_smem) return run(stream_kernel<BITS, KIND, TOK, true, W, OCC, 2, DT>);
        return run(stream_kernel<BITS, KIND, TOK, false, W, OCC, 2, DT>);
    }
    if constexpr (OCC == 1 && TOK == 1) {
        if (p.q == 8) return run(stream_kernel<BITS, KIND, TOK, true, W, OCC, 8, DT>);  // only chosen with x in shared memory
    }
    if (p.x_in_smem) return run(stream_kernel<BITS, KIND, TOK, true, W, OCC, SK_QMAX, DT>);
    return run(stream_kernel<BITS, KIND, TOK, false, W, OCC, SK_QMAX, DT>);
}
#endif

}  // namespace pot
