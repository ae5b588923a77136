// Prefill GEMM on 5th-generation tensor cores: Y[M,N] = X[M,K] W~^T, FP16 in, FP32 accumulate in
// tensor memory, FP16 out, with the PoT dequantization fused in (tiled weight layout).
//
// One CTA (one per SM) computes a 256-token x 128-feature tile of Y.  Per 64-wide K block (one pipeline stage, 48 KB;
// four stages):
//   warp 0 (one lane)  : TMA loads of the two X tiles (64-column boxes, 128-byte swizzle) into the stage;
//   warps 4..19        : "dequant producers", four groups of four warps that take the stages in turn -- each thread
//                        fetches the 32 codes of one weight row that the stage needs (8-byte loads from the tiled
//                        layout, prefetched three of the group's stages ahead), decodes them in registers with the
//                        mask / shift-add trick of Sec. 4.2 and writes the FP16 values into the stage's weight tile in
//                        exactly the layout the tensor core expects (K-major, 8-row x 128-byte atoms, 16-byte chunks
//                        XOR-swizzled with the row index), then fence.proxy.async + mbarrier arrive;
//   warps 1, 2 (one lane each) : the two MMA issuers take alternate stages; each waits for both operands, issues four
//                        tcgen05.mma (A = the 128 decoded weight rows, B = the 256 tokens: M = 128, N = 256, K = 16) into
//                        ITS OWN 256 columns of tensor memory (lane = weight row, column = token) and tcgen05.commit's
//                        the stage back to the producers.  One issuing thread leaves the tensor pipe idle for several
//                        hundred cycles per stage (barrier test, fence, commit, the pipe's start-up after a gap); two
//                        threads fill each other's gaps.
// After the last K block each issuer commits to a common barrier; the producer warps read the accumulators with
// tcgen05.ld (each warp its own 32-lane quarter), add the two issuers' sums in a fixed order, convert to FP16 and
// store (a warp writes 32 consecutive features of one token at a time).  The weights are re-decoded once per 256-token
// tile (M / 256 times overall), which is the price of never writing FP16 weights to HBM.
// By default the decoded weight tile of the large-M kernel does not go through shared memory at all (AT = 1): the
// producers -- two groups then -- write it into tensor memory (tcgen05.st, lane = weight row, 32 columns per stage behind
// the 256 accumulator columns) and the MMAs take their A operand from there; a stage of shared memory holds X only (six
// stages of 32 KB); both issuers work on every stage, issuer J multiplying the tile by token tile J into its own 128
// columns (see pf_issue_at).  The description above is the shared-memory-tile kernel, kept for the one-token-tile
// variant and as a selectable alternative.
// Batches of up to 64 tokens run a variant with one tile of M token rows (the TMA box holds exactly M rows, the MMA's
// N is M rounded up to 16), eight 24 KB stages and two TMA threads; with the weight ring in tensor memory: six stages that
// are whole 128-column blocks (two X tiles = 16 KB, 64 columns of weights, eight MMAs) and three producer groups.
//
// All mbarrier waits are bounded (see sync.cuh); a wait that gives up records a code and the CTA carries
// on, so a lost transaction cannot hang the GPU.  Tensor memory is released on every path.
#include <cuda.h>

#include <cstdlib>
#include <cstring>

#include <type_traits>

#include "common.cuh"
#include "layout.cuh"
#include "sync.cuh"

namespace pot {

constexpr int PF_BM = 128;      // tokens per X tile (TMA box rows; one MMA covers one or two of them as its N side)
constexpr int PF_MT = 2;        // X tiles per CTA of the large-M kernel: 256 tokens share one decoded weight tile
constexpr int PF_BN = 128;      // features (weight rows) per tile: the MMA's M side, the accumulator's lanes
constexpr int PF_SMALL_TOKENS = 64;     // largest batch of the one-token-tile kernel (its X stage holds 64 rows)
constexpr int PF_BK = 64;       // half a column block per stage (one 128-byte swizzle atom wide)
// Warps: 0 = TMA, 1 .. NI = MMA issuers, then (from a warp index that is a multiple of 2 or 4, so that warp & 3 walks the
// tensor-memory lane quarters in step) NG groups of four dequant / epilogue warps.
__host__ __device__ constexpr int pf_prod_warp0(int ni) { return ni == 2 ? 4 : 2; }
__host__ __device__ constexpr int pf_threads(int ng, int ni) { return (pf_prod_warp0(ni) + 4 * ng) * 32; }
constexpr int PF_ATOM_BYTES = 128 * 128;             // 128 rows x 64 halves
// a stage: MT X tiles (token tiles) + one weight tile
// (the one-tile kernel serves up to PF_SMALL_TOKENS tokens: 8 KB of X per stage, so that eight stages fit)
__host__ __device__ constexpr int pf_x_bytes(int mt) { return mt == 1 ? PF_SMALL_TOKENS * 128 : mt * PF_ATOM_BYTES; }
// (at = 1: the decoded weight tile lives in tensor memory, a stage of shared memory holds the X tiles only)
// K sub-blocks of 64 columns per stage: two in the one-tile kernel with the weight ring in tensor memory (a stage is then a
// whole 128-column block: half as many stage visits per byte for every role), one otherwise
// (wide = 1 asks for them in the 256-token kernel too: for a single wave of tiles, where the stage visits and not the tensor
// pipe set the pace)
__host__ __device__ constexpr int pf_bks(int mt, int at, int wide = 0) { return (at && (mt == 1 || wide)) ? 2 : 1; }
__host__ __device__ constexpr int pf_stage_bytes(int mt, int at = 0, int wide = 0) { return pf_x_bytes(mt) * pf_bks(mt, at, wide) + (at ? 0 : PF_ATOM_BYTES); }
constexpr size_t pf_smem_bytes(int stages, int mt, int at = 0, int wide = 0) { return 1024 /*align slack*/ + (size_t)stages * pf_stage_bytes(mt, at, wide) + 256 /*barriers*/; }
constexpr int PF_AT_ACC_COLS = 256;   // at = 1, 256-token tiles: accumulator columns (token t of the tile = column t), then 32 columns per stage of A
// at = 1, the one-tile kernel (up to 64 tokens): the two issuers' accumulators take 64 columns each, the A ring follows
constexpr int PF_AT1_ACC_STRIDE = PF_SMALL_TOKENS;
__host__ __device__ constexpr int pf_at_ring_col0(int mt) { return mt == 2 ? PF_AT_ACC_COLS : 2 * PF_AT1_ACC_STRIDE; }

// UMMA instruction descriptor: FP16 x FP16 -> FP32, both operands K-major, M = 128 (the weight rows of the tile are the
// A operand), N = n token rows of the X tile (the B operand), 16 <= n <= 256, n % 16 == 0
// (dt = 1: BF16 x BF16 -> FP32)
__host__ __device__ constexpr uint32_t pf_idesc(uint32_t n, uint32_t dt = 0) {
    return (1u << 4) /*D = F32*/ | (dt << 7) /*A = F16 / BF16*/ | (dt << 10) /*B = F16 / BF16*/ | ((n >> 3) << 17) |
           ((uint32_t)(PF_BN >> 4) << 24);
}

// FP32 sum -> FP16 (DT = 0) or BF16 (DT = 1) bit pattern, round to nearest even
template <int DT>
__device__ __forceinline__ uint16_t pf_out(float v) {
    if (DT == 0) return __half_as_ushort(__float2half_rn(v));
    return __bfloat16_as_ushort(__float2bfloat16_rn(v));
}

// shared-memory matrix descriptor, K-major, 128-byte swizzle: start >> 4, LBO = 1 (unused), SBO = 1024 B
// between 8-row groups, descriptor version 1, layout type 2 (SWIZZLE_128B)
__device__ __forceinline__ uint64_t pf_smem_desc(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)2 << 61);
}

// the descriptor's high word does not depend on the address
constexpr uint64_t PF_DESC_CONST = ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);

__device__ __forceinline__ void pf_tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                 "l"(map), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}
// tcgen05.mma, the two operand descriptors given as their low words + the common high word
__device__ __forceinline__ void pf_mma2(uint32_t d_tmem, uint32_t alo, uint32_t blo, uint32_t hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem),
        "r"(alo), "r"(blo), "r"(hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The producers' prefetch loads as volatile statements: issued exactly once and where the source puts them (ahead of the
// wait for the stage), never re-materialised behind it.
__device__ __forceinline__ uint2 pf_ldg_v2(const uint2* p) {
    uint2 v;
    asm volatile("ld.global.nc.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ uint4 pf_ldg_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t pf_ldg_u16(const uint16_t* p) {
    uint16_t v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return (uint32_t)v;
}
__device__ __forceinline__ void pf_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void pf_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,"
        "%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

// tcgen05.mma with the A operand in tensor memory (lane = row of A, one 32-bit column = two K elements)
__device__ __forceinline__ void pf_mma_ta(uint32_t d_tmem, uint32_t a_tmem, uint32_t blo, uint32_t hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "r"(blo), "r"(hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void pf_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,"
        "%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
        "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
        "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
        "r"(r[31])
        : "memory");
}

// Issuer J of the variant that keeps the decoded weight tile in tensor memory: it takes EVERY stage, multiplies the tile
// (A, from tensor memory: 128 weight rows x 64) by token tile J of the stage (B, 128 tokens, from shared memory) and
// accumulates into columns 128 J .. 128 J + 127 -- the two issuers share the weight tile and never the accumulator, so
// the order of the additions is fixed.  A stage is free again when every active issuer's MMAs on it have completed.
template <int J, int PF_STAGES, int DT, int BKS = 1>
__device__ __forceinline__ void pf_issue_at(uint32_t smem0, uint32_t bar0, uint32_t tmem_base, int nkb, int* err) {
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (PF_STAGES + s); };
    const uint32_t accum = bar0 + 8u * (2 * PF_STAGES);
    uint32_t blo[PF_STAGES];
#pragma unroll
    for (int s = 0; s < PF_STAGES; ++s)
        blo[s] = (uint32_t)pf_smem_desc(smem0 + (uint32_t)s * pf_stage_bytes(PF_MT, 1, BKS == 2) + (uint32_t)J * PF_ATOM_BYTES);
    constexpr uint32_t desc_hi = (uint32_t)(PF_DESC_CONST >> 32);
    constexpr uint32_t SLOT = 32u * BKS;   // tensor-memory columns of a stage's weights
    const uint32_t d0 = tmem_base + (uint32_t)(J * PF_BM);
    const uint32_t a0 = tmem_base + (uint32_t)PF_AT_ACC_COLS;
    const uint32_t idesc = pf_idesc(PF_BM, DT);
    uint32_t ready = mbar_test(full(0), 0);
    uint32_t ph = 0;
    for (int kb0 = 0; kb0 < nkb; kb0 += PF_STAGES, ph ^= 1u) {
#pragma unroll
        for (int s = 0; s < PF_STAGES; ++s) {
            const int kb = kb0 + s;
            if (kb >= nkb) break;
            if (!ready && !mbar_wait(full(s), ph)) {
                if (err) atomicCAS(err, 0, 0x20 | (kb << 8));
            }
            ready = 0;
            if (kb + 1 < nkb) ready = mbar_test(full((s + 1) % PF_STAGES), s + 1 >= PF_STAGES ? ph ^ 1u : ph);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int ks = 0; ks < BKS * (PF_BK / 16); ++ks)   // sub-block ks / 4: its X tiles follow the first sub-block's
                pf_mma_ta(d0, a0 + SLOT * (uint32_t)s + (uint32_t)(8 * ks),
                          blo[s] + (uint32_t)(((ks >> 2) * PF_MT * PF_ATOM_BYTES + (ks & 3) * 32) >> 4), desc_hi, idesc,
                          (s != 0 || ks != 0) ? 1u : (uint32_t)(kb0 != 0));
            pf_commit(empty(s));
        }
    }
    pf_commit(accum);
}

// Issuer J of the one-tile kernel with the weight tile in tensor memory: as pf_issue (alternate stages, its own
// accumulator -- 64 columns at 64 J), with the A operand taken from the stage's 32 columns of the ring.
template <int J, int NI, int PF_STAGES, int DT>
__device__ __forceinline__ void pf_issue_at1(uint32_t smem0, uint32_t bar0, uint32_t tmem_base, int nkb, uint32_t n_tok, int* err) {
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (PF_STAGES + s); };
    const uint32_t accum = bar0 + 8u * (2 * PF_STAGES);
    uint32_t blo[PF_STAGES];
#pragma unroll
    for (int s = 0; s < PF_STAGES; ++s) blo[s] = (uint32_t)pf_smem_desc(smem0 + (uint32_t)s * pf_stage_bytes(1, 1));
    constexpr uint32_t desc_hi = (uint32_t)(PF_DESC_CONST >> 32);
    constexpr int BKS = pf_bks(1, 1);                       // 64-column sub-blocks per stage
    constexpr uint32_t SLOT = 32u * BKS;                    // tensor-memory columns of a stage's weights
    const uint32_t d0 = tmem_base + (uint32_t)(J * PF_AT1_ACC_STRIDE);
    const uint32_t a0 = tmem_base + (uint32_t)pf_at_ring_col0(1);
    const uint32_t idesc = pf_idesc(n_tok, DT);
    uint32_t ready = mbar_test(full(J), 0);
    uint32_t ph = 0;
    for (int kb0 = 0; kb0 < nkb; kb0 += PF_STAGES, ph ^= 1u) {
#pragma unroll
        for (int s = J; s < PF_STAGES; s += NI) {
            const int kb = kb0 + s;
            if (kb >= nkb) break;
            if (!ready && !mbar_wait(full(s), ph)) {
                if (err) atomicCAS(err, 0, 0x20 | (kb << 8));
            }
            ready = 0;
            if (kb + NI < nkb) ready = mbar_test(full((s + NI) % PF_STAGES), s + NI >= PF_STAGES ? ph ^ 1u : ph);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int ks = 0; ks < BKS * (PF_BK / 16); ++ks)   // sub-block ks / 4 of the stage: its own X tile, the next 32 columns of A
                pf_mma_ta(d0, a0 + SLOT * (uint32_t)s + (uint32_t)(8 * ks),
                          blo[s] + (uint32_t)(((ks >> 2) * pf_x_bytes(1) + (ks & 3) * 32) >> 4), desc_hi, idesc,
                          (s != J || ks != 0) ? 1u : (uint32_t)(kb0 != 0));
            pf_commit(empty(s));
        }
    }
    pf_commit(accum);
}

// The MMA issuer J of NI (one thread): takes the stages kb = J, J + NI, ... of the CTA's nkb stages and accumulates them
// into its own accumulator (128 weight rows = lanes, n_tok token columns).  One thread's dependent instructions retire every ~5 cycles and the tensor pipe
// idles meanwhile, so what the loop needs per MMA is prepared first: the low descriptor word of every stage's tiles (the
// high word is a constant); the loop is unrolled over the stages so that these stay in registers and a K step is one
// add.  A barrier test costs a few hundred cycles even when the phase is long complete, so the test for the issuer's
// next stage is put in flight before the MMAs of this one are issued and examined afterwards.
template <int J, int NI, int PF_STAGES, int MT, int DT = 0>
__device__ __forceinline__ void pf_issue(uint32_t smem0, uint32_t bar0, uint32_t tmem_base, int nkb, uint32_t n_tok, int* err) {
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (PF_STAGES + s); };
    const uint32_t accum = bar0 + 8u * (2 * PF_STAGES);
    uint32_t alo[PF_STAGES], blo[PF_STAGES];
#pragma unroll
    for (int s = 0; s < PF_STAGES; ++s) {
        const uint32_t a = smem0 + (uint32_t)s * pf_stage_bytes(MT);
        alo[s] = (uint32_t)pf_smem_desc(a);
        blo[s] = (uint32_t)pf_smem_desc(a + pf_x_bytes(MT));
    }
    constexpr uint32_t desc_hi = (uint32_t)(PF_DESC_CONST >> 32);
    const uint32_t d0 = tmem_base + (uint32_t)(J * PF_BM * MT);   // this issuer's accumulator: 128 features x (128 MT) token columns
    const uint32_t idesc = pf_idesc(n_tok, DT);
    uint32_t ready = mbar_test(full(J), 0);
    uint32_t ph = 0;
    for (int kb0 = 0; kb0 < nkb; kb0 += PF_STAGES, ph ^= 1u) {
#pragma unroll
        for (int s = J; s < PF_STAGES; s += NI) {
            const int kb = kb0 + s;
            if (kb >= nkb) break;
            if (!ready && !mbar_wait(full(s), ph)) {
                if (err) atomicCAS(err, 0, 0x20 | (kb << 8));
            }
            ready = 0;
            if (kb + NI < nkb) ready = mbar_test(full((s + NI) % PF_STAGES), s + NI >= PF_STAGES ? ph ^ 1u : ph);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int ks = 0; ks < PF_BK / 16; ++ks)  // A = the decoded weight tile, B = the X tile(s): one MMA covers all tokens
                pf_mma2(d0, blo[s] + (uint32_t)((ks * 32) >> 4), alo[s] + (uint32_t)((ks * 32) >> 4), desc_hi, idesc,
                        (s != J || ks != 0) ? 1u : (uint32_t)(kb0 != 0));
            pf_commit(empty(s));  // the stage is free again once these MMAs have read it
        }
    }
    pf_commit(accum);  // this issuer's accumulators are complete once all its MMAs have finished
}

// PF_STAGES stages, NG producer groups (K block kb is decoded by group kb % NG into stage kb % PF_STAGES), NI issuers with
// their own accumulators, MT token tiles of 128 per CTA.  PF_STAGES is a multiple of NG and of NI: a stage buffer is
// always filled by the same group, loaded by the same TMA thread and read by the same issuer, so every parity wait is
// made by a thread that has itself seen the barrier's previous phase (a waiter two phases behind could not tell).
// Instantiated as <bits, 4, 4, 2, 2> (M > 64: 256-token tiles, four 48 KB stages) and <bits, 8, 4, 2, 1> (M <= 64: one
// tile of up to 64 tokens, eight 24 KB stages -- a stage buffer's round trip producer -> issuer -> tensor pipe ->
// producer is ~2000 cycles whatever the tile holds, so more buffers = more stages per unit of time).
// AT = 1 (MT = 2, NI = 2 only): the producers write the decoded weight tile into tensor memory (tcgen05.st) instead of
// shared memory and the MMAs take their A operand from there, which removes a third of the shared-memory traffic of a
// stage (16 KB written + 16 KB read of 96 KB); see pf_issue_at for the issuers' division of work.  Instantiated as
// <bits, 6, 2, 2, 2, dt, 1>: 256 accumulator columns + 6 x 32 columns of A = 448 of the 512 columns.
// NGP of the NG groups decode, the others only take part in the epilogue (measured slower than NGP = NG = 2 -- the
// waiting groups poll the accumulator barrier through the whole main loop -- and not instantiated).
template <int BITS, int PF_STAGES, int NG, int NI, int MT, int DT = 0, int AT = 0, int NGP = NG, int WIDE = 0>  // DT = 1: BF16 activations, weights and output
__global__ void __launch_bounds__(pf_threads(NG, NI), 1)
pot_gemm_prefill_kernel(const __grid_constant__ CUtensorMap xmap, const uint4* __restrict__ packed,
                        const uint16_t* __restrict__ scales, int64_t N, int64_t K, int G, int64_t M,
                        uint16_t* __restrict__ Y, float* __restrict__ partial, unsigned* __restrict__ counters,
                        int tiles_m, int n_full, int tail_splits, int* __restrict__ err) {
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment: the swizzle atoms and the matrix descriptors assume it
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    static_assert(AT == 0 || NI == 2, "the tensor-memory weight tile is built for two issuers");
    constexpr bool AT2 = AT && MT == 2;   // both issuers on every stage, one token tile each (else: alternate stages)
    constexpr int BKS = pf_bks(MT, AT, WIDE);   // 64-column sub-blocks per stage
    constexpr int STAGE_BYTES = pf_stage_bytes(MT, AT, WIDE);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)PF_STAGES * STAGE_BYTES);
    // bars: full[S] (TMA bytes + one arrival per producer warp), empty[S], accum, then the tensor-memory base address
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * PF_STAGES + 1);
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (PF_STAGES + s); };
    const uint32_t accum = bar0 + 8u * (2 * PF_STAGES);

    constexpr int PROD_WARP0 = pf_prod_warp0(NI);
    constexpr int NPT = NG * 128;                       // producer / epilogue threads
    constexpr int TMEM_COLS = AT ? 512 : NI * PF_BN * MT;  // MT accumulators per issuer; AT: 256 accumulator columns + the A ring
    static_assert((NGP % 2 == 0 || BKS == 2) && NGP <= NG && (AT2 || PF_STAGES % NI == 0) && PF_STAGES % NGP == 0,
                  "a group always decodes the same half of a column block; a stage buffer belongs to one issuer and one group");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Work items in launch order: the first n_full are whole output tiles; each of the remaining ("tail") tiles is cut
    // into tail_splits items along K, so that the last, partly filled wave of CTAs is short.  Tiles are numbered
    // with the token tile running fastest (CTAs that decode the same weight tile run together).
    auto item = [&](int& tile, int& zsplit, int& splits) {
        if ((int)blockIdx.x < n_full) {
            tile = (int)blockIdx.x; zsplit = 0; splits = 1;
        } else {
            const int j = (int)blockIdx.x - n_full;
            tile = n_full + j / tail_splits; zsplit = j % tail_splits; splits = tail_splits;
        }
    };
    int64_t m0, n0, cb0, cb1;
    {
        int tile, zsplit, splits;
        item(tile, zsplit, splits);
        m0 = (int64_t)(tile % tiles_m) * (PF_BM * MT);
        n0 = (int64_t)(tile / tiles_m) * PF_BN;
        // split item z of a tile owns column blocks [cb0, cb1), two stages each
        cb0 = (int64_t)zsplit * (K / 128) / splits;
        cb1 = ((int64_t)zsplit + 1) * (K / 128) / splits;
    }
    const int64_t ncb = K / 128;
    // a tile with at most 128 real tokens (decode batches, the ragged last token tile) uses one accumulator only
    const int n_mt = M - m0 > PF_BM ? MT : 1;
    // token rows the MMA reads from the X stage: whole tiles, or (one-tile kernel) the batch rounded up to the MMA's N step
    const uint32_t n_tok = MT == 1 ? (uint32_t)((M + 15) & ~(int64_t)15) : (uint32_t)(n_mt * PF_BM);  // MT == 1: M <= 64
    const int nkb = (int)((2 / BKS) * (cb1 - cb0));   // stages of this item
    const int kb0 = (int)((2 / BKS) * cb0);

    // ---- dequant producers, part 1 (before the set-up below, so that the first loads of codes and scales -- constants,
    // they do not depend on the previous kernel -- are in flight while the barriers and the tensor memory are set up and
    // the kernel waits for its predecessor): thread = one weight row; group g owns the stages with kb % NGP == g, hence
    // (NGP is even) always the same half of the records.
    const int pt = threadIdx.x - 32 * PROD_WARP0;          // 0 .. NPT-1 for the producer warps
    const int grp = pt >> 7, row = pt & 127, half = grp & 1;
    const int64_t n = n0 + row;
    const bool row_ok = n < N;
    const int64_t rb = n >> 4;
    const int r = (int)(n & 15);
    const int spg = 128 / G;
    // The packed codes are prefetched PF_DEPTH - 1 of the group's stages ahead.  Every 16-byte plane of the
    // row holds one word of each quarter; the group needs quarters 2*grp and 2*grp + 1: 8 bytes per plane.
    // (A double-width stage -- BKS = 2 -- takes the whole record: 16 bytes per plane, and both groups' scales.)
    constexpr int PF_DEPTH = BKS == 2 ? 3 : 4;
    uint32_t rec[PF_DEPTH][2 * BKS * BITS];
    uint32_t sc2[PF_DEPTH][BKS];
    auto load = [&](int kb, int buf) {
        if (row_ok) {
            const int64_t cbx = cb0 + (BKS == 2 ? kb : (kb >> 1));   // the stage's column block
            // tiled scales: the unit's values sit together, rows r and r + 8 of a group in one word
            const int64_t so = (rb * ncb + cbx) * (16 * spg);
            if constexpr (BKS == 2) {
                const uint4* unit = packed + (rb * ncb + cbx) * (16 * BITS);
#pragma unroll
                for (int t = 0; t < BITS; ++t) {
                    const uint4 q = pf_ldg_v4(unit + t * 16 + r);
                    rec[buf][4 * t + 0] = q.x; rec[buf][4 * t + 1] = q.y; rec[buf][4 * t + 2] = q.z; rec[buf][4 * t + 3] = q.w;
                }
                sc2[buf][0] = pf_ldg_u16(scales + so + potl::scale_tile_index(r, 0));
                sc2[buf][BKS - 1] = pf_ldg_u16(scales + so + potl::scale_tile_index(r, spg == 2 ? 1 : 0));
            } else {
                const uint2* unit = reinterpret_cast<const uint2*>(packed + (rb * ncb + cbx) * (16 * BITS));
#pragma unroll
                for (int t = 0; t < BITS; ++t) {
                    const uint2 q = pf_ldg_v2(unit + (t * 16 + r) * 2 + half);
                    rec[buf][2 * t + 0] = q.x; rec[buf][2 * t + 1] = q.y;
                }
                sc2[buf][0] = pf_ldg_u16(scales + so + potl::scale_tile_index(r, spg == 2 ? half : 0));  // raw bits: any arithmetic here would stall on the load
            }
        }
    };
    const int nmine = (warp >= PROD_WARP0 && grp < NGP && nkb > grp) ? (nkb - grp + NGP - 1) / NGP : 0;   // stages kb = grp, grp + NGP, ...
#pragma unroll
    for (int p = 0; p < PF_DEPTH - 1; ++p)
        if (p < nmine) load(NGP * p + grp, p);

    if (threadIdx.x == 0) {
        for (int s = 0; s < PF_STAGES; ++s) {
            mbar_init(full(s), 1 + 4);  // the TMA thread's expect_tx arrival + one arrival per warp of the group that fills the stage
            mbar_init(empty(s), AT2 ? n_mt : 1);  // AT2: every active issuer reads every stage
        }
        mbar_init(accum, AT2 ? n_mt : NI);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // allocate the accumulator columns of tensor memory (whole warp), base address lands in shared memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0 || (NI == 2 && warp == 3)) {
        // ---------------- TMA producers: MT X tiles (64 columns x 128 tokens each) per stage ----------------
        // One thread needs ~600 cycles per stage (barrier wait, expect_tx, TMA instruction: three long latencies in a
        // row), which paces batches of a few tokens; there warp 3 (idle next to two issuers) takes every other
        // stage.  With big boxes the TMA unit is the slower part and a second thread only adds contention.
        const int n_tma = (NI == 2 && MT == 1) ? 2 : 1;
        if (lane == 0 && (warp == 0 || n_tma == 2)) {
            uint32_t ready = 0;  // the test of the next stage's barrier is in flight while this stage's copies are issued
            for (int kb = warp == 0 ? 0 : 1; kb < nkb; kb += n_tma) {
                const int s = kb % PF_STAGES;
                if (kb >= PF_STAGES && !ready && !mbar_wait(empty(s), (uint32_t)((kb / PF_STAGES - 1) & 1))) {
                    if (err) atomicCAS(err, 0, 0x10 | (kb << 8));
                }
                const int kn = kb + n_tma;
                ready = (kn < nkb && kn >= PF_STAGES) ? mbar_test(empty(kn % PF_STAGES), (uint32_t)((kn / PF_STAGES - 1) & 1)) : 0u;
                // MT == 1 (M <= 64): the box holds exactly the M token rows -- the TMA unit spends time on every row of a
                // box, in range or not; the rows of the tile that nothing writes belong to tokens that are never stored
                mbar_expect_tx(full(s), MT == 1 ? (uint32_t)M * 128u * BKS : (uint32_t)n_mt * PF_ATOM_BYTES * BKS);
                const uint32_t a = smem_u32(smem + (size_t)s * STAGE_BYTES);
                if constexpr (BKS == 2 && MT == 1) {  // (one-tile kernel) the two 64-column tiles of the stage's column block
                    pf_tma_load_2d(a, &xmap, (kb0 + kb) * 2 * PF_BK, (int)m0, full(s));
                    pf_tma_load_2d(a + pf_x_bytes(1), &xmap, (kb0 + kb) * 2 * PF_BK + PF_BK, (int)m0, full(s));
                } else if constexpr (BKS == 2) {      // [sub-block][token tile] tiles of 16 KB
#pragma unroll
                    for (int sub = 0; sub < 2; ++sub)
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
                            if (mt < n_mt)
                                pf_tma_load_2d(a + (sub * MT + mt) * PF_ATOM_BYTES, &xmap, ((kb0 + kb) * 2 + sub) * PF_BK, (int)m0 + mt * PF_BM, full(s));
                } else {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
                        if (mt < n_mt) pf_tma_load_2d(a + mt * PF_ATOM_BYTES, &xmap, (kb0 + kb) * PF_BK, (int)m0 + mt * PF_BM, full(s));
                }
            }
        }
    } else if (warp <= NI) {
        // ---------------- MMA issuers (one thread each) ------------------------------------------------
        if (lane == 0) {
            if constexpr (AT2) {
                if (warp == 1) pf_issue_at<0, PF_STAGES, DT, BKS>(smem_u32(smem), bar0, tmem_base, nkb, err);
                else if (n_mt == 2) pf_issue_at<1, PF_STAGES, DT, BKS>(smem_u32(smem), bar0, tmem_base, nkb, err);
            } else if constexpr (AT) {
                if (warp == 1) pf_issue_at1<0, NI, PF_STAGES, DT>(smem_u32(smem), bar0, tmem_base, nkb, n_tok, err);
                else pf_issue_at1<NI - 1, NI, PF_STAGES, DT>(smem_u32(smem), bar0, tmem_base, nkb, n_tok, err);
            } else {
                if (NI == 1 || warp == 1) pf_issue<0, NI, PF_STAGES, MT, DT>(smem_u32(smem), bar0, tmem_base, nkb, n_tok, err);
                else pf_issue<NI - 1, NI, PF_STAGES, MT, DT>(smem_u32(smem), bar0, tmem_base, nkb, n_tok, err);
            }
        }
    } else if (warp >= PROD_WARP0) {
        // ---------------- dequant producers, part 2 (then epilogue) -----------------------------------
        // The groups of four warps take the stages in turn: a stage visit costs a warp a fixed ~1000 cycles of
        // hand-off latency (barrier test, fence, arrive), so more stages must be in preparation at once.
        // Stage kb covers columns 64*kb .. 64*kb+63, i.e. half (kb & 1) of column block kb / 2.
        for (int i4 = 0; i4 < nmine; i4 += PF_DEPTH) {
#pragma unroll
            for (int buf = 0; buf < PF_DEPTH; ++buf) {
                const int i = i4 + buf;
                if (i >= nmine) break;
                const int kb = NGP * i + grp;
                if (i + PF_DEPTH - 1 < nmine) load(kb + NGP * (PF_DEPTH - 1), (buf + PF_DEPTH - 1) % PF_DEPTH);
                const int s = kb % PF_STAGES;
                if (kb >= PF_STAGES) {
                    // Every lane polls (the warp is about to WRITE the stage).  One polling lane + __syncwarp() left the
                    // warp running as two groups (lane 0 / the rest) through the whole decode in some builds: every
                    // load and store issued twice.
                    if (!mbar_wait(empty(s), (uint32_t)((kb / PF_STAGES - 1) & 1))) {
                        if (err && lane == 0) atomicCAS(err, 0, 0x30 | (kb << 8));
                    }
                    __syncwarp();
                }
                if constexpr (AT && BKS == 2) {
                    // a whole record: the two 64-column halves in turn, 32 packed pairs = 32 columns of this thread's lane each
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");  // (behind the wait for the stage)
#pragma unroll
                    for (int hb = 0; hb < 2; ++hb) {
                        uint32_t sh = sc2[buf][hb];
                        if (DT == 1) sh = __bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half((uint16_t)sh))));
                        const uint32_t sh2 = sh * 0x10001u;
                        uint32_t wa[32];
#pragma unroll
                        for (int T2 = 0; T2 < 2; ++T2) {
                            uint32_t w2[16];
                            if (row_ok) {
                                if (DT == 0) potl::pot_decode32<BITS, 4>(rec[buf], 2 * hb + T2, sh2, w2);
                                else potl::pot_decode32_bf16<BITS, 4>(rec[buf], 2 * hb + T2, sh2, w2);
                            } else {
#pragma unroll
                                for (int q = 0; q < 16; ++q) w2[q] = 0u;
                            }
#pragma unroll
                            for (int q = 0; q < 16; ++q) wa[16 * T2 + q] = w2[q];
                        }
                        pf_st32(tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(pf_at_ring_col0(MT) + 64 * s + 32 * hb), wa);
                    }
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(full(s));
                    continue;
                }
                uint32_t s16 = sc2[buf][0];
                if (DT == 1) s16 = __bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half((uint16_t)s16))));
                const uint32_t s2 = s16 * 0x10001u;  // scale pattern in both halves
                if constexpr (AT) {
                    // the row's 64 weights of this stage = 32 packed pairs = 32 columns of this thread's tensor-memory lane
                    uint32_t wa[32];
#pragma unroll
                    for (int T2 = 0; T2 < 2; ++T2) {
                        uint32_t w2[16];
                        if (row_ok) {
                            if (DT == 0) potl::pot_decode32<BITS, 2>(rec[buf], T2, s2, w2);
                            else potl::pot_decode32_bf16<BITS, 2>(rec[buf], T2, s2, w2);
                        } else {
#pragma unroll
                            for (int q = 0; q < 16; ++q) w2[q] = 0u;
                        }
#pragma unroll
                        for (int q = 0; q < 16; ++q) wa[16 * T2 + q] = w2[q];
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");  // (behind the wait for the stage)
                    pf_st32(tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(pf_at_ring_col0(MT) + 32 * s), wa);
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(full(s));
                    continue;
                }
                unsigned char* brow = smem + (size_t)s * STAGE_BYTES + pf_x_bytes(MT) + row * 128;
#pragma unroll
                for (int T2 = 0; T2 < 2; ++T2) {
                    uint32_t w2[16];
                    if (row_ok) {
                        if (DT == 0) potl::pot_decode32<BITS, 2>(rec[buf], T2, s2, w2);
                        else potl::pot_decode32_bf16<BITS, 2>(rec[buf], T2, s2, w2);
                    } else {
#pragma unroll
                        for (int q = 0; q < 16; ++q) w2[q] = 0u;
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {  // 4 chunks of 8 halves; chunk index inside the 128-byte row
                        const int chunk = 4 * T2 + c;
                        *reinterpret_cast<uint4*>(brow + ((chunk ^ (row & 7)) << 4)) =
                            make_uint4(w2[4 * c], w2[4 * c + 1], w2[4 * c + 2], w2[4 * c + 3]);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(full(s));
            }
        }
        // ---------------- epilogue: tensor memory -> registers -> FP16 -> Y --------------------------
        if (!mbar_wait(accum, 0)) {
            if (err) atomicCAS(err, 0, 0x40);
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // A bounded wait that gave up (here or in any CTA of the launch) has left its code in the error word: a tile that may
        // have been built from a stage that never arrived is not stored.  (The roles' loops themselves carry on to their
        // bounds: control flow added to them costs the tensor pipe several per cent.)
        const bool gave_up = err != nullptr && *reinterpret_cast<volatile int*>(err) != 0;
        // Lane = weight row (feature), column = token.  Warp (q, part): features n0 + 32 q .. + 31 (a warp may only touch its
        // own quarter of the lanes), token columns part * 32 CH .. + 32 CH - 1 (CH chunks of 32 per warp).
        const int q = warp & 3;
        const int part = (warp - PROD_WARP0) >> 2;
        const int64_t feat = n0 + 32 * q + lane;
        int tile, zsplit, splits;  // recomputed here rather than kept in registers across the main loop
        item(tile, zsplit, splits);
        const int tail_index = tile - n_full;   // index of the tile among the split ones
        const int64_t rows_alloc = M < PF_BM * MT ? M : PF_BM * MT;  // token rows kept per tile in the workspace
        // 32-column chunks per warp: the NG warps of a lane quarter share the tile's columns (the one-tile kernel holds at
        // most PF_SMALL_TOKENS tokens: two chunks, whatever NG is)
        // (chunks part, part + NG, ... of the tile's 32-column chunks; the one-tile kernel holds at most PF_SMALL_TOKENS tokens)
        constexpr int NCH = MT == 1 ? PF_SMALL_TOKENS / 32 : MT * PF_BM / 32;
        constexpr int CH = (NCH + NG - 1) / NG;
#pragma unroll
        for (int cc = 0; cc < CH; ++cc) {
            if (part + cc * NG >= NCH) break;
            const int col = (part + cc * NG) * 32;
            if (m0 + col >= M) break;             // (warp-uniform) no token in these columns
            uint32_t v[32];
            pf_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)col, v);
            if (NI == 2 && !AT2 && nkb > 1) {     // add the second issuer's sums (odd K blocks) to the first's: a fixed order
                                                  // (an item of a single stage -- K = 128 with 128-column stages -- has none)
                uint32_t v1[32];
                pf_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)((AT ? PF_AT1_ACC_STRIDE : PF_BM * MT) + col), v1);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) + __uint_as_float(v1[i]));
            } else {
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            }
            if (feat < N && !gave_up && in_range(m0 + col < M && m0 >= 0 && feat >= 0 && (splits == 1 || (tail_index >= 0 && zsplit >= 0 && zsplit < splits)), err, 0x60)) {
                if (splits == 1) {  // a warp stores 32 consecutive features (64 bytes) of one token at a time
                    uint16_t* dst = Y + (m0 + col) * N + feat;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (m0 + col + i < M) dst[(int64_t)i * N] = pf_out<DT>(__uint_as_float(v[i]));
                } else {  // this split's partial sums: [tail tile][split][token of the tile][128 features] FP32
                    float* dst = partial + (((int64_t)tail_index * splits + zsplit) * rows_alloc + col) * PF_BN + (32 * q + lane);
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (m0 + col + i < M) dst[(int64_t)i * PF_BN] = __uint_as_float(v[i]);
                }
            }
        }
        if (splits > 1 && !gave_up && in_range(tail_index >= 0 && partial != nullptr && counters != nullptr, err, 0x61)) {
            // The CTA that delivers the last split of a tile (an arrival counter tells it) adds the splits in
            // ascending order -- the result does not depend on timing -- and writes Y.
            __shared__ unsigned s_prev;
            __threadfence();
            asm volatile("bar.sync 2, %0;" ::"n"(NPT) : "memory");
            if (threadIdx.x == 32 * PROD_WARP0) s_prev = atomicAdd(&counters[tail_index], 1u);
            asm volatile("bar.sync 2, %0;" ::"n"(NPT) : "memory");
            if (s_prev == (unsigned)splits - 1u) {
                __threadfence();
                // The epilogue threads walk the tile in 16-byte pieces, consecutive threads on consecutive
                // pieces (coalesced), four pieces per thread in flight; the splits are added in ascending order.
                const float* tile0 = partial + (int64_t)tail_index * splits * rows_alloc * PF_BN;
                const int64_t split_stride = rows_alloc * PF_BN;
                const int npieces = (int)(rows_alloc * PF_BN / 4);
                for (int p0 = pt; p0 < npieces; p0 += 4 * NPT) {
                    float4 acc4[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) acc4[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int z = 0; z < splits; ++z) {
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int pc = p0 + u * NPT;
                            if (pc < npieces) {
                                const float4 t = __ldcg(reinterpret_cast<const float4*>(tile0 + z * split_stride) + pc);
                                acc4[u].x += t.x; acc4[u].y += t.y; acc4[u].z += t.z; acc4[u].w += t.w;
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int pc = p0 + u * NPT;
                        const int64_t row = m0 + pc / (PF_BN / 4), colx = n0 + 4 * (pc % (PF_BN / 4));
                        if (pc < npieces && row < M && colx < N) {  // N % 16 == 0: a piece is inside or outside as a whole
                            const uint32_t h0 = (uint32_t)pf_out<DT>(acc4[u].x) | ((uint32_t)pf_out<DT>(acc4[u].y) << 16);
                            const uint32_t h1 = (uint32_t)pf_out<DT>(acc4[u].z) | ((uint32_t)pf_out<DT>(acc4[u].w) << 16);
                            *reinterpret_cast<uint2*>(Y + row * N + colx) = make_uint2(h0, h1);
                        }
                    }
                }
                if (threadIdx.x == 32 * PROD_WARP0) counters[tail_index] = 0u;  // leave the workspace ready for the next call
            }
        }
    }
    // ---------------- teardown: everyone is done with tensor memory, the allocating warp frees it --------
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(TMEM_COLS) : "memory");
    }
}

// cuTensorMapEncodeTiled, looked up through the runtime so that the library does not link against libcuda
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
    static std::atomic<EncodeTiledFn> cache{nullptr};
    EncodeTiledFn f = cache.load(std::memory_order_acquire);
    if (!f) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess || !p) return nullptr;
        f = (EncodeTiledFn)p;
        cache.store(f, std::memory_order_release);
    }
    return f;
}

bool gemm_prefill_supported(int64_t M, int64_t N, int64_t K, int bits, int group) {
    (void)bits; (void)group;
    // TMA needs the X row pitch (2K bytes) to be a multiple of 16 -- implied by K % 128 == 0 -- and 32-bit box coordinates
    return M > 0 && N % 16 == 0 && K % 128 == 0 && M < (int64_t(1) << 31) && K < (int64_t(1) << 31);
}
// How the output tiles become work items.  One CTA per SM (148 slots); the tiles of the last, partly filled wave -- or all
// tiles when they cover at most half of the SMs -- are cut along K into `splits` items each (FP32 partial sums + an
// arrival counter per such tile in the workspace), at least four column blocks per item.
struct PrefillPlan {
    int tiles_m, tiles, n_full, n_tail, splits;
    int64_t rows_alloc;
    size_t counter_bytes, ws_bytes;
};
static PrefillPlan prefill_plan(int64_t M, int64_t N, int64_t K) {
    PrefillPlan p{};
    p.tiles_m = (int)((M + PF_BM * PF_MT - 1) / (PF_BM * PF_MT));
    p.tiles = p.tiles_m * (int)((N + PF_BN - 1) / PF_BN);
    const int slots = kSmCount;
    const int rem = p.tiles % slots;
    int tail = 0;
    if (2 * p.tiles <= slots) tail = p.tiles;            // small problem: every tile is split
    else if (p.tiles > slots && rem > 0 && 2 * rem <= slots) tail = rem;  // the last wave fills at most half of the slots
    int64_t s = tail > 0 ? slots / tail : 1;
    const int64_t max_by_k = (K / 128) / 4;
    if (s > max_by_k) s = max_by_k;
    if (s > 8 && tail != p.tiles) s = 8;
    if (s > 16) s = 16;
    if (s < 2) { s = 1; tail = 0; }
    p.splits = (int)s;
    p.n_tail = tail;
    p.n_full = p.tiles - tail;
    p.rows_alloc = M < PF_BM * PF_MT ? M : PF_BM * PF_MT;
    p.counter_bytes = tail ? ((size_t)tail * 4 + 255) / 256 * 256 : 0;
    p.ws_bytes = tail ? p.counter_bytes + (size_t)tail * (size_t)s * (size_t)p.rows_alloc * PF_BN * 4 : 0;
    return p;
}
// arrival counters (must start at zero; the kernel leaves them at zero) + FP32 partial sums of the split tiles
size_t gemm_prefill_workspace(int64_t M, int64_t N, int64_t K, int, int) { return prefill_plan(M, N, K).ws_bytes; }

static int* prefill_error_ptr();

// Where the large-M kernel keeps the decoded weight tile: in tensor memory (the producers write it with tcgen05.st, the
// MMAs read their A operand there).  That takes a third of the traffic off shared memory, and a stage of shared memory
// then holds X only, so six stages fit instead of four, and two producer groups keep up: measured 0.85 - 0.88 of the
// cuBLAS burst figure on the six 70B points against 0.80 - 0.86 with the tile in shared memory (four stages, four
// groups).  POT_PREFILL_WEIGHT_TILE = smem selects the shared-memory kernel (a diagnostic switch: the tests run all variants).
static bool prefill_weight_tile_in_tmem() {
    const char* e = getenv("POT_PREFILL_WEIGHT_TILE");
    return !(e && e[0] == 's');
}
// POT_PREFILL_WEIGHT_TILE = tmem-narrow keeps the 256-token kernel on its 64-column stages even for a single wave of CTAs
// (diagnostic: the tests run that kernel on small shapes this way)
static bool prefill_wide_stages_allowed() {
    const char* e = getenv("POT_PREFILL_WEIGHT_TILE");
    return !(e && strcmp(e, "tmem-narrow") == 0);
}

pot_status_t gemm_prefill_launch(const void* packed, const void* scales, int64_t N, int64_t K, int bits, int group,
                                 const void* X, int64_t M, void* Y, void* workspace, size_t ws_bytes, cudaStream_t s, int dt) {
    const PrefillPlan pl = prefill_plan(M, N, K);
    if (pl.ws_bytes > 0 && (!workspace || ws_bytes < pl.ws_bytes)) return POT_ERR_WORKSPACE;
    unsigned* counters = (unsigned*)workspace;
    float* partial = pl.ws_bytes > 0 ? (float*)((char*)workspace + pl.counter_bytes) : nullptr;
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return POT_ERR_CUDA;
    CUtensorMap xmap;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)(M <= PF_SMALL_TOKENS ? M : PF_BM)};  // the one-tile kernel: no padding rows
    const cuuint32_t estr[2] = {1, 1};
    if (encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(X), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return POT_ERR_CUDA;
    const dim3 grid((unsigned)(pl.n_full + pl.n_tail * pl.splits));
    auto run = [&](auto kernel, int stages, int mt, int at = 0, int ng = 4, int wide = 0) -> pot_status_t {
        const size_t smem = pf_smem_bytes(stages, mt, at, wide);
        const dim3 block((unsigned)pf_threads(ng, 2));
        if (!allow_max_dynamic_smem(kernel)) return POT_ERR_CUDA;
        return launch_pdl(kernel, grid, block, smem, s, xmap, (const uint4*)packed, (const uint16_t*)scales, N, K, group, M,
                          (uint16_t*)Y, partial, counters, pl.tiles_m, pl.n_full, pl.splits, prefill_error_ptr());
    };
    // two issuers, one CTA per SM; for batches of up to 64 tokens: one token tile, three producer groups, six stages of a whole
    // 128-column block with the weight ring in tensor memory (four groups, eight 24 KB stages with the tile in shared memory)
    if (dt == 1) {
        if (M <= PF_SMALL_TOKENS && prefill_weight_tile_in_tmem()) {
            if (bits == 2) return run(pot_gemm_prefill_kernel<2, 6, 3, 2, 1, 1, 1>, 6, 1, 1, 3);
            if (bits == 3) return run(pot_gemm_prefill_kernel<3, 6, 3, 2, 1, 1, 1>, 6, 1, 1, 3);
            return run(pot_gemm_prefill_kernel<4, 6, 3, 2, 1, 1, 1>, 6, 1, 1, 3);
        }
        if (M <= PF_SMALL_TOKENS) {
            if (bits == 2) return run(pot_gemm_prefill_kernel<2, 8, 4, 2, 1, 1>, 8, 1);
            if (bits == 3) return run(pot_gemm_prefill_kernel<3, 8, 4, 2, 1, 1>, 8, 1);
            return run(pot_gemm_prefill_kernel<4, 8, 4, 2, 1, 1>, 8, 1);
        }
        if (prefill_weight_tile_in_tmem() && grid.x <= (unsigned)kSmCount && prefill_wide_stages_allowed()) {
            if (bits == 2) return run(pot_gemm_prefill_kernel<2, 3, 3, 2, 2, 1, 1, 3, 1>, 3, 2, 1, 3, 1);
            if (bits == 3) return run(pot_gemm_prefill_kernel<3, 3, 3, 2, 2, 1, 1, 3, 1>, 3, 2, 1, 3, 1);
            return run(pot_gemm_prefill_kernel<4, 3, 3, 2, 2, 1, 1, 3, 1>, 3, 2, 1, 3, 1);
        }
        if (prefill_weight_tile_in_tmem()) {
            if (bits == 2) return run(pot_gemm_prefill_kernel<2, 6, 2, 2, 2, 1, 1>, 6, 2, 1, 2);
            if (bits == 3) return run(pot_gemm_prefill_kernel<3, 6, 2, 2, 2, 1, 1>, 6, 2, 1, 2);
            return run(pot_gemm_prefill_kernel<4, 6, 2, 2, 2, 1, 1>, 6, 2, 1, 2);
        }
        if (bits == 2) return run(pot_gemm_prefill_kernel<2, 4, 4, 2, 2, 1>, 4, 2);
        if (bits == 3) return run(pot_gemm_prefill_kernel<3, 4, 4, 2, 2, 1>, 4, 2);
        return run(pot_gemm_prefill_kernel<4, 4, 4, 2, 2, 1>, 4, 2);
    }
    if (M <= PF_SMALL_TOKENS && prefill_weight_tile_in_tmem()) {  // six stages of a whole 128-column block (16 KB of X), three producer groups; the A ring fills tensor memory
        if (bits == 2) return run(pot_gemm_prefill_kernel<2, 6, 3, 2, 1, 0, 1>, 6, 1, 1, 3);
        if (bits == 3) return run(pot_gemm_prefill_kernel<3, 6, 3, 2, 1, 0, 1>, 6, 1, 1, 3);
        return run(pot_gemm_prefill_kernel<4, 6, 3, 2, 1, 0, 1>, 6, 1, 1, 3);
    }
    if (M <= PF_SMALL_TOKENS) {
        if (bits == 2) return run(pot_gemm_prefill_kernel<2, 8, 4, 2, 1>, 8, 1);
        if (bits == 3) return run(pot_gemm_prefill_kernel<3, 8, 4, 2, 1>, 8, 1);
        return run(pot_gemm_prefill_kernel<4, 8, 4, 2, 1>, 8, 1);
    }
    // A single wave of CTAs (65 .. 256 tokens on decode-sized matrices) is paced by the stage visits, not by the tensor
    // pipe: three stages of a whole 128-column block (64 KB of X, 64 columns of weights, three producer groups), as in the
    // one-tile kernel (15360 x 5120 at 65 .. 128 tokens: 27.5 - 28.5 -> 22.2 - 23.1 us).
    const bool one_wave = grid.x <= (unsigned)kSmCount && prefill_wide_stages_allowed();
    if (prefill_weight_tile_in_tmem() && one_wave) {
        if (bits == 2) return run(pot_gemm_prefill_kernel<2, 3, 3, 2, 2, 0, 1, 3, 1>, 3, 2, 1, 3, 1);
        if (bits == 3) return run(pot_gemm_prefill_kernel<3, 3, 3, 2, 2, 0, 1, 3, 1>, 3, 2, 1, 3, 1);
        return run(pot_gemm_prefill_kernel<4, 3, 3, 2, 2, 0, 1, 3, 1>, 3, 2, 1, 3, 1);
    }
    if (prefill_weight_tile_in_tmem()) {  // two producer groups, six stages (32 KB of X each), the A ring in tensor memory
        if (bits == 2) return run(pot_gemm_prefill_kernel<2, 6, 2, 2, 2, 0, 1>, 6, 2, 1, 2);
        if (bits == 3) return run(pot_gemm_prefill_kernel<3, 6, 2, 2, 2, 0, 1>, 6, 2, 1, 2);
        return run(pot_gemm_prefill_kernel<4, 6, 2, 2, 2, 0, 1>, 6, 2, 1, 2);
    }
    if (bits == 2) return run(pot_gemm_prefill_kernel<2, 4, 4, 2, 2>, 4, 2);
    if (bits == 3) return run(pot_gemm_prefill_kernel<3, 4, 4, 2, 2>, 4, 2);
    return run(pot_gemm_prefill_kernel<4, 4, 4, 2, 2>, 4, 2);
}

static int* prefill_error_ptr() { return error_ptr(ERR_PREFILL); }

}  // namespace pot

// Diagnostic: reads and clears the device error word of the prefill kernel (0 = every bounded wait completed;
// 0x10 / 0x20 / 0x30 / 0x40 in the low byte = the TMA warp / the MMA warp / a dequant warp / the epilogue gave
// up waiting, bits 8.. = the K block).  Synchronises the device.
