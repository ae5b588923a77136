// Ring-buffered streaming kernel for the decode GEMV (PoT and the uniform twin) and the small-batch
// GEMM on the tiled layout; the multiply-accumulate runs on warp-level tensor-core MMAs.
//
// One persistent CTA per SM.  A producer warp streams the CTA's share of the packed codes from
// HBM into a shared-memory ring with 1-D bulk copies (cp.async.bulk + mbarrier transaction
// counts), several steps (up to 20 KB) per copy since the share is one contiguous byte range in the
// tiled layout; the bytes in flight therefore cost no registers, and the whole share of a short
// matrix can be requested before the first byte arrives.  Consumer warps take the ring stages
// round-robin, pull their share of the records out of shared memory (one word per lane and plane), decode
// them in registers (integer mask / shift-add into the scale's bit pattern) and accumulate in
// FP32 with warp-level MMAs whose A fragment is the decoded weights (B = the activation vector in
// every column for the GEMV, one token per column for the small batch).
//
// Work decomposition: the matrix is a sequence of steps; step g = 16 rows x 512 columns
// (row block g / spr, columns 512 * (g % spr)).  CTA b owns the contiguous range
// [b*G/grid, (b+1)*G/grid), so every SM streams the same number of bytes (+-1 step).  Each step
// yields 16 (x tokens) FP32 partial sums; when a row block needs more than one step they go to a
// slot of the workspace indexed by (row block, step) and the warp that delivers the last slot
// of a row block (a per-row-block counter tells it) adds the slots in ascending column order --
// the result is independent of timing.  No warp ever waits for another CTA.
//
// Every mbarrier wait is bounded: after kSpinLimit polls the waiter records an error code in
// *err (when given), and carries on without the data, so a lost copy cannot hang the GPU.
#pragma once
#include "common.cuh"
#include "layout.cuh"

namespace pot {

constexpr uint32_t kSpinLimit = 1u << 22;


enum RingMode { RG_POT_MMA = 2, RG_POT_MMA1 = 3, RG_POT_MMA1W = 4, RG_UINT_MMA1 = 5, RG_UINT_MMA1W = 6 };

constexpr int RG_Q = 5;  // steps per ring slot (one bulk copy) = warps per consumer group
// Consumer groups per CTA: slot m is consumed by group m % groups, warp i of it takes step i.  The tensor-core
// GEMV needs fewer registers per thread, so one more group of warps fits (RG_POT_MMA1W); whether that pays
// depends on how evenly the CTA's steps divide among the warps, see launch_gemv_mma.
__host__ __device__ constexpr int rg_groups(int mode) { return (mode == RG_POT_MMA1W || mode == RG_UINT_MMA1W) ? 4 : 3; }
__host__ __device__ constexpr int rg_consumers(int mode) { return rg_groups(mode) * RG_Q; }
__host__ __device__ constexpr int rg_threads(int mode) { return (rg_consumers(mode) + 1) * 32; }
__host__ __device__ constexpr int rg_unit_bytes(int bits) { return 256 * bits; }
__host__ __device__ constexpr int rg_slot_bytes(int bits) { return RG_Q * 4 * rg_unit_bytes(bits); }

struct RingPlan {
    int grid;
    int spr;
    int64_t total_steps;
    int stages;
    bool x_in_smem;
    size_t x_bytes;      // shared-memory bytes for the staged activations (0 if read from global)
    size_t cmb_bytes;    // shared-memory bytes for combining the steps of a row block inside the CTA (0 = off)
    size_t smem_bytes;   // total dynamic shared memory
    size_t ws_counters;
    size_t ws_bytes;
};

inline RingPlan plan_ring(int64_t N, int64_t K, int64_t M, int bits, int tok, int groups = 3) {
    RingPlan p;
    const int64_t nrb = N / 16, ncb = K / 128;
    p.spr = (int)((ncb + 3) / 4);
    p.total_steps = nrb * p.spr;
    p.grid = (int)(p.total_steps < kSmCount ? p.total_steps : kSmCount);
    // the small-batch mode stages a full tile of eight tokens (fragment order), whatever M is
    const size_t xb = (size_t)(tok > 1 ? tok : M) * (size_t)K * 2;
    p.x_in_smem = xb <= (tok > 1 ? 96 : 64) * 1024;
    p.x_bytes = p.x_in_smem ? (xb + 127) / 128 * 128 : 0;
    const int64_t per_cta = (p.total_steps + p.grid - 1) / p.grid;
    // per step one slot of 16*tok floats, plus one counter per local row block
    p.cmb_bytes = (size_t)(per_cta + 1) * 64 * (size_t)tok + (size_t)(per_cta / p.spr + 3) * 4;
    p.cmb_bytes = (p.cmb_bytes + 127) / 128 * 128;
    if (p.spr == 1 || p.cmb_bytes > 48 * 1024) p.cmb_bytes = 0;
    const size_t budget = 200 * 1024 - p.x_bytes - p.cmb_bytes - 1024;  // room for barriers and the runtime's reserve
    int64_t st = (int64_t)(budget / (size_t)rg_slot_bytes(bits));
    const int64_t slots_needed = (per_cta + RG_Q - 1) / RG_Q;
    if (st > 63) st = 63;
    // A slot that is reused must always come back to the same group of consumer warps (see the kernel):
    // the ring length is a multiple of the number of groups unless it holds the CTA's whole share.
    if (st >= slots_needed) st = slots_needed;
    else st = st / groups * groups;
    if (st < 1) st = 1;
    p.stages = (int)st;
    p.smem_bytes = 1024 + p.x_bytes + p.cmb_bytes + (size_t)p.stages * (size_t)rg_slot_bytes(bits);
    p.ws_counters = ((size_t)nrb * 4 + 255) / 256 * 256;
    p.ws_bytes = p.spr > 1 ? p.ws_counters + (size_t)nrb * (size_t)p.spr * 16 * (size_t)tok * 4 : 0;
    return p;
}

// ---- mbarrier / bulk-copy primitives ---------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// bounded wait: false after kSpinLimit unsuccessful polls
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}
// one non-blocking test (1 = the phase with this parity has completed)
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done;
}
// same, but polling with the non-blocking test_wait: a waiter that is parked inside try_wait can take on the
// order of a microsecond to resume, which is too slow for hand-offs that happen every few hundred cycles
__device__ __forceinline__ bool mbar_wait_spin(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
template <int NC>
__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(NC * 32) : "memory"); }

__device__ __forceinline__ void rg_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// MODE RG_POT_MMA1(W) / RG_UINT_MMA1(W): M = 1.  MODE RG_POT_MMA: M <= 8*MT tokens.
// RG_POT_MMA1 is the GEMV on the warp-level tensor-core path: the activation vector fills every column of the
// MMA's B operand, lane (gid, tig) owns quarter tig of the records of rows gid and gid + 8 -- exactly its share
// of the A fragment -- and the MMA adds up the four quarters, so there is no cross-lane reduction and the
// multiply-accumulate costs one instruction per 256 weights instead of one per weight.
struct RingArgs {
    const uint4* packed;
    const uint16_t* scales;
    const uint16_t* zeros;
    int64_t N, K;
    int G, spr;
    int64_t total_steps;
    int stages, x_bytes, cmb_bytes;
    const __half* X;
    int M;
    __half* Y;
    float* partial;
    unsigned* counters;
};

__device__ __forceinline__ void mbar_inval(uint32_t bar) { asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory"); }

// One GEMV / small-batch GEMM, executed by the whole CTA.  CHAIN = false: the body of a stand-alone launch (chained
// to its neighbours in the stream by programmatic dependent launch).  CHAIN = true: operation `op` of a persistent
// kernel that runs a list of dependent operations; `sync` is its grid-wide arrival counter: every CTA arrives when
// it has delivered its part of an operation, and the consumers of the next operation wait for all CTAs before
// they touch the activations (the producer warp does not wait: the weights are constants, it streams ahead).
template <int BITS, int MODE, int MT, int XMODE, bool CHAIN>  // XMODE: 0 = x from global, 1 = x staged in shared memory
__device__ __forceinline__ void ring_body(const RingArgs& ra, int* __restrict__ err, unsigned* sync, int op, int prev_stages) {
    const uint4* __restrict__ packed = ra.packed;
    const uint16_t* __restrict__ scales = ra.scales;
    const uint16_t* __restrict__ zeros = ra.zeros;
    const int64_t N = ra.N, K = ra.K;
    const int G = ra.G, spr = ra.spr;
    const int64_t total_steps = ra.total_steps;
    const int stages = ra.stages, x_bytes = ra.x_bytes, cmb_bytes = ra.cmb_bytes;
    const __half* __restrict__ X = ra.X;
    const int M = ra.M;
    __half* __restrict__ Y = ra.Y;
    float* __restrict__ partial = ra.partial;
    unsigned* __restrict__ counters = ra.counters;
    constexpr bool XSMEM = (XMODE != 0);
    constexpr bool MMA = (MODE == RG_POT_MMA);
    constexpr bool UNIFORM_TC = (MODE == RG_UINT_MMA1 || MODE == RG_UINT_MMA1W);  // the twin on the tensor-core path
    constexpr int RG_CONSUMERS = rg_consumers(MODE), RG_GROUPS = rg_groups(MODE);
    constexpr bool MMA1 = (MODE == RG_POT_MMA1 || MODE == RG_POT_MMA1W) || UNIFORM_TC;
    static_assert(!MMA || MT == 1, "one tile of eight tokens");
    constexpr int TOK = MMA ? 8 * MT : 1;
    constexpr int SLOT = rg_slot_bytes(BITS);
    constexpr int UB = rg_unit_bytes(BITS);
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);  // full[stages], empty[stages]  (<= 1024 bytes)
    const uint4* xs = reinterpret_cast<const uint4*>(smem + 1024);
    float* cmb = reinterpret_cast<float*>(smem + 1024 + x_bytes);  // [nsteps][16*TOK] partial slots, then counters
    unsigned char* ring = smem + 1024 + x_bytes + cmb_bytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t ncb = K / 128;
    const int64_t g_begin = (int64_t)blockIdx.x * total_steps / gridDim.x;
    const int64_t g_end = ((int64_t)blockIdx.x + 1) * total_steps / gridDim.x;
    const int nsteps = (int)(g_end - g_begin);
    const int nmacro = (nsteps + RG_Q - 1) / RG_Q;
    // global unit index (16 rows x 128 columns each, stored contiguously) at which step g starts
    auto unit_index = [&](int64_t g) -> int64_t {  // the step count fits 32 bits: cheap division
        const uint32_t rbq = (uint32_t)g / (uint32_t)spr;
        return (int64_t)rbq * ncb + 4 * (int64_t)((uint32_t)g - rbq * (uint32_t)spr);
    };

    if constexpr (CHAIN) {  // the previous operation's barriers (another ring length) make room first
        if ((int)threadIdx.x < 2 * prev_stages) mbar_inval(smem_u32(&bars[threadIdx.x]));
        __syncthreads();
    }
    if (threadIdx.x < stages) {  // one thread per ring slot
        mbar_init(smem_u32(&bars[threadIdx.x]), 1);                // full: the producer's expect_tx arrival
        mbar_init(smem_u32(&bars[stages + threadIdx.x]), RG_Q);    // empty: one arrival per consumed step
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    unsigned* cmb_cnt = reinterpret_cast<unsigned*>(cmb + (size_t)(nsteps + 1) * 16 * TOK);
    if (cmb_bytes) {
        for (int i = threadIdx.x; i < nsteps / spr + 3; i += blockDim.x) cmb_cnt[i] = 0u;
    }
    __syncthreads();
    if constexpr (!CHAIN) pdl_launch_dependents();

    if (warp == RG_CONSUMERS) {
        // ---------------- producer: weights do not depend on the previous kernel, start at once ----------
        if (lane == 0) {
            for (int m = 0; m < nmacro; ++m) {
                const int slot = m % stages;
                if (m >= stages) {
                    if (!mbar_wait(smem_u32(&bars[stages + slot]), (uint32_t)((m / stages - 1) & 1))) {
                        if (err) atomicCAS(err, 0, 1 | (m << 8) | (nsteps << 16));  // first failure wins
                    }
                }
                const int64_t gs = g_begin + (int64_t)m * RG_Q;
                const int64_t ge = gs + RG_Q < g_end ? gs + RG_Q : g_end;
                const int64_t u0 = unit_index(gs);
                const uint32_t bytes = (uint32_t)((unit_index(ge) - u0) * UB);
                const uint32_t full = smem_u32(&bars[slot]);
                mbar_expect_tx(full, bytes);
                bulk_g2s(smem_u32(ring + (size_t)slot * SLOT), packed + u0 * (16 * BITS), bytes, full);
            }
        }
    } else {
    // -------------------- consumers --------------------------------------------------------------------
    const int gid = lane >> 2, tig = lane & 3;  // MMA fragment coordinates: rows gid and gid + 8, quarter tig
    const int gpr = (int)(K / G);
    const int spg = 128 / G;

    // scales (and zero-points) of a step are fetched one step ahead, straight from global memory.  The
    // buffers keep the raw 16-bit loads: any arithmetic on them here would make the warp wait for the load.
    // sc1 / zp1: the scale (zero-point) of this lane's quarter, for both rows and the four units of a step
    uint32_t sc1[2][8], zp1[2][UNIFORM_TC ? 8 : 1];
    auto load_scales = [&](int64_t rb, int c, int buf) {
        // one 64-bit address per step; the eight loads use constant offsets from it
        const int64_t so = (rb * 16 + gid) * gpr + (int64_t)c * (4 * spg) + (spg == 2 ? (tig >> 1) : 0);
        const uint16_t* s0 = scales + so;
        const int64_t up = 8 * (int64_t)gpr;
        const int nu = (int)(ncb - 4 * (int64_t)c);  // units of this step (>= 4 except at the ragged end of a row)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                uint32_t v = 0x3C00u;
                if (u < nu) v = (uint32_t)__ldg(s0 + (h ? up : 0) + (spg == 2 ? 2 * u : u));
                sc1[buf][h * 4 + u] = v;
                if constexpr (UNIFORM_TC) {
                    uint32_t z = 0u;
                    if (u < nu) z = (uint32_t)__ldg(zeros + so + (h ? up : 0) + (spg == 2 ? 2 * u : u));
                    zp1[buf][h * 4 + u] = z;
                }
            }
    };
    // Slot (bulk copy) m holds steps m*Q .. m*Q+Q-1 and belongs to warp group m % GROUPS; warp i of the group
    // takes step m*Q + i.  A warp therefore meets the barriers of "its" slots once per fill and in order,
    // which is what the one-bit phase parity of an mbarrier requires.
    const int grp = warp / RG_Q, wig = warp - grp * RG_Q;
    const int j_first = grp * RG_Q + wig;             // this warp's first step (local index)
    constexpr int J_STRIDE = RG_GROUPS * RG_Q;         // distance between two of its steps (= RG_CONSUMERS)
    // (row block, step in row block) of this warp's current step, advanced without divisions
    int64_t rb = g_begin / spr;
    int c = (int)(g_begin - rb * spr) + j_first;
    while (c >= spr) { c -= spr; ++rb; }
    if (j_first < nsteps) load_scales(rb, c, 0);

    if constexpr (!CHAIN) {
        pdl_wait();  // x, Y and the workspace may belong to the previous kernel in the stream
    } else if (op > 0) {
        // every CTA must have delivered operation op - 1: `sync` counts arrivals since the kernel started
        if (threadIdx.x == 0) {
            const unsigned need = (unsigned)op * gridDim.x;
            bool ok = false;
            for (uint32_t i = 0; i < kSpinLimit && !ok; ++i) {
                unsigned v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(sync) : "memory");
                ok = v >= need;
            }
            if (!ok && err) atomicCAS(err, 0, 3 | (op << 8));
        }
        consumer_bar_sync<RG_CONSUMERS>();
    }
    if constexpr (XSMEM) {
        uint4* dst = reinterpret_cast<uint4*>(smem + 1024);
        const uint4* src = reinterpret_cast<const uint4*>(X);
        if constexpr (MMA) {
            // 16-byte chunk (token, unit, quarter t, part j) goes to ((unit * 4 + j) * 4 + t) * 8 + token: the 32
            // lanes of a warp (token = gid, t = tig) then read 512 contiguous bytes.  Tokens >= M stay unwritten:
            // their columns of the product are never delivered.
            const int kc = (int)(K / 8);
            constexpr int NT = RG_CONSUMERS * 32;
            for (int token = 0; token < M; ++token)
                for (int c0 = threadIdx.x; c0 < kc; c0 += 4 * NT) {  // four loads in flight per thread
                    uint4 v[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (c0 + i * NT < kc) v[i] = __ldg(src + (int64_t)token * kc + c0 + i * NT);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int cc = c0 + i * NT;
                        if (cc < kc) dst[((((cc >> 4) * 4 + (cc & 3)) * 4 + ((cc >> 2) & 3)) << 3) + token] = v[i];
                    }
                }
        } else {
            const int n16 = (int)(K / 8);
            for (int i = threadIdx.x; i < n16; i += RG_CONSUMERS * 32) {
                const uint4 v = __ldg(src + i);
                // chunk (quarter t, part j) of a unit goes to position j * 4 + t: the four lanes tig = 0..3 then read
                // 64 contiguous bytes
                dst[(i & ~15) | ((i & 3) << 2) | ((i >> 2) & 3)] = v;
            }
        }
        consumer_bar_sync<RG_CONSUMERS>();
    }

    const int64_t rb_first = g_begin / spr;
    int m = grp, slot = grp % stages;        // this warp's current slot fill, ring slot and barrier phase
    uint32_t phase = (uint32_t)((grp / stages) & 1);
    for (int j2 = j_first; j2 < nsteps; j2 += 2 * J_STRIDE) {
#pragma unroll
      for (int buf = 0; buf < 2; ++buf) {  // two steps per trip so that the scale buffers are indexed statically
        const int j = j2 + buf * J_STRIDE;
        if (j >= nsteps) break;
        int64_t rb_next = rb;
        int c_next = c + J_STRIDE;
        while (c_next >= spr) { c_next -= spr; ++rb_next; }
        if (j + J_STRIDE < nsteps) load_scales(rb_next, c_next, buf ^ 1);
        if (!mbar_wait(smem_u32(&bars[slot]), phase)) {
            if (err && lane == 0) atomicCAS(err, 0, 2 | (m << 8) | (warp << 16) | (j << 24));
        }
        float r0 = 0.f, r1 = 0.f;  // GEMV: the sums of rows gid and gid + 8
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        {
            // units between the slot's first step (wig steps back) and this one, without divisions
            int64_t rb_s = rb;
            int c_s = c - wig;
            while (c_s < 0) { c_s += spr; --rb_s; }
            const int64_t uoff = (rb * ncb + 4 * (int64_t)c) - (rb_s * ncb + 4 * (int64_t)c_s);
            // PoT: plane k of a unit holds word k of every (row, quarter): this lane's word sits at byte 4 * lane.
            // Uniform twin: the quarter's words sit at record words 2*tig, 2*tig+1 (n = 2), 2*tig, 2*tig+1, 8+tig
            // (n = 3) or 4*tig .. 4*tig+3 (n = 4); record word w is byte (w / 4) * 256 + row * 16 + (w % 4) * 4.
            const unsigned char* ubase = ring + (size_t)slot * SLOT + uoff * UB + (UNIFORM_TC ? gid * 16 : lane * 4);
            int woff[BITS];
#pragma unroll
            for (int k = 0; k < BITS; ++k) {
                const int w = BITS == 4 ? 4 * tig + k : (k < 2 ? 2 * tig + k : 8 + tig);
                woff[k] = UNIFORM_TC ? (w >> 2) * 256 + (w & 3) * 4 : k * 256;
            }
            float acc1[2][4];
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc1[i][e] = 0.f;
            // RELEASE_EARLY: the step's records are copied to registers and the slot is handed back before the
            // arithmetic (the small-batch mode has few slots, its activations take most of the shared memory)
            constexpr bool RELEASE_EARLY = MMA;
            uint32_t wreg[RELEASE_EARLY ? 4 : 1][2][BITS];
            if constexpr (RELEASE_EARLY) {
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int k = 0; k < BITS; ++k) {
                            wreg[u][h][k] = 0u;
                            if (4 * (int64_t)c + u < ncb)
                                wreg[u][h][k] = *reinterpret_cast<const uint32_t*>(ubase + u * UB + woff[k] + h * 128);
                        }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars[stages + slot]));  // one step of the slot is consumed
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int64_t cbu = 4 * (int64_t)c + u;
                if (cbu < ncb) {  // the same for the whole warp
                    uint32_t w[2][BITS];
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int k = 0; k < BITS; ++k) {
                            if constexpr (RELEASE_EARLY) w[h][k] = wreg[u][h][k];
                            else w[h][k] = *reinterpret_cast<const uint32_t*>(ubase + u * UB + woff[k] + h * 128);
                        }
                    uint32_t xq[16];  // 32 activations of quarter tig (of token gid): the B fragments of eight MMAs
                    if constexpr (MMA1) {
                        const uint4* xp = (XSMEM ? xs : reinterpret_cast<const uint4*>(X)) + cbu * 16 + (XSMEM ? tig : tig * 4);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint4 v = XSMEM ? xp[4 * i] : __ldg(xp + i);
                            xq[4 * i + 0] = v.x; xq[4 * i + 1] = v.y; xq[4 * i + 2] = v.z; xq[4 * i + 3] = v.w;
                        }
                    } else {
                        const uint4* xp = XSMEM ? xs + (cbu * 16 + tig) * 8 + gid
                                                : reinterpret_cast<const uint4*>(X) + (gid < M ? (int64_t)gid * (K / 8) : 0) + cbu * 16 + tig * 4;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 v = make_uint4(0, 0, 0, 0);
                            if (XSMEM) v = xp[32 * i];
                            else if (gid < M) v = __ldg(xp + i);
                            xq[4 * i + 0] = v.x; xq[4 * i + 1] = v.y; xq[4 * i + 2] = v.z; xq[4 * i + 3] = v.w;
                        }
                    }
                    uint32_t lo[16], hi[16];
                    if constexpr (UNIFORM_TC) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            // the quarter's words, placed where uint_decode_pairs16 looks for blocks 0 and 1
                            uint32_t q[BITS == 3 ? 9 : BITS];
#pragma unroll
                            for (int k = 0; k < BITS; ++k) q[(BITS == 3 && k == 2) ? 8 : k] = w[h][k];
                            potl::UintParams pr;
                            pr.s2 = potl::bits_h2(sc1[buf][h * 4 + u] * 0x10001u);
                            pr.z = potl::bits_h2(zp1[buf][h * 4 + u] * 0x10001u);
                            uint32_t a8[8], b8[8];
                            potl::uint_decode_pairs16<BITS>(q, 0, pr, a8);
                            potl::uint_decode_pairs16<BITS>(q, 1, pr, b8);
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                (h ? hi : lo)[i] = a8[i];
                                (h ? hi : lo)[8 + i] = b8[i];
                            }
                        }
                    } else {
                        potl::pot_decode32<BITS, 1>(w[0], 0, sc1[buf][u] * 0x10001u, lo);
                        potl::pot_decode32<BITS, 1>(w[1], 0, sc1[buf][4 + u] * 0x10001u, hi);
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j)  // two accumulators: half the length of the dependent chain
                        rg_mma(acc1[j & 1], lo[2 * j], hi[2 * j], lo[2 * j + 1], hi[2 * j + 1], xq[2 * j], xq[2 * j + 1]);
                }
            }
            if constexpr (!RELEASE_EARLY) {
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars[stages + slot]));  // one step of the slot is consumed
            }
            r0 = acc1[0][0] + acc1[1][0];   // GEMV: every column of the product holds the same sums
            r1 = acc1[0][2] + acc1[1][2];
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[e] = acc1[0][e] + acc1[1][e];
        }
        // ---- deliver the step's partial sums -----------------------------------------------------------
        // spr == 1: the step is the whole row block, write Y.  Otherwise the 16*TOK sums go to a slot:
        // in shared memory when every step of the row block belongs to this CTA (the common case),
        // else in the global workspace; whoever fills the last slot adds them in ascending column order.
        const bool whole = (spr == 1);
        const int64_t rb_g0 = rb * spr;  // first step of this row block
        const bool local = cmb_bytes && rb_g0 >= g_begin && rb_g0 + spr <= g_end;
        float* pslot = whole ? nullptr
                            : (local ? cmb + (size_t)(rb_g0 - g_begin + c) * (16 * TOK)
                                     : partial + (rb_g0 + c) * (16 * TOK));
        if (!MMA) {
            if (tig == 0) {
                if (whole) {
                    Y[rb * 16 + gid] = __float2half_rn(r0);
                    Y[rb * 16 + gid + 8] = __float2half_rn(r1);
                } else {
                    pslot[gid] = r0;
                    pslot[gid + 8] = r1;
                }
            }
        } else {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int row = gid + 8 * (e >> 1), token = 8 * mt + 2 * tig + (e & 1);
                    if (whole) {
                        if (token < M) Y[(int64_t)token * N + rb * 16 + row] = __float2half_rn(acc[4 * mt + e]);
                    } else {
                        if (token < M) pslot[token * 16 + row] = acc[4 * mt + e];
                    }
                }
        }
        if (!whole) {
            unsigned prev = 0;
            if (local) {
                __threadfence_block();
                __syncwarp();
                if (lane == 0) prev = atomicAdd(&cmb_cnt[rb - rb_first], 1u);
            } else {
                __threadfence();
                __syncwarp();
                if (lane == 0) prev = atomicAdd(&counters[rb], 1u);
            }
            prev = __shfl_sync(0xffffffffu, prev, 0);
            if (prev == (unsigned)spr - 1u) {  // this warp delivered the last slot of the row block
                if (local) __threadfence_block(); else __threadfence();
                const float* first = local ? cmb + (size_t)(rb_g0 - g_begin) * (16 * TOK) : partial + rb_g0 * (16 * TOK);
                for (int e = lane; e < 16 * (MMA ? M : 1); e += 32) {
                    const int row = e & 15, token = e >> 4;
                    float sum = 0.f;
                    if (local) {
                        for (int q = 0; q < spr; ++q) sum += first[(size_t)q * (16 * TOK) + e];
                    } else {
                        for (int q = 0; q < spr; ++q) sum += __ldcg(first + (size_t)q * (16 * TOK) + e);
                    }
                    if (token < M) Y[(int64_t)token * N + rb * 16 + row] = __float2half_rn(sum);
                }
                if (!local && lane == 0) counters[rb] = 0u;  // leave the workspace ready for the next call
            }
        }
        rb = rb_next;
        c = c_next;
        m += RG_GROUPS;
        slot += RG_GROUPS;
        while (slot >= stages) { slot -= stages; phase ^= 1u; }
      }
    }
    }  // consumers
    if constexpr (CHAIN) {
        __syncthreads();  // the CTA's part of this operation is delivered (and its ring and barriers are idle)
        if (threadIdx.x == 0) {
            __threadfence();
            atomicAdd(sync, 1u);
        }
    }
}

template <int BITS, int MODE, int MT, int XMODE>
__global__ void __launch_bounds__(rg_threads(MODE), 1)
ring_kernel(const RingArgs ra, int* __restrict__ err) {
    ring_body<BITS, MODE, MT, XMODE, false>(ra, err, nullptr, 0, 0);
}

// Persistent kernel over a list of dependent GEMVs (PoT codes, tiled layout, M = 1, activations staged in shared
// memory): one launch instead of one per operation.  Launched cooperatively (all CTAs resident), since the CTAs wait
// for one another between operations.  sync[0]: arrivals (see ring_body), sync[1]: CTAs that have finished the list;
// the last of them puts both back to zero for the next launch.
template <int BITS>
__global__ void __launch_bounds__(rg_threads(RG_POT_MMA1), 1)
ring_chain_kernel(const RingArgs* __restrict__ ops, int n_ops, unsigned* sync, int* __restrict__ err) {
    int prev_stages = 0;
    for (int op = 0; op < n_ops; ++op) {
        const RingArgs ra = ops[op];
        ring_body<BITS, RG_POT_MMA1, 1, 1, true>(ra, err, sync, op, prev_stages);
        prev_stages = ra.stages;
    }
    if (threadIdx.x == 0) {
        const unsigned d = atomicAdd(sync + 1, 1u);
        if (d == gridDim.x - 1) {  // every CTA has left its last wait
            sync[0] = 0u;
            sync[1] = 0u;
            __threadfence();
        }
    }
}

// Device error word shared by the ring kernels (0 = no bounded wait ever gave up).  One copy per
// translation unit that includes this header; ring_error_ptr() returns this GPU's address of it.
static __device__ int g_ring_error;
inline int* ring_error_ptr() {
    static std::atomic<int*> cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    int* p = cache[dev].load(std::memory_order_acquire);
    if (!p) {
        void* q = nullptr;
        if (cudaGetSymbolAddress(&q, g_ring_error) != cudaSuccess) return nullptr;
        p = (int*)q;
        cache[dev].store(p, std::memory_order_release);
    }
    return p;
}
// Reads and clears the error word (synchronises the device).  -1 if it cannot be read.
inline int ring_error_fetch() {
    int v = -1, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_ring_error, sizeof(int)) != cudaSuccess) return -1;
    cudaMemcpyToSymbol(g_ring_error, &zero, sizeof(int));
    return v;
}

// Host side.  `err` may be nullptr.
inline RingArgs ring_args(const RingPlan& p, const void* packed, const void* scales, const void* zeros, int64_t N, int64_t K,
                          int group, const void* X, int M, void* Y, void* workspace) {
    RingArgs ra;
    ra.packed = (const uint4*)packed;
    ra.scales = (const uint16_t*)scales;
    ra.zeros = (const uint16_t*)zeros;
    ra.N = N; ra.K = K; ra.G = group; ra.spr = p.spr;
    ra.total_steps = p.total_steps;
    ra.stages = p.stages; ra.x_bytes = (int)p.x_bytes; ra.cmb_bytes = (int)p.cmb_bytes;
    ra.X = (const __half*)X; ra.M = M; ra.Y = (__half*)Y;
    ra.counters = (unsigned*)workspace;
    ra.partial = workspace ? (float*)((char*)workspace + p.ws_counters) : nullptr;
    return ra;
}
template <int BITS, int MODE, int MT>
pot_status_t launch_ring(const void* packed, const void* scales, const void* zeros, int64_t N, int64_t K, int group,
                         const void* X, int M, void* Y, void* workspace, int* err, cudaStream_t s) {
    const RingPlan p = plan_ring(N, K, M, BITS, MODE == RG_POT_MMA ? 8 * MT : 1, rg_groups(MODE));
    auto run = [&](auto kernel) -> pot_status_t {
        if (!allow_max_dynamic_smem(kernel)) return POT_ERR_CUDA;
        const RingArgs ra = ring_args(p, packed, scales, zeros, N, K, group, X, M, Y, workspace);
        return launch_pdl(kernel, dim3((unsigned)p.grid), dim3(rg_threads(MODE)), p.smem_bytes, s, ra, err);
    };
    if (p.x_in_smem) return run(ring_kernel<BITS, MODE, MT, 1>);
    return run(ring_kernel<BITS, MODE, MT, 0>);
}

// GEMV on the warp-level tensor-core path with 15 or 20 consumer warps: a warp works through whole steps, so the
// time is (steps per warp, rounded up) x (time per step, about 1.2 x longer when 20 warps share the SM).
template <int BITS, bool UNIFORM_CODES = false>
pot_status_t launch_gemv_mma(const void* packed, const void* scales, const void* zeros, int64_t N, int64_t K, int group,
                             const void* x, void* y, void* workspace, int* err, cudaStream_t s) {
    const RingPlan p = plan_ring(N, K, 1, BITS, 1, 3);
    const int64_t per_cta = (p.total_steps + p.grid - 1) / p.grid;
    const double t3 = (double)((per_cta + 14) / 15), t4 = 1.2 * (double)((per_cta + 19) / 20);
    constexpr int NARROW = UNIFORM_CODES ? RG_UINT_MMA1 : RG_POT_MMA1, WIDE = UNIFORM_CODES ? RG_UINT_MMA1W : RG_POT_MMA1W;
    if (t4 < t3) return launch_ring<BITS, WIDE, 1>(packed, scales, zeros, N, K, group, x, 1, y, workspace, err, s);
    return launch_ring<BITS, NARROW, 1>(packed, scales, zeros, N, K, group, x, 1, y, workspace, err, s);
}

}  // namespace pot
