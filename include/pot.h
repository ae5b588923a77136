/*
 * pot.h -- C ABI of the B200 (sm_100a) PoT-PTQ inference library.
 *
 * The library implements the inference hot path of PoT-PTQ: n-bit power-of-two weight codes
 * (one sign bit + an (n-1)-bit exponent E, one FP16 scale S per group of G weights along the
 * reduction dimension) are unpacked to FP16/BF16 with integer bit manipulation and either
 * stored (pot_dequant) or consumed directly by a GEMV / GEMM.
 *
 * Notation (paper, Sec. 3.1): W is [N, K] row-major, N = output features, K = input features
 * (the reduction dimension); y = W x.  Groups are G contiguous elements of a row.
 * q_max = 2^(n-1) - 1.  A code is  sign << (n-1) | E  (the paper's "S0 E1 E2" for n = 3).
 *
 * General conventions
 *   - Unless a parameter is marked HOST, every data pointer is a DEVICE pointer owned by the
 *     caller.  The library allocates nothing, keeps no per-call state and never synchronises;
 *     every call enqueues its work on `stream` (a cudaStream_t passed as void*, NULL = the
 *     default stream) and returns.
 *   - Argument errors are detected on the host and returned BEFORE anything is launched.
 *     POT_ERR_CUDA reports a failed launch.  Kernels never trap.
 *   - Base pointers must be 16-byte aligned.  K % 128 == 0 and K % G == 0, bits in {2,3,4},
 *     G in {64,128}.  (K % 128 == 0 makes every packed row a multiple of 16 bytes.)
 *   - Scale contract: every scale is a normal FP16 number whose exponent field e satisfies
 *     1 <= e and e + q_max <= 30, i.e. S in [2^-14, (2 - 2^-10) * 2^(15 - q_max)].  Inside that
 *     range adding E to the exponent field is exactly multiplication by 2^E; outside it
 *     (zero, subnormal, too large) the results are unspecified but no call faults.
 *     pot_quantize_ref never produces an illegal scale; pot_validate_scales counts them.
 *
 * Interchange ("canonical") layout of the codes -- the paper does not specify one:
 *   row i is a little-endian bit stream of K*n/8 bytes; code k occupies bits [n*k, n*k+n)
 *   counted from the least significant bit of byte 0.  Example, n = 3: codes
 *   011,101,000,111,000,010,100,000 -> bytes 2B 0E 11.   Scales: [N, K/G] row-major FP16.
 *
 * Kernel ("tiled") layout, produced by pot_repack: a size-preserving bijection of the same
 * bits (exactly n bits per weight, no padding) that lets a warp fetch the codes of a
 * 16-row x 128-column block with fully coalesced 16-byte loads and place two weights in a
 * 32-bit lane with one mask and one shift-add.  It requires N % 16 == 0.  See pot_repack.
 */
#ifndef POT_B200_H
#define POT_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    POT_OK = 0,
    POT_ERR_NULL = 1,        /* a required pointer is NULL                                   */
    POT_ERR_UNSUPPORTED = 2, /* bits not in {2,3,4}, G not in {64,128}, unknown enum value   */
    POT_ERR_SHAPE = 3,       /* N, M <= 0; K % 128 != 0; K % G != 0; tiled layout with N % 16 */
    POT_ERR_ALIGN = 4,       /* a base pointer is not 16-byte aligned                        */
    POT_ERR_WORKSPACE = 5,   /* workspace NULL or smaller than the *_workspace_bytes value   */
    POT_ERR_SCALE_RANGE = 6, /* reserved for callers that act on pot_validate_scales          */
    POT_ERR_CUDA = 7         /* the CUDA runtime reported an error for this call's launch     */
} pot_status_t;

typedef enum { POT_F16 = 0, POT_BF16 = 1 } pot_dtype_t;

/* How pot_quantize_ref chooses the group scale (paper: scale search is Algorithm 1). */
typedef enum {
    POT_SCALE_TOP = 0,      /* S = max|w| * 2^-q_max : the top level 2^q_max * S sits on max|w| */
    POT_SCALE_PAPER_S0 = 1, /* S = fp16(max|w| / (2^q_max - 1)) : Algorithm 1's s0 with b = 1   */
    POT_SCALE_GIVEN = 2,    /* S is supplied by the caller (must satisfy the scale contract)    */
    POT_SCALE_SEARCH = 3    /* S = s0 * b*, b* from Algorithm 1's 200-point grid search          */
} pot_scale_rule_t;

typedef enum { POT_LAYOUT_CANONICAL = 0, POT_LAYOUT_TILED = 1 } pot_layout_t;

/* Which uniform-INT dequantization kernel to run (same result, bit for bit). */
typedef enum {
    UINT_KERNEL_FAST = 0,  /* packed-half arithmetic: integer -> FP16 by exponent splicing, HSUB2, HMUL2 */
    UINT_KERNEL_NAIVE = 1  /* per-element int -> float convert, subtract, multiply, convert back  */
} uint_kernel_t;

const char* pot_status_string(pot_status_t s);

/* ---- sizes (host arithmetic only; 0 on invalid arguments) ------------------------------- */
size_t pot_packed_bytes(int64_t N, int64_t K, int bits);          /* N * K * bits / 8          */
size_t pot_scales_bytes(int64_t N, int64_t K, int group);         /* N * (K / group) * 2       */
/* Scratch needed by pot_gemv / uint_gemv with the tiled layout (arrival counters of the row
 * blocks + FP32 partial sums); may be 0.  The workspace must be ZERO before its first use; every
 * call leaves its counters at zero again, so consecutive calls of the SAME entry point with the
 * SAME (N, K, bits, group) may reuse one buffer without clearing it.  The position of the
 * counters inside the buffer depends on the shape: a buffer handed to a call with another shape
 * (or to pot_gemm) must be cleared to zero first.  Two calls that may run concurrently
 * (different streams) need different workspaces.                                              */
size_t pot_gemv_workspace_bytes(int64_t N, int64_t K, int bits, int group);
/* Scratch needed by pot_gemm for the given M; may be 0.                                       */
size_t pot_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int bits, int group);

/* Number of kernels this process has launched through the library (diagnostic counter). */
uint64_t pot_launch_count(void);
/* Diagnostics.  Every wait inside the streaming GEMV / small-batch GEMM kernels is bounded; a wait that
 * gives up records a code in a device word instead of hanging the GPU.  These calls synchronise the
 * device, return that word (0 = no wait ever gave up) and clear it.                                   */
int pot_debug_gemv_error(void);
/* Host arithmetic only: the launch plan pot_gemv (uniform = 0) / uint_gemv (uniform = 1) would use for a tiled shape:
 * CTAs per SM (1 or 2), whether CTA ranges end on row-block boundaries (1) or the units are split evenly and partial
 * sums cross CTAs through the workspace (0), slots per warp ring, units per slot (2, 4 or 8), and whether x is staged
 * in shared memory.                                                                                                  */
pot_status_t pot_debug_gemv_plan(int64_t N, int64_t K, int bits, int group, int uniform, int* ctas_per_sm,
                                 int* row_block_split, int* ring_slots, int* units_per_slot, int* x_in_smem);
int pot_debug_gemm_error(void);
int pot_debug_prefill_error(void);

/*
 * pot_quantize_ref -- reference PoT quantizer (Eq. 2; groups per Sec. 3.1).  Set-up code: it
 * makes the inputs of the hot path and is not part of the timed path.
 *   W_f16      [N,K] FP16, finite values.
 *   scales_f16 [N,K/G] FP16: read when rule == POT_SCALE_GIVEN, written otherwise (after
 *              clamping into the legal scale range; an all-zero group gets 2^-14).
 *   packed_out [N, K*bits/8] canonical layout.
 * Per weight: sign = [w < 0] (so -0 -> +), E = clamp(round(log2(|w|/S)), 0, q_max), evaluated
 * exactly (threshold test on w^2 against 2^(2k+1) S^2 in FP64; |w| = 0 gives E = 0).
 */
pot_status_t pot_quantize_ref(const void* W_f16, int64_t N, int64_t K, int bits, int group,
                              pot_scale_rule_t rule, void* scales_f16, void* packed_out, void* stream);

/*
 * pot_validate_scales -- counts scales outside the scale contract: the integer add of Sec. 4.2 equals the
 * multiplication by 2^E of Eq. 1 only for normal FP16 scales whose exponent field e satisfies 1 <= e and
 * e + q_max <= 30 (the paper does not discuss zero, subnormal or overflowing scales).  A caller that gets a non-zero
 * count should treat its scales as POT_ERR_SCALE_RANGE.
 *   d_bad_count: device int32; the kernel ADDS the number of offending entries (zero it first).
 */
pot_status_t pot_validate_scales(const void* scales_f16, int64_t count, int bits, int32_t* d_bad_count,
                                 void* stream);

/*
 * pot_repack -- canonical -> tiled (direction 0) or tiled -> canonical (direction 1).
 * Both buffers hold pot_packed_bytes(N,K,bits) bytes and must not overlap.  N % 16 == 0.
 *
 * Tiled layout: the matrix is cut into units of 16 rows x 128 columns (one unit per row block
 * rb = i/16 and column block cb = k/128, stored in [rb][cb] order, 16*128*n/8 bytes each).
 * A unit holds n "planes" of 256 bytes; plane k stores, for row r of the unit, 16 bytes at
 * offset k*256 + r*16: word k of each of the four 32-column quarters of that row's 128-code
 * record (record word index 4k + quarter).  Inside a word the PoT codes are laid out as byte
 * lanes shaped like an 8-bit float (exponent bits from bit 2, sign at bit 7, after a rotation),
 * so that one rotate + one mask extract four codes and one multiply-add per pair places them
 * in the FP16 exponent / sign fields; the uniform codes are plain n-bit fields with the two
 * codes of a pair 16 bits apart.  csrc/layout.cuh has the bit map; pot_layout_bit reports it.
 */
pot_status_t pot_repack(const void* src, void* dst, int64_t N, int64_t K, int bits, int direction,
                        void* stream);

/*
 * pot_repack_scales -- per-group parameters (the FP16 scales; also the uniform twin's zero-points) between the
 * row-major [N, K/G] interchange layout and the tiled layout that goes with pot_repack (direction 0: row-major ->
 * tiled, 1: back).  Same bytes, same size, N % 16 == 0; the buffers must not overlap.  (The paper fixes no storage
 * order for the scales of Sec. 3.1; this one is the library's.)  The 16 * (128 / G) parameters of one unit are
 * stored together, units in [rb][cb] order like the codes, so a kernel that streams a contiguous range of units
 * fetches their scales with the same kind of contiguous copy; inside a unit the values of rows r and r + 8 of a
 * group share a 32-bit word (halfword index ((s * 8 + r % 8) * 2 + r / 8) for group s of the unit).
 * EVERY entry point that takes `layout == POT_LAYOUT_TILED` expects both the codes (pot_repack / uint_repack) and
 * the per-group parameters (pot_repack_scales) in tiled form.
 */
pot_status_t pot_repack_scales(const void* src, void* dst, int64_t N, int64_t K, int group, int direction,
                               void* stream);
/* Host arithmetic only: halfword index, inside the tiled parameter array, of the value of (row, group g of the row). */
pot_status_t pot_layout_scale_index(int64_t N, int64_t K, int group, int64_t row, int64_t g, int64_t* index);

/* Host arithmetic only: position (32-bit word index inside the 4n-word record, bit index) of
 * bit b of code q (0 <= q < 128) in the tiled layout.  kind 0 = PoT codes, 1 = uniform codes. */
pot_status_t pot_layout_bit(int bits, int kind, int q, int b, int* word, int* bit);

/*
 * pot_dequant -- the paper's dequantization kernel (Sec. 4.2): extract the exponent field with
 * an AND mask, move the sign to bit 15, OR them, align to the FP16 exponent (bit 10; bit 7 for
 * BF16) and integer-add to the scale's bit pattern.  No floating-point instruction touches the
 * weights.  packed is canonical; W_out is [N,K] row-major of out_dtype (2 bytes per element).
 * BF16: the FP16 scale is converted once per group to BF16 (round to nearest even).
 */
pot_status_t pot_dequant(const void* packed, const void* scales_f16, int64_t N, int64_t K, int bits,
                         int group, pot_dtype_t out_dtype, void* W_out, void* stream);

/*
 * pot_gemv -- batch-1 decode: y = W~ x with W~ the FP16 reconstruction (Eq. 1), FP32
 * accumulation, FP16 output.  Codes are decoded in registers with the integer-add trick (Sec.
 * 4.2).  Tiled layout: every warp streams its own contiguous share of the codes and scales
 * through a private shared-memory ring, the decoded FP16 weights are the A fragments of
 * warp-level tensor-core MMAs whose B columns all hold x, and the matrix is split evenly across
 * all warps of the GPU (partial sums of a row block that spans warps are added in a fixed order --
 * in shared memory inside a CTA, through `workspace` across CTAs -- so results are bit-identical
 * run to run).  Canonical layout: a CUDA-core kernel with warp-shuffle reduction.
 *   x_f16 [K], y_f16 [N]; workspace >= pot_gemv_workspace_bytes(N,K,bits,group), 16-byte aligned
 *   (may be NULL when that size is 0).  `layout` says how `packed` is arranged.
 * Ordering on the stream: the fused kernels (pot_gemv, pot_gemm, uint_gemv and their BF16 forms) are launched so that
 * they may START while the previous kernel of the stream is still draining; they fetch codes and scales at once and
 * wait for that kernel to end before they read x or write y and the workspace.  x, y and the workspace may therefore
 * be produced / still be in use by the preceding call; the CODES AND SCALES MUST BE COMPLETE before the preceding
 * kernel of the stream starts.  Every kernel of this library that writes codes or scales (pot_quantize_ref,
 * pot_repack, pot_repack_scales, the uint_ forms) keeps its successors from starting early, so call sequences built
 * from this library are always safe; a caller who writes codes or scales with a kernel of their own that releases its
 * dependents early (programmatic dependent launch) must synchronise before the first GEMV that reads them.
 */
pot_status_t pot_gemv(const void* packed, const void* scales_f16, int64_t N, int64_t K, int bits,
                      int group, pot_layout_t layout, const void* x_f16, void* y_f16,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * pot_gemv_bf16 -- pot_gemv with BF16 activations, BF16 reconstruction and BF16 output.  The paper's kernel (Sec. 4.2)
 * is written for FP16; the same integer add applies to BF16 with the exponent at bit 7: the group's FP16 scale is
 * rounded once to BF16 (round to nearest even) and E is added to that pattern, w~ = +-2^E * bf16(S) exactly, as in
 * pot_dequant with POT_BF16.  x_bf16 [K], y_bf16 [N]; everything else as pot_gemv (same layouts, same workspace).
 * In the tiled layout the codes keep their FP16-shaped bit map, so the BF16 decode needs two mask / multiply-add
 * pairs per register where FP16 needs one: expect a slower kernel at equal bytes.
 */
pot_status_t pot_gemv_bf16(const void* packed, const void* scales_f16, int64_t N, int64_t K, int bits,
                           int group, pot_layout_t layout, const void* x_bf16, void* y_bf16,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * pot_gemv_host -- pot_gemv for a caller whose activations and results live in HOST memory
 * (ideally pinned): copies x_host [K] to d_x, runs pot_gemv, copies the result to y_host [N],
 * all asynchronously on `stream`.  The weights stay resident on the device.
 *   x_host, y_host: HOST pointers.  d_x (>= 2K bytes) and d_y (>= 2N bytes): device staging
 *   buffers owned by the caller.  The caller synchronises the stream before reading y_host.
 */
pot_status_t pot_gemv_host(const void* packed, const void* scales_f16, int64_t N, int64_t K, int bits,
                           int group, pot_layout_t layout, const void* x_host, void* y_host,
                           void* d_x, void* d_y, void* workspace, size_t workspace_bytes, void* stream);

/*
 * pot_gemv_noalloc -- pot_gemv (tiled layout) for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a packaging convenience of this library.)
 * Who needs it: a plug-in inside a host application that owns every byte of device memory and
 * gives the plug-in no allocator -- for example an inference server whose serving loop may
 * never run into the device-wide synchronisation that cudaMalloc / cudaFree imply.  Such a
 * caller has nowhere to get the split-K workspace of pot_gemv from.  Here the workspace is a
 * fixed array of pot_gemv_noalloc_max_scratch_bytes() = 1 MiB that is part of the library image:
 * every GPU that loads the library holds it until the process exits.
 *   - Arguments as for pot_gemv with layout = POT_LAYOUT_TILED; inputs and outputs are still the
 *     caller's device buffers.  The call itself allocates and frees nothing.
 *   - A shape whose workspace (pot_gemv_workspace_bytes) exceeds the array is rejected with
 *     POT_ERR_WORKSPACE before anything is enqueued.
 *   - The first call on each device (with that device current) looks the array's device address
 *     up through the runtime.  Make that first call outside of any stream capture.
 *   - All calls share the one array per GPU and it keeps the last call's contents; each call
 *     clears the part that must start at zero on `stream`.  Calls that may overlap on the same
 *     GPU (different streams) race on it -- serialise them, or use pot_gemv with own workspaces.
 */
size_t pot_gemv_noalloc_max_scratch_bytes(void);
pot_status_t pot_gemv_noalloc(const void* packed_tiled, const void* scales_f16, int64_t N, int64_t K,
                              int bits, int group, const void* x_f16, void* y_f16, void* stream);

/*
 * pot_gemm -- the matrix product that the dequantized weights feed (Sec. 4.2, last paragraph; reconstruction by
 * Eq. 1, decode by the integer add of Sec. 4.2): Y = X W~^T for M tokens: X_f16 [M,K] row-major, Y_f16 [M,N] row-major, FP32
 * accumulation, FP16 output.  M = 1 runs pot_gemv's kernel.  2 <= M <= 8 (decode batches) runs the streaming
 * tensor-core kernel of pot_gemv with one token per MMA column, the weights decoded straight into MMA
 * fragments (5 <= M <= 8 only while 16 K bytes of activations fit in shared memory beside the rings: K <= 8192 or so);
 * larger M runs the tcgen05 kernel: TMA loads of X tiles, weights decoded into swizzled shared-memory tiles,
 * accumulators in tensor memory (two issuing threads with an accumulator each, added in a fixed
 * order: the result does not depend on timing); the tiles of a last, at most half-filled wave
 * of CTAs -- or all tiles when they cover at most half of the SMs -- are split along K (FP32
 * partial sums and arrival counters in `workspace`, added in a fixed order).  The tcgen05
 * kernel requires layout == POT_LAYOUT_TILED.
 *   workspace >= pot_gemm_workspace_bytes(M,N,K,bits,group), 16-byte aligned, zero before its
 *   first use (the kernels leave the counters at zero); may be NULL when that size is 0.
 */
pot_status_t pot_gemm(const void* packed, const void* scales_f16, int64_t N, int64_t K, int bits,
                      int group, pot_layout_t layout, const void* X_f16, int64_t M, void* Y_f16,
                      void* workspace, size_t workspace_bytes, void* stream);

/* pot_gemm_bf16 -- pot_gemm with BF16 activations X_bf16 [M,K], BF16 reconstruction (see pot_gemv_bf16) and BF16
 * output Y_bf16 [M,N]; same routes (streaming kernel, tcgen05 kernel with the BF16 instruction kind, canonical
 * fallback), same workspace sizes.                                                                              */
pot_status_t pot_gemm_bf16(const void* packed, const void* scales_f16, int64_t N, int64_t K, int bits,
                           int group, pot_layout_t layout, const void* X_bf16, int64_t M, void* Y_bf16,
                           void* workspace, size_t workspace_bytes, void* stream);

/* ---- uniform-INT (zero-point) twin at the same bits and group size ------------------------
 * The baseline the paper compares against (first equation of Sec. 4.1): w~ = (W_Q + Z) o S.
 * Here the stored zero-point z is non-negative (Z = -z): codes q in [0, 2^n - 1] in the same
 * canonical bit-stream layout, scales_f16 and zeros_f16 [N,K/G] FP16 (zeros hold the integer z
 * as an FP16 number, so storage is n + 32/G bits per weight).  w~ = fp16((q - z) * s): the
 * integer difference is exact and the product is rounded once.
 */
pot_status_t uint_quantize_ref(const void* W_f16, int64_t N, int64_t K, int bits, int group,
                               void* scales_f16, void* zeros_f16, void* packed_out, void* stream);
pot_status_t uint_dequant(const void* packed, const void* scales_f16, const void* zeros_f16, int64_t N,
                          int64_t K, int bits, int group, uint_kernel_t kernel, void* W_out_f16, void* stream);
pot_status_t uint_gemv(const void* packed, const void* scales_f16, const void* zeros_f16, int64_t N,
                       int64_t K, int bits, int group, pot_layout_t layout, const void* x_f16, void* y_f16,
                       void* workspace, size_t workspace_bytes, void* stream);
/* canonical <-> tiled for uniform codes (same unit/plane structure as pot_repack; the n-bit
 * integer is kept as one field, see csrc/layout.cuh).  direction 0: canonical -> tiled.       */
pot_status_t uint_repack(const void* src, void* dst, int64_t N, int64_t K, int bits, int direction,
                         void* stream);

#ifdef __cplusplus
}
#endif
#endif /* POT_B200_H */
