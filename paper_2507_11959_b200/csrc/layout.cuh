// Bit map of the kernel ("tiled") layout and the register decoders that go with it.
//
// One "record" = the 128 codes of one row inside one 128-column block = 4n 32-bit words.
// The map below says where bit b of code q (0 <= q < 128) lives: (word index, bit position).
//
// PoT codes ("byte-lane" map).  Quarter T = q / 32 of the record owns the n words 4k + T
// (k = 0..n-1; word k of every quarter sits in 16-byte plane k of the row).  A quarter decodes
// into eight "decoded words" i = 0..7 of four byte lanes each; byte lane l of decoded word i is
// column 32T + 4i + perm[l], perm = {0, 2, 1, 3} -- so lanes (0, 2) and (1, 3), which sit 16
// bits apart, are pairs of ADJACENT columns.  Inside a byte lane the code is stored in the shape
// of an 8-bit float with five exponent bits: exponent bits from bit 2 upwards, sign at bit 7
// (five above the exponent's low bit), after a rotation of the word:
//   * as FP8 operand : (rot(w) & mask) | 0x40..  is the byte pattern of +-2^(E+1) -- one
//                      logic operation per four weights.  No kernel in this tree consumes that form: FP8 GEMVs built on
//                      it (warp-level m16n8k32 MMAs, which this GPU emulates with conversions on the ALUs, and
//                      tcgen05 MMAs with the weights in tensor memory) were exact but slower than the FP16 route;
//   * as FP16 pair   : (rot(w) & mask16) * 2^8 + scale  (lanes 0, 2)  and
//                      (rot(w) & mask16 << 8) + scale   (lanes 1, 3)  -- the mask / shift /
//                      integer add into the scale's bit pattern of Sec. 4.2 of the paper.
// A "plane" (word k, anchor a) stores exponent bit e of lane l at bit (8l + a + e) mod 32 and the
// sign at (8l + a + 5) mod 32; rotating the word right by a - 2 brings it into place.
//  PoT n = 2 : words k = 0, 1; anchors 0, 2, 4, 6; decoded word i = 4k + a/2.
//  PoT n = 3 : words k = 0, 1, 2 with anchors {1,3}, {4,6}, {5,7}: decoded word i = 2k + (0|1).
//              Each word keeps two spare bits per byte lane ({5,7}, {0,2}, {1,3}); they hold
//              decoded word 6 = {sign: word 0 bit 7, E0: word 1 bit 2, E1: word 2 bit 3} (all in
//              place) and decoded word 7 = {sign: word 0 bit 5, E0: word 1 bit 0, E1: word 2
//              bit 1} (in place after a shift left by 2).
//  PoT n = 4 : words k = 0..3, decoded word i = 2k + (0|1): plane 0 in place (E at 2,3,4, sign
//              at 7), plane 1 = {E0, E1 at 0, 1; sign at 5} (rotate left 2) + {E2 at 6} (rotate
//              right 2).
// Uniform codes keep the n-bit integer as one field, pairs 16 bits apart:
//  n = 2 at 2p + 16h (p < 8, word q/16), n = 4 at 4p + 16h (p < 4, word q/8), n = 3 as two
//  planes: words 0..7 hold the low two bits as fields 2p + 16h, words 8..11 the high bit at
//  (q%32)/2 + 16h  (pair p = (q % codes-per-word) / 2, half h = q % 2).
#pragma once
#include <cstdint>

namespace potl {

enum Kind { KIND_POT = 0, KIND_UINT = 1 };

struct BitPos {
    int word;
    int bit;
};

// where bit b of code q is stored inside the record (b < n-1: exponent bits, b = n-1: sign, for PoT)
__host__ __device__ inline BitPos record_bit(int bits, int kind, int q, int b) {
    BitPos r;
    if (kind == KIND_POT) {
        const int T = q >> 5, c = q & 31;
        const int i = c >> 2;                                       // decoded word
        const int l = ((c & 1) << 1) | ((c >> 1) & 1);              // byte lane: perm is its own inverse
        const bool sign = (b == bits - 1);
        int k, pos;
        if (bits == 2) {
            k = i >> 2;
            pos = 8 * l + 2 * (i & 3) + (sign ? 5 : 0);
        } else if (bits == 4) {
            k = i >> 1;
            if ((i & 1) == 0) pos = 8 * l + (sign ? 7 : 2 + b);
            else pos = 8 * l + (sign ? 5 : (b == 2 ? 6 : b));
        } else {
            if (i < 6) {
                k = i >> 1;
                const int a = (k == 0 ? 1 : (k == 1 ? 4 : 5)) + 2 * (i & 1);
                pos = 8 * l + a + (sign ? 5 : b);
            } else if (i == 6) {
                k = sign ? 0 : 1 + b;
                pos = 8 * l + (sign ? 7 : 2 + b);
            } else {
                k = sign ? 0 : 1 + b;
                pos = 8 * l + (sign ? 5 : b);
            }
        }
        r.word = 4 * k + T;
        r.bit = pos & 31;
        return r;
    }
    const int h = q & 1;
    if (bits == 2) {
        r.word = q >> 4;
        r.bit = 2 * ((q & 15) >> 1) + 16 * h + b;
    } else if (bits == 3) {
        if (b < 2) {
            r.word = q >> 4;
            r.bit = 2 * ((q & 15) >> 1) + 16 * h + b;
        } else {
            r.word = 8 + (q >> 5);
            r.bit = ((q & 31) >> 1) + 16 * h;
        }
    } else {
        r.word = q >> 3;
        r.bit = 4 * ((q & 7) >> 1) + 16 * h + b;
    }
    return r;
}

// Tiled per-group parameters (scales, and the uniform twin's zero-points): the 16 * (128 / G) values of one unit
// (16 rows x 128 columns) are stored together, units in the same [row block][column block] order as the codes, so a
// kernel that streams a contiguous range of units streams a contiguous range of their scales too.  Inside a unit,
// rows r and r + 8 of one group share a 32-bit word (r in the low half): halfword index ((s * 8 + r % 8) * 2 + r / 8)
// for group s (0 .. 128/G - 1) of row r -- exactly the two rows a lane of the warp-level MMA owns.
__host__ __device__ inline int scale_tile_index(int r, int s) { return (((s << 3) | (r & 7)) << 1) | (r >> 3); }
// halfword index of the value of (row i, group g) in the tiled array
__host__ __device__ inline int64_t scale_tiled_index(int64_t i, int64_t g, int64_t K, int G) {
    const int spg = 128 / G;
    const int64_t ncb = K / 128, cb = g / spg;
    return ((i >> 4) * ncb + cb) * (16 * spg) + scale_tile_index((int)(i & 15), (int)(g - cb * spg));
}

#ifdef __CUDACC__
// ---------------------------------------------------------------------------------------------
// Register decoders for the PoT byte-lane map.
// rotated_words<BITS>(w, d): the quarter's n words -> its eight decoded words, every code rotated
// into place (exponent from bit 2, sign at bit 7 of its byte lane) but NOT yet masked; decoded
// words whose bits wrap nowhere when shifted left are left unrotated, low(i) positions below their place.
// ---------------------------------------------------------------------------------------------
// t * c + s as ONE multiply-add instruction (written in PTX: left to itself the compiler turns the power-of-two
// multiplier into separate shift / logic / add instructions, which costs a third more issue slots in the decode)
__device__ __forceinline__ uint32_t mad(uint32_t t, uint32_t c, uint32_t s) {
    uint32_t d;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(t), "r"(c), "r"(s));
    return d;
}
__device__ __forceinline__ uint32_t rotr(uint32_t v, int s) { return __funnelshift_r(v, v, s); }
__device__ __forceinline__ uint32_t rotl(uint32_t v, int s) { return __funnelshift_l(v, v, s); }
// bitwise select: mask bits from a, the others from b (one LOP3)
__device__ __forceinline__ uint32_t sel(uint32_t a, uint32_t b, uint32_t mask) { return (a & mask) | (b & ~mask); }

template <int BITS>
struct PotLanes;
template <>
struct PotLanes<2> {
    static constexpr uint32_t MASK = 0x84848484u;
    static __host__ __device__ constexpr int low(int i) { return (i & 3) == 0 ? 2 : 0; }
    static __device__ __forceinline__ void rotate(const uint32_t (&w)[2], uint32_t (&d)[8]) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            d[4 * k + 0] = w[k];          // two positions low
            d[4 * k + 1] = w[k];
            d[4 * k + 2] = rotr(w[k], 2);
            d[4 * k + 3] = rotr(w[k], 4);
        }
    }
};
template <>
struct PotLanes<3> {
    static constexpr uint32_t MASK = 0x8C8C8C8Cu;
    static __host__ __device__ constexpr int low(int i) { return i == 0 ? 1 : (i == 7 ? 2 : 0); }
    static __device__ __forceinline__ void rotate(const uint32_t (&w)[3], uint32_t (&d)[8]) {
        d[0] = w[0];                      // one position low
        d[1] = rotr(w[0], 1);
        d[2] = rotr(w[1], 2);
        d[3] = rotr(w[1], 4);
        d[4] = rotr(w[2], 3);
        d[5] = rotr(w[2], 5);
        d[6] = sel(sel(w[0], w[1], 0x80808080u), w[2], 0x84848484u);
        d[7] = sel(sel(w[0], w[1], 0x20202020u), w[2], 0x21212121u);  // two positions low
    }
};
template <>
struct PotLanes<4> {
    static constexpr uint32_t MASK = 0x9C9C9C9Cu;
    static __host__ __device__ constexpr int low(int) { return 0; }
    static __device__ __forceinline__ void rotate(const uint32_t (&w)[4], uint32_t (&d)[8]) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            d[2 * k] = w[k];
            d[2 * k + 1] = sel(rotl(w[k], 2), rotr(w[k], 2), 0x8C8C8C8Cu);
        }
    }
};

// Decode 32 consecutive codes (16 pairs): quarter T (0..3) of a record held in registers
// (rec[STRIDE * k + T] = word k of the quarter; STRIDE = 4 for a whole record).  out[p] = bit pattern of half2{ w~[2p], w~[2p+1] }:
// mask, align with the FP16 exponent / sign (the multiply by a power of two is the shift) and
// integer-add to the scale's bit pattern `sc2` (both halves) -- Sec. 4.2 of the paper.
template <int BITS, int STRIDE = 4>
__device__ __forceinline__ void pot_decode32(const uint32_t* rec, int T, uint32_t sc2, uint32_t (&out)[16]) {
    using L = PotLanes<BITS>;
    constexpr uint32_t MA = L::MASK & 0x00FF00FFu, MB = L::MASK & 0xFF00FF00u;
    uint32_t w[BITS], d[8];
#pragma unroll
    for (int k = 0; k < BITS; ++k) w[k] = rec[STRIDE * k + T];
    L::rotate(w, d);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        // fields that sit low(i) positions below their place: the alignment shift goes into the multiplier
        out[2 * i] = mad(d[i] & (MA >> L::low(i)), 1u << (8 + L::low(i)), sc2);
        out[2 * i + 1] = mad(d[i] & (MB >> L::low(i)), 1u << L::low(i), sc2);
    }
}

// t * c (upper 32 bits of the product) + s as one instruction: a right shift by 32 - log2(c) fused with the add
__device__ __forceinline__ uint32_t madhi(uint32_t t, uint32_t c, uint32_t s) {
    uint32_t d;
    asm("mad.hi.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(t), "r"(c), "r"(s));
    return d;
}

// The same decode for BF16 (1 sign, 8 exponent, 7 mantissa bits): out[p] = bit pattern of bfloat162{ w~[2p], w~[2p+1] }
// with w~ = +-2^E * bf16(S); sc2 holds the BF16-rounded scale in both halves.  The byte lanes were shaped for FP16 (sign
// five positions above the exponent's low bit); in BF16 the exponent's low bit is bit 7 and the sign eight positions
// above it, so exponent and sign are masked and aligned separately: two mask / multiply-add pairs per register instead
// of one (for the upper byte lanes the exponent moves DOWN, which the high half of a multiply-add does).
template <int BITS, int STRIDE = 4>
__device__ __forceinline__ void pot_decode32_bf16(const uint32_t* rec, int T, uint32_t sc2, uint32_t (&out)[16]) {
    using L = PotLanes<BITS>;
    constexpr uint32_t EM = L::MASK & 0x7F7F7F7Fu, SM = L::MASK & 0x80808080u;
    constexpr uint32_t LA = 0x00FF00FFu, LB = 0xFF00FF00u;
    uint32_t w[BITS], d[8];
#pragma unroll
    for (int k = 0; k < BITS; ++k) w[k] = rec[STRIDE * k + T];
    L::rotate(w, d);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int p = L::low(i);
        // lower byte lanes (columns 2p', 2p'+1 of the pair 2i): exponent from bit 2 - p up to bit 7, sign to bit 15
        const uint32_t ea = mad(d[i] & ((EM & LA) >> p), 1u << (5 + p), sc2);
        out[2 * i] = mad(d[i] & ((SM & LA) >> p), 1u << (8 + p), ea);
        // upper byte lanes: exponent from bit 10 - p down to bit 7, sign from bit 15 - p up to bit 15
        const uint32_t eb = madhi(d[i] & ((EM & LB) >> p), 1u << (29 + p), sc2);
        out[2 * i + 1] = p == 0 ? (eb | (d[i] & (SM & LB))) : mad(d[i] & ((SM & LB) >> p), 1u << p, eb);
    }
}

// ---------------------------------------------------------------------------------------------
// Uniform-INT twin on the same tiled layout: w~ = (q - z) * s with q spliced under the exponent
// of 1024 (0x6400 | q = 1024 + q as FP16), an exact subtraction, and one rounding multiply.
// zm2 = half2(1024 + z), s2 = half2(s).  A field that sits at mantissa bit b > 0 gives
// 1024 + q * 2^b; the fused multiply-add (h * 2^-b - (1024 * 2^-b + z)) is still exact.
// ---------------------------------------------------------------------------------------------
struct UintParams {
    __half2 s2;    // scale
    __half2 z;     // zero-point z (an integer 0..2^n-1)
};

__device__ __forceinline__ uint32_t h2_bits(__half2 v) { return *reinterpret_cast<uint32_t*>(&v); }
__device__ __forceinline__ __half2 bits_h2(uint32_t v) { return *reinterpret_cast<__half2*>(&v); }

// field of width W at mantissa bit b (b + W <= 10) of both halves -> half2(q - z)
template <int B>
__device__ __forceinline__ __half2 uint_field(uint32_t masked, __half2 z) {
    const __half2 h = bits_h2(masked | 0x64006400u);
    if (B == 0) return __hsub2(h, __hadd2(z, __float2half2_rn(1024.0f)));
    const float inv = 1.0f / (float)(1 << B);
    return __hfma2(h, __float2half2_rn(inv), __hneg2(__hadd2(z, __float2half2_rn(1024.0f * inv))));
}

template <int BITS>
__device__ __forceinline__ void uint_decode_pairs16(const uint32_t* rec, int blk, const UintParams& pr, uint32_t (&out)[8]);

template <>
__device__ __forceinline__ void uint_decode_pairs16<2>(const uint32_t* rec, int blk, const UintParams& pr, uint32_t (&out)[8]) {
    const uint32_t w = rec[blk];
    const uint32_t u = w >> 10;
    __half2 d[8];
    d[0] = uint_field<0>(w & 0x00030003u, pr.z);
    d[1] = uint_field<2>(w & 0x000C000Cu, pr.z);
    d[2] = uint_field<4>(w & 0x00300030u, pr.z);
    d[3] = uint_field<6>(w & 0x00C000C0u, pr.z);
    d[4] = uint_field<8>(w & 0x03000300u, pr.z);
    d[5] = uint_field<0>(u & 0x00030003u, pr.z);
    d[6] = uint_field<2>(u & 0x000C000Cu, pr.z);
    d[7] = uint_field<4>(u & 0x00300030u, pr.z);
#pragma unroll
    for (int p = 0; p < 8; ++p) out[p] = h2_bits(__hmul2(d[p], pr.s2));
}

template <>
__device__ __forceinline__ void uint_decode_pairs16<4>(const uint32_t* rec, int blk, const UintParams& pr, uint32_t (&out)[8]) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const uint32_t w = rec[2 * blk + i];
        const uint32_t u = w >> 8;
        out[4 * i + 0] = h2_bits(__hmul2(uint_field<0>(w & 0x000F000Fu, pr.z), pr.s2));
        out[4 * i + 1] = h2_bits(__hmul2(uint_field<4>(w & 0x00F000F0u, pr.z), pr.s2));
        out[4 * i + 2] = h2_bits(__hmul2(uint_field<0>(u & 0x000F000Fu, pr.z), pr.s2));
        out[4 * i + 3] = h2_bits(__hmul2(uint_field<4>(u & 0x00F000F0u, pr.z), pr.s2));
    }
}

// n = 3: low two bits from the field plane, high bit from the bit plane, merged with one multiply-add
template <>
__device__ __forceinline__ void uint_decode_pairs16<3>(const uint32_t* rec, int blk, const UintParams& pr, uint32_t (&out)[8]) {
    const uint32_t we = rec[blk];
    const uint32_t ws = rec[8 + (blk >> 1)] >> (8 * (blk & 1));
    const __half2 zm = __hadd2(pr.z, __float2half2_rn(1024.0f));
#pragma unroll
    for (int p = 0; p < 8; ++p) {
        const uint32_t lo = ((we >> (2 * p)) & 0x00030003u) | 0x64006400u;
        const uint32_t hb = (ws >> p) & 0x00010001u;
        const uint32_t h = hb * 4u + lo;  // 1024 + q
        out[p] = h2_bits(__hmul2(__hsub2(bits_h2(h), zm), pr.s2));
    }
}

template <int BITS>
__device__ __forceinline__ void uint_decode32(const uint32_t* rec, int T, const UintParams& pr, uint32_t (&out)[16]) {
    uint32_t a[8], b[8];
    uint_decode_pairs16<BITS>(rec, 2 * T, pr, a);
    uint_decode_pairs16<BITS>(rec, 2 * T + 1, pr, b);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        out[i] = a[i];
        out[8 + i] = b[i];
    }
}
#endif  // __CUDACC__

}  // namespace potl
