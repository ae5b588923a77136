// Bit map of the kernel ("tiled") layout and the register decoders that go with it.
//
// One "record" = the 128 codes of one row inside one 128-column block = 4n 32-bit words.
// The map below says where bit b of code q (0 <= q < 128) lives: (word index, bit position).
// Codes 2P and 2P+1 ("pair" P) always sit 16 bits apart in one word, so that one AND mask
// and one multiply-add (shift left + add the scale's bit pattern, Sec. 4.2 of the paper)
// produce both halves of a half2.  The PoT maps additionally put the sign bit where the same
// shift moves it to bit 15 (n = 2), or in a position of its own (n = 3, 4).
//
//  PoT n = 2 : word w = q/16 holds codes 16w..16w+15; pair p = (q%16)/2, half h = q%2.
//              The word is a ring of 32 positions; a code anchored at even position a has
//              its exponent bit at a and its sign at a+5 (mod 32):
//                p <= 5 : anchor 2p + 16h           (decoded straight from the word)
//                p == 6 : anchor 28 (h=0), 12 (h=1) (decoded after rotating the word left by 8)
//                p == 7 : anchor 30 (h=0), 14 (h=1)
//  PoT n = 3 : the record is four "triples" of three words; triple T = q/32 holds pairs
//              P = (q%32)/2 = 0..15.  Pair P < 15 lives in word 3T + P/5 as slot d = P%5:
//                d < 4 : exponent at bits 3d, 3d+1 and sign at 3d+5 (+16h) -- the sign sits five
//                        positions above the exponent's low bit, so ONE mask and ONE shift-add
//                        place both (these are 12 of every 16 pairs);
//                d = 4 : exponent at bits 12,13 and sign already at bit 15 (+16h);
//              pair 15 is spread over bit 2 (+16h) of the three words: exponent bit 0 in word
//              3T, exponent bit 1 in word 3T+1, sign in word 3T+2.
//              (The uniform twin keeps the plain plane map: words 0..7 hold the low two bits as
//              fields 2p + 16h, words 8..11 the high bit at (q%32)/2 + 16h.)
//  PoT n = 4 : word w = q/8 holds codes 8w..8w+7; pair p = (q%8)/2; exponent at bits
//              3p + 16h + {0,1,2}, sign at bit 12 + p + 16h.
//  uniform   : the n-bit integer code as a field: n = 2 at 2p + 16h (p < 8), n = 4 at
//              4p + 16h (p < 4), n = 3 as for PoT n = 3 (low two bits / high bit planes).
#pragma once
#include <cstdint>

namespace potl {

enum Kind { KIND_POT = 0, KIND_UINT = 1 };

struct BitPos {
    int word;
    int bit;
};

// where bit b of code q is stored inside the record
__host__ __device__ inline BitPos record_bit(int bits, int kind, int q, int b) {
    BitPos r;
    const int h = q & 1;
    if (bits == 2) {
        r.word = q >> 4;
        const int p = (q & 15) >> 1;
        if (kind == KIND_UINT) {
            r.bit = 2 * p + 16 * h + b;
        } else {
            int anchor;
            if (p <= 5) anchor = 2 * p + 16 * h;
            else if (p == 6) anchor = h ? 12 : 28;
            else anchor = h ? 14 : 30;
            r.bit = (b == 0) ? anchor : ((anchor + 5) & 31);
        }
    } else if (bits == 3 && kind == KIND_UINT) {
        if (b < 2) {
            r.word = q >> 4;
            r.bit = 2 * ((q & 15) >> 1) + 16 * h + b;
        } else {
            r.word = 8 + (q >> 5);
            r.bit = ((q & 31) >> 1) + 16 * h;
        }
    } else if (bits == 3) {
        const int T = q >> 5, P = (q & 31) >> 1;
        if (P < 15) {
            const int d = P % 5;
            r.word = 3 * T + P / 5;
            if (d < 4) r.bit = 3 * d + 16 * h + (b < 2 ? b : 5);
            else r.bit = 16 * h + (b < 2 ? 12 + b : 15);
        } else {
            r.word = 3 * T + b;
            r.bit = 2 + 16 * h;
        }
    } else {
        r.word = q >> 3;
        const int p = (q & 7) >> 1;
        if (kind == KIND_UINT) r.bit = 4 * p + 16 * h + b;
        else r.bit = (b < 3) ? (3 * p + 16 * h + b) : (12 + p + 16 * h);
    }
    return r;
}

#ifdef __CUDACC__
// ---------------------------------------------------------------------------------------------
// Register decoders.  `sc2` is the group scale's FP16 bit pattern replicated in both halves.
// Each returns the bit pattern of half2{ w~[2P], w~[2P+1] } for pair P of the record.
// mad(t, c, s) = t * c + s is one IMAD: the multiply by a power of two is the shift that aligns
// the exponent with FP16 bit 10 and the sign with bit 15, the add is the "fixed-point integer
// addition" into the scale (Sec. 4.2).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t mad(uint32_t t, uint32_t c, uint32_t s) { return t * c + s; }
__device__ __forceinline__ uint32_t rotl(uint32_t v, int s) { return __funnelshift_l(v, v, s); }

template <int BITS>
struct PotDecoder;

// n = 2 : 16 codes (8 pairs) per word, 2 operations per pair + one rotate per word.
template <>
struct PotDecoder<2> {
    static constexpr int WORDS = 8;
    static constexpr int PAIRS_PER_WORD = 8;
    // out[8]: pairs 8w .. 8w+7
    static __device__ __forceinline__ void word(uint32_t w, uint32_t sc2, uint32_t (&out)[8]) {
#pragma unroll
        for (int p = 0; p < 6; ++p) out[p] = mad(w & (0x00210021u << (2 * p)), 1u << (10 - 2 * p), sc2);
        const uint32_t r = rotl(w, 8);
        out[6] = mad(r & 0x02100210u, 64u, sc2);
        out[7] = mad(r & 0x08400840u, 16u, sc2);
    }
};

// n = 4 : 8 codes (4 pairs) per word; exponent and sign are placed by two multiply-adds.
template <>
struct PotDecoder<4> {
    static constexpr int WORDS = 16;
    static constexpr int PAIRS_PER_WORD = 4;
    static __device__ __forceinline__ void word(uint32_t w, uint32_t sc2, uint32_t (&out)[4]) {
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const uint32_t e = mad(w & (0x00070007u << (3 * p)), 1u << (10 - 3 * p), sc2);
            if (p == 3) out[p] = e | (w & 0x80008000u);
            else out[p] = mad(w & (0x10001000u << p), 1u << (3 - p), e);
        }
    }
};

// n = 3 : three words hold 16 pairs (see the map at the top of this file).
template <>
struct PotDecoder<3> {
    static constexpr int WORDS = 12;
    // out[16]: pairs 16T .. 16T+15 of the record, from words w0, w1, w2 of triple T
    static __device__ __forceinline__ void triple(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t sc2,
                                                  uint32_t (&out)[16]) {
        const uint32_t w[3] = {w0, w1, w2};
#pragma unroll
        for (int j = 0; j < 3; ++j) {
#pragma unroll
            for (int d = 0; d < 4; ++d) out[5 * j + d] = mad(w[j] & (0x00230023u << (3 * d)), 1u << (10 - 3 * d), sc2);
            // slot 4: exponent at bits 12,13 (two positions too high), sign in place at bit 15
            const uint32_t e = (__funnelshift_r(w[j], w[j], 2) & 0x0C000C00u) + sc2;
            out[5 * j + 4] = e | (w[j] & 0x80008000u);
        }
        uint32_t y = mad(w0 & 0x00040004u, 1u << 8, sc2);
        y = mad(w1 & 0x00040004u, 1u << 9, y);
        out[15] = mad(w2 & 0x00040004u, 1u << 13, y);
    }
};

// Decode 32 consecutive codes (16 pairs): quarter T (0..3) of a record held in registers.
template <int BITS>
__device__ __forceinline__ void pot_decode32(const uint32_t* rec, int T, uint32_t sc2, uint32_t (&out)[16]);

template <>
__device__ __forceinline__ void pot_decode32<2>(const uint32_t* rec, int T, uint32_t sc2, uint32_t (&out)[16]) {
    uint32_t a[8], b[8];
    PotDecoder<2>::word(rec[2 * T], sc2, a);
    PotDecoder<2>::word(rec[2 * T + 1], sc2, b);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        out[i] = a[i];
        out[8 + i] = b[i];
    }
}
template <>
__device__ __forceinline__ void pot_decode32<3>(const uint32_t* rec, int T, uint32_t sc2, uint32_t (&out)[16]) {
    PotDecoder<3>::triple(rec[3 * T], rec[3 * T + 1], rec[3 * T + 2], sc2, out);
}
template <>
__device__ __forceinline__ void pot_decode32<4>(const uint32_t* rec, int T, uint32_t sc2, uint32_t (&out)[16]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t a[4];
        PotDecoder<4>::word(rec[4 * T + i], sc2, a);
#pragma unroll
        for (int k = 0; k < 4; ++k) out[4 * i + k] = a[k];
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
