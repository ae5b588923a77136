/*
 * pot_oracle.c -- plain CPU oracle for the PoT-PTQ inference path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the GPU library must compute.  It shares no code, header, table or constant
 * with the CUDA sources and is never called from the product path: only the test
 * suite, the smoke check and the bench's CPU-baseline / reference legs load it.
 *
 * Everything is evaluated in FP64 (or exact integers) straight from the paper's
 * definitions; there is no blocking, fusion or bit trickery here:
 *
 *   - PoT format and reconstruction          : Eq. 1  (w~ = S * P * 2^E), Sec. 3.1
 *   - round-to-nearest PoT quantizer         : Eq. 2  (E = clamp(round(log2(|W|/S)), 0, q_max))
 *   - group-wise scales along the reduction  : group constraint of Sec. 3.1
 *   - base scale s0 and the multiplier grid  : Algorithm 1 (Step 1)
 *   - uniform (zero-point) baseline          : first equation of Sec. 4.1, w~ = (W_Q + Z) o S
 *   - FP16 field layout                      : Sec. 4.1 (1 sign, 5 exponent, 10 mantissa bits)
 *
 * The paper is silent on how n-bit codes are packed into bytes; the interchange
 * layout used here is: a code is  sign << (n-1) | E  (the paper's "S0 E1 E2" for n = 3),
 * row i is a little-endian bit stream, code k sits at bits [n*k, n*k+n) of the row.
 *
 * Parity status: every function below is pinned by the CPU test-suite (exact rational
 * arithmetic, numpy's independent half conversion, numpy matmul, hand-derived fixtures,
 * invariants, and the integer-add formulation of Sec. 4.2 as an independent route).
 * po_scale_search (Algorithm 1) is pinned by brute force and by its optimality invariant.
 * po_matmul_bf16 (the contraction on the BF16 reconstruction, BF16 activations) is pinned by numpy
 * on float32-view conversions and a closed form.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define PO_RULE_TOP 0      /* S = max|w| * 2^-q_max : top level sits exactly on max|w|          */
#define PO_RULE_PAPER_S0 1 /* S = max|w| / (2^q_max - 1) : Algorithm 1's s0 taken literally      */
#define PO_RULE_GIVEN 2    /* S supplied by the caller                                           */

#define PO_F16 0
#define PO_BF16 1

int po_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------- number formats */

/* FP16 -> FP64, exact.  Sec. 4.1: x = (-1)^S * 2^(E-15) * 1.M ; E = 0 is the subnormal range. */
double po_f16_to_f64(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int m = h & 0x3FF;
    double v;
    if (e == 0x1F) v = m ? NAN : INFINITY;
    else if (e == 0) v = ldexp((double)m, -24);
    else v = ldexp((double)(1024 + m), e - 25);
    return sign ? -v : v;
}

/* FP64 -> FP16, round to nearest even.  *inexact (optional) is set when rounding happened. */
uint16_t po_f64_to_f16(double v, int* inexact) {
    uint16_t sign = signbit(v) ? 0x8000 : 0;
    double a = fabs(v);
    if (inexact) *inexact = 0;
    if (isnan(v)) return 0x7E00;
    if (isinf(v)) return sign | 0x7C00;
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);          /* a = f * 2^e, f in [0.5, 1)  ->  a in [2^(e-1), 2^e) */
    int ue = e - 1;              /* unbiased exponent of the leading bit */
    if (ue < -14) ue = -14;      /* subnormal range shares the exponent of the smallest normal */
    double scaled = ldexp(a, 10 - ue);   /* units of the last mantissa place; exact */
    double r = nearbyint(scaled);        /* default rounding mode = ties to even */
    if (inexact && r != scaled) *inexact = 1;
    long q = (long)r;                    /* in [0, 2048] */
    long bits;
    if (q < 1024) bits = q;                                  /* subnormal (or zero after rounding) */
    else bits = ((long)(ue + 15) << 10) + (q - 1024);        /* q == 2048 carries into the exponent */
    if (bits >= 0x7C00) { if (inexact) *inexact = 1; bits = 0x7C00; }
    return sign | (uint16_t)bits;
}

/* BF16 (1 sign, 8 exponent with bias 127, 7 mantissa) -> FP64, exact. */
double po_bf16_to_f64(uint16_t b) {
    int sign = (b >> 15) & 1;
    int e = (b >> 7) & 0xFF;
    int m = b & 0x7F;
    double v;
    if (e == 0xFF) v = m ? NAN : INFINITY;
    else if (e == 0) v = ldexp((double)m, -133);
    else v = ldexp((double)(128 + m), e - 134);
    return sign ? -v : v;
}

/* FP64 -> BF16, round to nearest even. */
uint16_t po_f64_to_bf16(double v, int* inexact) {
    uint16_t sign = signbit(v) ? 0x8000 : 0;
    double a = fabs(v);
    if (inexact) *inexact = 0;
    if (isnan(v)) return 0x7FC0;
    if (isinf(v)) return sign | 0x7F80;
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);
    int ue = e - 1;
    if (ue < -126) ue = -126;
    double scaled = ldexp(a, 7 - ue);
    double r = nearbyint(scaled);
    if (inexact && r != scaled) *inexact = 1;
    long q = (long)r;                    /* in [0, 256] */
    long bits;
    if (q < 128) bits = q;
    else bits = ((long)(ue + 127) << 7) + (q - 128);
    if (bits >= 0x7F80) { if (inexact) *inexact = 1; bits = 0x7F80; }
    return sign | (uint16_t)bits;
}

static int po_qmax(int bits) { return (1 << (bits - 1)) - 1; }

static int po_args_ok(int64_t N, int64_t K, int bits, int G) {
    return N >= 0 && K >= 0 && bits >= 2 && bits <= 4 && G > 0 && (K % G) == 0 && ((K * bits) % 8) == 0;
}

/* Legal scale range: a normal FP16 number whose exponent field e satisfies 1 <= e and
 * e + q_max <= 30, so that S * 2^q_max is still a finite normal FP16 number. */
uint16_t po_clamp_scale_bits(uint16_t sbits, int bits) {
    uint16_t lo = 0x0400;
    uint16_t hi = (uint16_t)(((30 - po_qmax(bits)) << 10) | 0x3FF);
    if (sbits < lo) return lo;
    if (sbits > hi) return hi;
    return sbits;
}

int po_scale_in_range(uint16_t sbits, int bits) {
    return sbits == po_clamp_scale_bits(sbits, bits);
}

/* ---------------------------------------------------------------- Eq. 2: the quantizer */

/* One exponent, literally Eq. 2 in FP64.  |w| = 0 gives log2(0) = -inf, which clamps to 0.
 * An exact tie (|w|/S = 2^(k+1/2)) cannot occur for binary floating-point w and S, so the
 * rounding rule of round() never matters; rint is used. */
static int po_exponent(double w, double S, int qmax) {
    double t = rint(log2(fabs(w) / S));
    if (t < 0.0) t = 0.0;
    if (t > (double)qmax) t = (double)qmax;
    return (int)t;
}

/*
 * Quantize W [N,K] (FP16 bit patterns, row-major, groups of G along K).
 *   rule TOP / PAPER_S0 : scales are computed and written to S [N, K/G] (FP16 bits),
 *                         then clamped into the legal range (an all-zero group gets 2^-14);
 *   rule GIVEN          : S is read as supplied (the caller guarantees the legal range).
 * codes [N,K]: one code per byte, sign << (bits-1) | E, sign = 1 iff w < 0 (so +-0 -> +).
 * Returns 0, -1 for bad arguments, -2 if W holds a NaN/Inf, -3 if a GIVEN scale is illegal.
 */
int po_quantize(const uint16_t* W, int64_t N, int64_t K, int bits, int G, int rule,
                uint16_t* S, uint8_t* codes) {
    if (!po_args_ok(N, K, bits, G) || rule < 0 || rule > 2) return -1;
    const int qmax = po_qmax(bits);
    const int64_t ng = K / G;
    int status = 0;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        for (int64_t g = 0; g < ng; ++g) {
            const uint16_t* wg = W + i * K + g * G;
            double amax = 0.0;
            int bad = 0;
            for (int k = 0; k < G; ++k) {
                double w = po_f16_to_f64(wg[k]);
                if (!isfinite(w)) bad = 1;
                if (fabs(w) > amax) amax = fabs(w);
            }
            if (bad) {
#pragma omp atomic write
                status = -2;
                continue;
            }
            uint16_t sb;
            if (rule == PO_RULE_GIVEN) {
                sb = S[i * ng + g];
                if (!po_scale_in_range(sb, bits)) {
#pragma omp atomic write
                    status = -3;
                    continue;
                }
            } else {
                double s = (rule == PO_RULE_TOP) ? ldexp(amax, -qmax)
                                                 : amax / (double)((1 << qmax) - 1);
                sb = po_clamp_scale_bits(po_f64_to_f16(s, NULL), bits);
                S[i * ng + g] = sb;
            }
            const double Sd = po_f16_to_f64(sb);
            for (int k = 0; k < G; ++k) {
                double w = po_f16_to_f64(wg[k]);
                int sign = (w < 0.0) ? 1 : 0;
                int E = po_exponent(w, Sd, qmax);
                codes[i * K + g * G + k] = (uint8_t)((sign << (bits - 1)) | E);
            }
        }
    }
    return status;
}

/* ---------------------------------------------------------------- packing */

void po_pack(const uint8_t* codes, int64_t N, int64_t K, int bits, uint8_t* packed) {
    const int64_t row_bytes = K * bits / 8;
    memset(packed, 0, (size_t)(N * row_bytes));
    for (int64_t i = 0; i < N; ++i) {
        uint8_t* row = packed + i * row_bytes;
        for (int64_t k = 0; k < K; ++k) {
            unsigned c = codes[i * K + k];
            for (int b = 0; b < bits; ++b) {
                int64_t pos = k * bits + b;
                if ((c >> b) & 1u) row[pos >> 3] |= (uint8_t)(1u << (pos & 7));
            }
        }
    }
}

static unsigned po_code_at(const uint8_t* row, int64_t k, int bits) {
    unsigned c = 0;
    for (int b = 0; b < bits; ++b) {
        int64_t pos = k * bits + b;
        c |= (unsigned)((row[pos >> 3] >> (pos & 7)) & 1u) << b;
    }
    return c;
}

void po_unpack(const uint8_t* packed, int64_t N, int64_t K, int bits, uint8_t* codes) {
    const int64_t row_bytes = K * bits / 8;
    for (int64_t i = 0; i < N; ++i)
        for (int64_t k = 0; k < K; ++k)
            codes[i * K + k] = (uint8_t)po_code_at(packed + i * row_bytes, k, bits);
}

/* ---------------------------------------------------------------- Eq. 1: dequantization */

/* One reconstructed weight in FP64: (-1)^sign * 2^E * S  (Eq. 1).
 * For BF16 output the group scale is first rounded to BF16 (the paper is FP16-only; this is
 * the reading taken for BF16: one rounding of the scale, then exact power-of-two scaling). */
static double po_value(unsigned code, uint16_t sbits, int bits, int dtype) {
    int sign = (code >> (bits - 1)) & 1;
    int E = (int)(code & (unsigned)po_qmax(bits));
    double S = po_f16_to_f64(sbits);
    if (dtype == PO_BF16) S = po_bf16_to_f64(po_f64_to_bf16(S, NULL));
    double v = S * ldexp(1.0, E);
    return sign ? -v : v;
}

/*
 * packed [N, K*bits/8], S [N, K/G] -> out [N,K] bit patterns of FP16 (dtype 0) or BF16 (dtype 1).
 * Returns the number of outputs whose conversion to the 16-bit type had to round
 * (0 whenever the scales are in the legal range), or -1 for bad arguments.
 */
int64_t po_dequant(const uint8_t* packed, const uint16_t* S, int64_t N, int64_t K, int bits, int G,
                   int dtype, uint16_t* out) {
    if (!po_args_ok(N, K, bits, G) || dtype < 0 || dtype > 1) return -1;
    const int64_t row_bytes = K * bits / 8, ng = K / G;
    int64_t rounded = 0;
#pragma omp parallel for schedule(static) reduction(+ : rounded)
    for (int64_t i = 0; i < N; ++i) {
        const uint8_t* row = packed + i * row_bytes;
        for (int64_t k = 0; k < K; ++k) {
            double v = po_value(po_code_at(row, k, bits), S[i * ng + k / G], bits, dtype);
            int inexact;
            out[i * K + k] = (dtype == PO_F16) ? po_f64_to_f16(v, &inexact) : po_f64_to_bf16(v, &inexact);
            rounded += inexact;
        }
    }
    return rounded;
}

/* ---------------------------------------------------------------- the contraction */

/*
 * Y[m, r] = sum_k w~[rows[r], k] * x[m, k]   and   A[m, r] = sum_k |w~ * x|   in FP64,
 * with w~ the FP16 reconstruction of Eq. 1 (dtype F16) taken to FP64 exactly.
 * rows == NULL means all N rows (n_rows must equal N).  X is [M,K] FP16 bits, Y and A are
 * [M, n_rows] row-major doubles.  Sum order: k ascending, one accumulator.
 */
int po_matmul(const uint8_t* packed, const uint16_t* S, int64_t N, int64_t K, int bits, int G,
              const uint16_t* X, int64_t M, const int64_t* rows, int64_t n_rows,
              double* Y, double* A) {
    if (!po_args_ok(N, K, bits, G) || M < 0 || n_rows < 0) return -1;
    if (!rows && n_rows != N) return -1;
    const int64_t row_bytes = K * bits / 8, ng = K / G;
    int status = 0;
#pragma omp parallel
    {
        double* wrow = (double*)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_rows; ++r) {
            int64_t i = rows ? rows[r] : r;
            if (i < 0 || i >= N || !wrow) {
#pragma omp atomic write
                status = -1;
                continue;
            }
            const uint8_t* row = packed + i * row_bytes;
            for (int64_t k = 0; k < K; ++k) {
                double v = po_value(po_code_at(row, k, bits), S[i * ng + k / G], bits, PO_F16);
                wrow[k] = po_f16_to_f64(po_f64_to_f16(v, NULL));
            }
            for (int64_t m = 0; m < M; ++m) {
                double y = 0.0, a = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    double p = wrow[k] * po_f16_to_f64(X[m * K + k]);
                    y += p;
                    a += fabs(p);
                }
                Y[m * n_rows + r] = y;
                A[m * n_rows + r] = a;
            }
        }
        free(wrow);
    }
    return status;
}

/*
 * The same contraction on the BF16 reconstruction with BF16 activations: w~ = (-1)^sign 2^E bf16_rne(S) (the paper's
 * Sec. 4.2 is FP16-only; BF16 is this build's extension of the same integer add at exponent bit 7, with the scale
 * rounded once to BF16), x[m,k] BF16 bit patterns, FP64 sums in the order k ascending.
 */
int po_matmul_bf16(const uint8_t* packed, const uint16_t* S, int64_t N, int64_t K, int bits, int G,
                   const uint16_t* X, int64_t M, const int64_t* rows, int64_t n_rows,
                   double* Y, double* A) {
    if (!po_args_ok(N, K, bits, G) || M < 0 || n_rows < 0) return -1;
    if (!rows && n_rows != N) return -1;
    const int64_t row_bytes = K * bits / 8, ng = K / G;
    int status = 0;
#pragma omp parallel
    {
        double* wrow = (double*)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_rows; ++r) {
            int64_t i = rows ? rows[r] : r;
            if (i < 0 || i >= N || !wrow) {
#pragma omp atomic write
                status = -1;
                continue;
            }
            const uint8_t* row = packed + i * row_bytes;
            for (int64_t k = 0; k < K; ++k) {
                double v = po_value(po_code_at(row, k, bits), S[i * ng + k / G], bits, PO_BF16);
                wrow[k] = po_bf16_to_f64(po_f64_to_bf16(v, NULL));
            }
            for (int64_t m = 0; m < M; ++m) {
                double y = 0.0, a = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    double p = wrow[k] * po_bf16_to_f64(X[m * K + k]);
                    y += p;
                    a += fabs(p);
                }
                Y[m * n_rows + r] = y;
                A[m * n_rows + r] = a;
            }
        }
        free(wrow);
    }
    return status;
}

/* ---------------------------------------------------------------- Algorithm 1 (Step 1) */

/*
 * Data-agnostic scale initialisation, one group at a time, exactly in the order of
 * Algorithm 1: s0 = max|w| / (2^q_max - 1); candidates b = 0.01*i, i = 1..200;
 * E(b) by Eq. 2 with scale s0*b; Q1(b) = || w - s0*b*sign(w)*2^E(b) ||^2; strict '<' keeps
 * the first (smallest) minimiser.  All arithmetic in FP64 on the real-valued candidate
 * scale (the paper's S is real during calibration); the winner s* = s0*b* is rounded to
 * FP16 and clamped into the legal range only when stored.
 * S [N, K/G] receives the FP16 scales; bstar (optional) [N, K/G] receives the index i of b*.
 * An all-zero group has s0 = 0: every candidate gives Q1 = 0 and i = 1 is kept; the stored
 * scale is the clamped minimum 2^-14.
 */
int po_scale_search(const uint16_t* W, int64_t N, int64_t K, int bits, int G,
                    uint16_t* S, int32_t* bstar) {
    if (!po_args_ok(N, K, bits, G)) return -1;
    const int qmax = po_qmax(bits);
    const int64_t ng = K / G;
#pragma omp parallel for schedule(static)
    for (int64_t gi = 0; gi < N * ng; ++gi) {
        const uint16_t* wg = W + gi * G;
        double amax = 0.0;
        for (int k = 0; k < G; ++k) {
            double w = fabs(po_f16_to_f64(wg[k]));
            if (w > amax) amax = w;
        }
        const double s0 = amax / (double)((1 << qmax) - 1);
        double qmin = INFINITY;
        int best = 1;
        for (int i = 1; i <= 200; ++i) {
            const double b = 0.01 * (double)i;
            const double sb = s0 * b;
            double q1 = 0.0;
            for (int k = 0; k < G; ++k) {
                double w = po_f16_to_f64(wg[k]);
                double rec;
                if (sb > 0.0) {
                    int E = po_exponent(w, sb, qmax);
                    rec = sb * ldexp(1.0, E);
                    if (w < 0.0) rec = -rec;
                } else {
                    rec = 0.0;
                }
                q1 += (w - rec) * (w - rec);
            }
            if (q1 < qmin) { qmin = q1; best = i; }
        }
        S[gi] = po_clamp_scale_bits(po_f64_to_f16(s0 * (0.01 * (double)best), NULL), bits);
        if (bstar) bstar[gi] = best;
    }
    return 0;
}

/* ---------------------------------------------------------------- uniform (zero-point) twin */

/*
 * Asymmetric uniform quantizer at the same bits and group size (the baseline of Sec. 4.1):
 *   s = fp16((max - min) / (2^n - 1)), raised to at least 2^-14;
 *   z = clamp(rint(-min / s), 0, 2^n - 1);     q = clamp(rint(w / s) + z, 0, 2^n - 1).
 * The paper writes w~ = (W_Q + Z) o S; with the non-negative zero-point stored here, Z = -z.
 * S and Z are [N, K/G] FP16 bit patterns (Z holds the integer z as an FP16 number, so the
 * storage is n + 32/G bits per weight); codes [N,K] hold q, one per byte.
 */
int pu_quantize(const uint16_t* W, int64_t N, int64_t K, int bits, int G,
                uint16_t* S, uint16_t* Z, uint8_t* codes) {
    if (!po_args_ok(N, K, bits, G)) return -1;
    const int64_t ng = K / G;
    const double levels = (double)((1 << bits) - 1);
    int status = 0;
#pragma omp parallel for schedule(static)
    for (int64_t gi = 0; gi < N * ng; ++gi) {
        const uint16_t* wg = W + gi * G;
        double mn = INFINITY, mx = -INFINITY;
        int bad = 0;
        for (int k = 0; k < G; ++k) {
            double w = po_f16_to_f64(wg[k]);
            if (!isfinite(w)) bad = 1;
            if (w < mn) mn = w;
            if (w > mx) mx = w;
        }
        if (bad) {
#pragma omp atomic write
            status = -2;
            continue;
        }
        uint16_t sb = po_f64_to_f16((mx - mn) / levels, NULL);
        if (sb < 0x0400) sb = 0x0400;
        const double s = po_f16_to_f64(sb);
        double z = rint(-mn / s);
        if (z < 0.0) z = 0.0;
        if (z > levels) z = levels;
        S[gi] = sb;
        Z[gi] = po_f64_to_f16(z, NULL);
        for (int k = 0; k < G; ++k) {
            double q = rint(po_f16_to_f64(wg[k]) / s) + z;
            if (q < 0.0) q = 0.0;
            if (q > levels) q = levels;
            codes[gi * G + k] = (uint8_t)q;
        }
    }
    return status;
}

/* w~ = fp16((q - z) * s): the integer difference is exact, the product is rounded once. */
static uint16_t pu_value_bits(unsigned q, uint16_t sbits, uint16_t zbits) {
    double z = po_f16_to_f64(zbits);
    return po_f64_to_f16(((double)q - z) * po_f16_to_f64(sbits), NULL);
}

int pu_dequant(const uint8_t* packed, const uint16_t* S, const uint16_t* Z, int64_t N, int64_t K,
               int bits, int G, uint16_t* out) {
    if (!po_args_ok(N, K, bits, G)) return -1;
    const int64_t row_bytes = K * bits / 8, ng = K / G;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        const uint8_t* row = packed + i * row_bytes;
        for (int64_t k = 0; k < K; ++k)
            out[i * K + k] = pu_value_bits(po_code_at(row, k, bits), S[i * ng + k / G], Z[i * ng + k / G]);
    }
    return 0;
}

/* FP64 GEMV/GEMM on the uniform twin's FP16 reconstruction; same conventions as po_matmul. */
int pu_matmul(const uint8_t* packed, const uint16_t* S, const uint16_t* Z, int64_t N, int64_t K,
              int bits, int G, const uint16_t* X, int64_t M, const int64_t* rows, int64_t n_rows,
              double* Y, double* A) {
    if (!po_args_ok(N, K, bits, G) || M < 0 || n_rows < 0) return -1;
    if (!rows && n_rows != N) return -1;
    const int64_t row_bytes = K * bits / 8, ng = K / G;
    int status = 0;
#pragma omp parallel
    {
        double* wrow = (double*)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_rows; ++r) {
            int64_t i = rows ? rows[r] : r;
            if (i < 0 || i >= N || !wrow) {
#pragma omp atomic write
                status = -1;
                continue;
            }
            const uint8_t* row = packed + i * row_bytes;
            for (int64_t k = 0; k < K; ++k)
                wrow[k] = po_f16_to_f64(pu_value_bits(po_code_at(row, k, bits), S[i * ng + k / G], Z[i * ng + k / G]));
            for (int64_t m = 0; m < M; ++m) {
                double y = 0.0, a = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    double p = wrow[k] * po_f16_to_f64(X[m * K + k]);
                    y += p;
                    a += fabs(p);
                }
                Y[m * n_rows + r] = y;
                A[m * n_rows + r] = a;
            }
        }
        free(wrow);
    }
    return status;
}
