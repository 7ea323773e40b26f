/*
 * CPU oracle for the DPS dual-precision linear-layer path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, header, table or helper
 * with the CUDA path and must never be linked into, imported by or called from
 * the product path.  Only tests, the smoke check and the benchmark's
 * cpu-baseline leg may use it.
 *
 * What it follows (paper sections):
 *   - Nested split of an FP16 word into a persistent FP8 byte and a residual
 *     byte: "Mapper: Semi-Unified Memory Abstraction", paragraph "Persistent
 *     Region" (E5M2: all five exponent bits + two mantissa MSBs; E4M3: when the
 *     exponent MSB is zero, four exponent bits + three mantissa MSBs), and the
 *     restore paragraph that calls the residual "the lower FP8 byte".
 *   - Full mode combines the two tensors back into the original FP16 values;
 *     fast mode uses the FP8 tensor alone and never touches the residual:
 *     "Scheduler: Dual-Precision Execution", paragraph "Overall concept".
 *   - Per-layer encoding chosen offline from weight statistics, E5M2 for layers
 *     whose magnitudes fall outside what E4M3 expresses: same section,
 *     paragraph "Dual-mode serving (DPS) with asymmetric switching".
 *   - Dense and MoE (grouped) linear layers: same paragraph.
 *
 * Readings taken where the paper is silent (all listed in the design notes):
 *   truncation (bit selection), not rounding; E4M3 drops exponent bit e[4];
 *   the E4M3 residual's bit 7 is written 0 and ignored on read; E4M3 is
 *   eligible iff every word has bit 14 clear and max|w| <= 1.75 (the range the
 *   paper's source mentions), with an explicit E4M3 request accepted whenever
 *   bit 14 is clear everywhere and no byte lands on the 0x7F/0xFF code;
 *   activations stay FP16; the reference product is accumulated in FP64.
 *
 * Every function here is pinned by tests that do not use this file's own
 * arithmetic: exhaustive round trips, float8 casts of an independent library,
 * hand-derived IEEE-754 fixtures, closed-form bounds, brute force and a
 * library matmul on the unsplit weights.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_MODE_FAST = 0, ORACLE_MODE_FULL = 1 };
enum { ORACLE_ENC_AUTO = 0, ORACLE_ENC_E4M3 = 1, ORACLE_ENC_E5M2 = 2, ORACLE_ENC_E4M3_RN = 3, ORACLE_ENC_E5M2_RN = 4 };
enum { ORACLE_OK = 0, ORACLE_ERR_ARG = 1, ORACLE_ERR_DATA = 8 };

/* ---- IEEE-754 binary16 <-> binary64, written from the format definition ---- */

double oracle_half_to_double(uint16_t b) {
    int s = (b >> 15) & 1;
    int e = (b >> 10) & 0x1F;
    int m = b & 0x3FF;
    double v;
    if (e == 0) {
        v = ldexp((double)m, -24);            /* subnormal: m * 2^-10 * 2^-14 */
    } else if (e == 31) {
        v = m ? NAN : INFINITY;
    } else {
        v = ldexp((double)(1024 + m), e - 25); /* (1 + m/1024) * 2^(e-15) */
    }
    return s ? -v : v;
}

/* Round-to-nearest-even to binary16.  Informational output only: parity of the
 * GEMM is judged on the FP64 value. */
uint16_t oracle_double_to_half(double v) {
    uint16_t sign = signbit(v) ? 0x8000u : 0u;
    double a = fabs(v);
    if (isnan(v)) return (uint16_t)(sign | 0x7E00u);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7C00u);  /* rounds to +-inf */
    if (a == 0.0) return sign;
    int ex;
    (void)frexp(a, &ex);                  /* a = f * 2^ex, f in [0.5,1) */
    int e = ex - 1;                       /* a in [2^e, 2^(e+1)) */
    if (e < -14) e = -14;                 /* subnormal quantum is 2^-24 */
    double q = nearbyint(ldexp(a, 10 - e)); /* default mode: ties to even */
    /* q in [0, 2048]; q == 2048 means the mantissa carried into the exponent */
    uint32_t bits;
    if (e == -14 && q < 1024.0) {
        bits = (uint32_t)q;               /* subnormal (or zero) */
    } else {
        if (q >= 2048.0) { q = 1024.0; e += 1; }
        bits = ((uint32_t)(e + 15) << 10) | ((uint32_t)q - 1024u);
    }
    return (uint16_t)(sign | bits);
}

/* ---- encoding eligibility and selection ---- */

/* 1 if every word has bit 14 (exponent MSB) clear. */
static int all_exp_msb_zero(const uint16_t* w, int64_t n) {
    for (int64_t i = 0; i < n; ++i)
        if (w[i] & 0x4000u) return 0;
    return 1;
}

/* AUTO rule: E4M3 iff exponent MSB is zero everywhere and max|w| <= 1.75. */
int oracle_select_encoding(const uint16_t* w, int64_t n) {
    if (!all_exp_msb_zero(w, n)) return ORACLE_ENC_E5M2;
    for (int64_t i = 0; i < n; ++i)
        if (fabs(oracle_half_to_double(w[i])) > 1.75) return ORACLE_ENC_E5M2;
    return ORACLE_ENC_E4M3;
}

/* An explicit E4M3 request is legal iff the exponent MSB is zero everywhere
 * and no persistent byte would be 0x7F / 0xFF (all kept bits set). */
int oracle_e4m3_legal(const uint16_t* w, int64_t n) {
    for (int64_t i = 0; i < n; ++i) {
        if (w[i] & 0x4000u) return 0;
        if (((w[i] >> 7) & 0x7Fu) == 0x7Fu) return 0;
    }
    return 1;
}

/* ---- rounded nests (an extension; the paper describes bit selection only) ----
 * The stored pair is the truncated split of b' = b + h, h = half a unit of the last bit the
 * persistent byte keeps (E5M2: 0x0080, E4M3: 0x0040).  The persistent byte is then the FP8 value
 * nearest to the weight, ties away from zero (pinned in the tests against that definition), and
 * join(P, R) - h gives b back.  Legal iff no b' reaches an Inf / NaN code. */
static int is_rounded(int enc) { return enc == ORACLE_ENC_E4M3_RN || enc == ORACLE_ENC_E5M2_RN; }
static int base_of(int enc) {
    return enc == ORACLE_ENC_E4M3_RN ? ORACLE_ENC_E4M3 : enc == ORACLE_ENC_E5M2_RN ? ORACLE_ENC_E5M2 : enc;
}
static unsigned half_unit(int enc) { return enc == ORACLE_ENC_E4M3_RN ? 0x40u : enc == ORACLE_ENC_E5M2_RN ? 0x80u : 0u; }
static int known_enc(int enc) { return enc >= ORACLE_ENC_E4M3 && enc <= ORACLE_ENC_E5M2_RN; }

int oracle_rounded_legal(const uint16_t* w, int64_t n, int enc) {
    if (!is_rounded(enc)) return 0;
    const unsigned limit = enc == ORACLE_ENC_E5M2_RN ? 0x7C00u : 0x3F80u;
    for (int64_t i = 0; i < n; ++i)
        if ((w[i] & 0x7FFFu) + half_unit(enc) >= limit) return 0;
    return 1;
}

/* ---- split / reconstruct / fast value: one element ---- */

static void split_trunc(uint16_t b, int enc, uint8_t* p, uint8_t* r);
static uint16_t join_trunc(uint8_t p, uint8_t r, int enc);

static void split_one(uint16_t b, int enc, uint8_t* p, uint8_t* r) {
    split_trunc((uint16_t)(b + half_unit(enc)), base_of(enc), p, r);
}

/* residual == NULL-like use: the callers pass r = 0 AND full = 0 for the fast-mode value, which is
 * the value of the persistent byte itself, also for a rounded nest. */
static uint16_t join_one_mode(uint8_t p, uint8_t r, int enc, int full) {
    if (!full) return join_trunc(p, 0, base_of(enc));
    return (uint16_t)(join_trunc(p, r, base_of(enc)) - half_unit(enc));
}

static void split_trunc(uint16_t b, int enc, uint8_t* p, uint8_t* r) {
    unsigned s = (b >> 15) & 1u, e = (b >> 10) & 0x1Fu, m = b & 0x3FFu;
    if (enc == ORACLE_ENC_E5M2) {
        *p = (uint8_t)((s << 7) | (e << 2) | (m >> 8));   /* s e4..e0 m9 m8 */
        *r = (uint8_t)(m & 0xFFu);                        /* m7..m0 */
    } else {
        *p = (uint8_t)((s << 7) | ((e & 0xFu) << 3) | (m >> 7)); /* s e3..e0 m9..m7 */
        *r = (uint8_t)(m & 0x7Fu);                        /* 0 m6..m0 */
    }
}

static uint16_t join_trunc(uint8_t p, uint8_t r, int enc) {
    unsigned s = (p >> 7) & 1u;
    if (enc == ORACLE_ENC_E5M2) {
        unsigned e = (p >> 2) & 0x1Fu, mh = p & 3u;
        return (uint16_t)((s << 15) | (e << 10) | (mh << 8) | r);
    } else {
        unsigned e = (p >> 3) & 0xFu, mh = p & 7u;
        return (uint16_t)((s << 15) | (e << 10) | (mh << 7) | (r & 0x7Fu));
    }
}

/* FP16 -> (P, R).  enc must be E4M3 or E5M2 (the caller resolves AUTO with
 * oracle_select_encoding).  An illegal E4M3 request leaves the planes alone. */
int oracle_split(const uint16_t* w, uint8_t* p, uint8_t* r, int64_t n, int enc) {
    if (!known_enc(enc)) return ORACLE_ERR_ARG;
    if (enc == ORACLE_ENC_E4M3 && !oracle_e4m3_legal(w, n)) return ORACLE_ERR_DATA;
    if (is_rounded(enc) && !oracle_rounded_legal(w, n, enc)) return ORACLE_ERR_DATA;
    for (int64_t i = 0; i < n; ++i) split_one(w[i], enc, &p[i], &r[i]);
    return ORACLE_OK;
}

/* (P, R) -> original FP16 words (full mode's weights). */
int oracle_reconstruct(const uint8_t* p, const uint8_t* r, uint16_t* w, int64_t n, int enc) {
    if (!known_enc(enc)) return ORACLE_ERR_ARG;
    for (int64_t i = 0; i < n; ++i) w[i] = join_one_mode(p[i], r[i], enc, 1);
    return ORACLE_OK;
}

/* P alone -> FP16 words of the fast-mode weights (residual taken as zero). */
int oracle_fast_words(const uint8_t* p, uint16_t* w, int64_t n, int enc) {
    if (!known_enc(enc)) return ORACLE_ERR_ARG;
    for (int64_t i = 0; i < n; ++i) w[i] = join_one_mode(p[i], 0, enc, 0);
    return ORACLE_OK;
}

/* ---- linear layers ---- */

/* Effective weight of element i of a plane pair, as a double. */
static double eff_weight(int mode, int enc, const uint8_t* p, const uint8_t* r, int64_t i) {
    if (mode != ORACLE_MODE_FULL) return oracle_half_to_double(join_one_mode(p[i], 0, enc, 0)); /* fast mode never reads r */
    return oracle_half_to_double(join_one_mode(p[i], r[i], enc, 1));
}

/* y_ref[m][n] = sum_k x[m][k] * W_eff[n][k], FP64, k ascending.
 * x: FP16 words [M][K]; p, r: [N][K]; y_ref: double [M][N]; y_half (may be
 * NULL): FP16 rounding of y_ref.  threads <= 1 runs single-threaded; larger
 * values split the independent output columns n over OpenMP threads (the sum
 * for each output is still taken in the same order). */
int oracle_linear(int mode, int enc, const uint16_t* x, const uint8_t* p, const uint8_t* r,
                  double* y_ref, uint16_t* y_half, int64_t M, int64_t N, int64_t K, int threads) {
    if (mode != ORACLE_MODE_FAST && mode != ORACLE_MODE_FULL) return ORACLE_ERR_ARG;
    if (!known_enc(enc)) return ORACLE_ERR_ARG;
    if (M == 0 || N == 0) return ORACLE_OK;
    double* xd = (double*)malloc(sizeof(double) * (size_t)(M * K > 0 ? M * K : 1));
    if (!xd) return ORACLE_ERR_ARG;
    for (int64_t i = 0; i < M * K; ++i) xd[i] = oracle_half_to_double(x[i]);
    if (threads < 1) threads = 1;
#pragma omp parallel num_threads(threads)
    {
        double* wrow = (double*)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
#pragma omp for schedule(static)
        for (int64_t n = 0; n < N; ++n) {
            for (int64_t k = 0; k < K; ++k) wrow[k] = eff_weight(mode, enc, p, r, n * K + k);
            for (int64_t m = 0; m < M; ++m) {
                double acc = 0.0;
                for (int64_t k = 0; k < K; ++k) acc += xd[m * K + k] * wrow[k];
                y_ref[m * N + n] = acc;
                if (y_half) y_half[m * N + n] = oracle_double_to_half(acc);
            }
        }
        free(wrow);
    }
    free(xd);
    return ORACLE_OK;
}

/* Selected outputs only: out[i] = y_ref[ms[i]][ns[i]].  For full-size checks
 * where the whole product would take hours. */
int oracle_linear_at(int mode, int enc, const uint16_t* x, const uint8_t* p, const uint8_t* r,
                     int64_t M, int64_t N, int64_t K, const int64_t* ms, const int64_t* ns,
                     int64_t count, double* out) {
    if (mode != ORACLE_MODE_FAST && mode != ORACLE_MODE_FULL) return ORACLE_ERR_ARG;
    if (!known_enc(enc)) return ORACLE_ERR_ARG;
    for (int64_t i = 0; i < count; ++i) {
        int64_t m = ms[i], n = ns[i];
        if (m < 0 || m >= M || n < 0 || n >= N) return ORACLE_ERR_ARG;
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k)
            acc += oracle_half_to_double(x[m * K + k]) * eff_weight(mode, enc, p, r, n * K + k);
        out[i] = acc;
    }
    return ORACLE_OK;
}

/* Grouped (MoE) linear: for each row a,
 *   y_ref[a][:] = x[token_of_row ? token_of_row[a] : a][:] * W_eff(expert_of_row[a])^T
 * p, r: [E][N][K]; enc_per_expert: E entries; x: [T][K]; y_ref: [A][N].
 * Rows whose expert or token index is out of range are skipped (their outputs
 * are left untouched) and the call returns ORACLE_ERR_DATA after finishing the
 * valid rows.  rows_sel (may be NULL) restricts the work to the listed rows. */
int oracle_moe_linear(int mode, const int32_t* enc_per_expert, const uint16_t* x,
                      const int32_t* token_of_row, const int32_t* expert_of_row,
                      const uint8_t* p, const uint8_t* r, double* y_ref, uint16_t* y_half,
                      int64_t A, int64_t T, int64_t N, int64_t K, int32_t E,
                      const int64_t* rows_sel, int64_t n_sel, int threads) {
    if (mode != ORACLE_MODE_FAST && mode != ORACLE_MODE_FULL) return ORACLE_ERR_ARG;
    for (int32_t e = 0; e < E; ++e)
        if (!known_enc(enc_per_expert[e]))
            return ORACLE_ERR_ARG;
    int bad = 0;
    int64_t count = rows_sel ? n_sel : A;
    if (threads < 1) threads = 1;
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads) reduction(| : bad)
    for (int64_t i = 0; i < count; ++i) {
        int64_t a = rows_sel ? rows_sel[i] : i;
        if (a < 0 || a >= A) { bad |= 1; continue; }
        int64_t t = token_of_row ? (int64_t)token_of_row[a] : a;
        int64_t e = expert_of_row[a];
        if (e < 0 || e >= E || t < 0 || t >= T) { bad |= 1; continue; }
        const uint8_t* pe = p + (size_t)e * (size_t)N * (size_t)K;
        const uint8_t* re = r ? r + (size_t)e * (size_t)N * (size_t)K : NULL;
        int enc = enc_per_expert[e];
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k)
                acc += oracle_half_to_double(x[t * K + k]) * eff_weight(mode, enc, pe, re, n * K + k);
            y_ref[a * N + n] = acc;
            if (y_half) y_half[a * N + n] = oracle_double_to_half(acc);
        }
    }
    return bad ? ORACLE_ERR_DATA : ORACLE_OK;
}

/* ---- FP8 activations for fast mode (the paper's "doubling peak tensor-core throughput with
 * hardware support" option: "Persistent Region" paragraph, remark on FP8 execution).  The paper
 * gives no recipe; the reading taken (listed in the design notes) is per-token dynamic scaling:
 *   scale[m] = max_k |x[m][k]| / 448   (448 = largest finite E4M3 value; 1 if the row is all zero),
 *   q[m][k]  = E4M3( x[m][k] / scale[m] ), round to nearest even, saturating,
 * both computed in binary32 (the precision the decision is taken in), and
 *   y_ref[m][n] = scale[m] * sum_k value(q[m][k]) * W_fast[n][k]   in FP64.
 * E4M3 here is the 8-bit format with bias 7, no infinities, one NaN code per sign (0x7F / 0xFF),
 * subnormals with exponent field 0: value = (-1)^s 2^(e-7) (1 + m/8), or 2^-6 (m/8) for e = 0. */

double oracle_e4m3_to_double(uint8_t b) {
    int s = b >> 7, e = (b >> 3) & 0xF, m = b & 7;
    double v;
    if (e == 0xF && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return s ? -v : v;
}

/* binary32 -> E4M3, round to nearest even, values beyond 448 saturate to +-448, NaN -> 0x7F.
 * Written from the format: find the two neighbouring representable values and pick the nearer,
 * the one with even mantissa code on a tie. */
uint8_t oracle_float_to_e4m3(float f) {
    if (f != f) return 0x7F;
    uint8_t sign = (f < 0.0f || (f == 0.0f && 1.0f / f < 0.0f)) ? 0x80 : 0x00;
    double a = fabs((double)f);
    if (a >= 448.0) return sign | 0x7E;
    /* codes 0x00..0x7E are monotone in value: binary search for the largest code with value <= a */
    int lo = 0, hi = 0x7E;
    while (lo < hi) {
        int mid = (lo + hi + 1) / 2;
        if (oracle_e4m3_to_double((uint8_t)mid) <= a) lo = mid; else hi = mid - 1;
    }
    if (lo < 0x7E) {
        double below = oracle_e4m3_to_double((uint8_t)lo), above = oracle_e4m3_to_double((uint8_t)(lo + 1));
        double d0 = a - below, d1 = above - a;
        if (d1 < d0 || (d1 == d0 && (lo & 1))) lo += 1;
    }
    return sign | (uint8_t)lo;
}

/* x: FP16 words [M][K] -> q: E4M3 bytes [M][K], scale: binary32 [M]. */
int oracle_quantize_activations(const uint16_t* x, uint8_t* q, float* scale, int64_t M, int64_t K) {
    for (int64_t m = 0; m < M; ++m) {
        float amax = 0.0f;
        for (int64_t k = 0; k < K; ++k) {
            float v = (float)fabs(oracle_half_to_double(x[m * K + k]));
            if (v != v) return ORACLE_ERR_DATA;
            if (v > amax) amax = v;
        }
        if (isinf(amax)) return ORACLE_ERR_DATA;
        float sc = amax > 0.0f ? amax / 448.0f : 1.0f;   /* binary32 division, round to nearest */
        scale[m] = sc;
        for (int64_t k = 0; k < K; ++k) {
            float v = (float)oracle_half_to_double(x[m * K + k]);
            q[m * K + k] = oracle_float_to_e4m3(v / sc);   /* binary32 division, then one rounding to E4M3 */
        }
    }
    return ORACLE_OK;
}

/* y_ref[m][n] = scale[m] * sum_k value(q[m][k]) * W_fast[n][k], FP64, k ascending. */
int oracle_linear_fp8act(int enc, const uint8_t* q, const float* scale, const uint8_t* p, double* y_ref, int64_t M,
                         int64_t N, int64_t K, int threads) {
    if (!known_enc(enc)) return ORACLE_ERR_ARG;
    if (M == 0 || N == 0) return ORACLE_OK;
    double* xd = (double*)malloc(sizeof(double) * (size_t)(M * K > 0 ? M * K : 1));
    if (!xd) return ORACLE_ERR_ARG;
    for (int64_t i = 0; i < M * K; ++i) xd[i] = oracle_e4m3_to_double(q[i]);
    if (threads < 1) threads = 1;
#pragma omp parallel num_threads(threads)
    {
        double* wrow = (double*)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
#pragma omp for schedule(static)
        for (int64_t n = 0; n < N; ++n) {
            for (int64_t k = 0; k < K; ++k) wrow[k] = eff_weight(ORACLE_MODE_FAST, enc, p, NULL, n * K + k);
            for (int64_t m = 0; m < M; ++m) {
                double acc = 0.0;
                for (int64_t k = 0; k < K; ++k) acc += xd[m * K + k] * wrow[k];
                y_ref[m * N + n] = acc * (double)scale[m];
            }
        }
        free(wrow);
    }
    free(xd);
    return ORACLE_OK;
}

int oracle_version(void) { return 3; }
