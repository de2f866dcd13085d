/*
 * CPU oracle for the W4A8 (INT4-stored weights, FP8 E4M3 math) linear layer of
 * "Dual Precision Quantization".  TEST INFRASTRUCTURE ONLY -- see w4a8_oracle.h.
 *
 * Every function states the passage of the paper it follows.  Arithmetic that the
 * paper writes over the reals is carried out in double unless a step is declared
 * to be an fp32 operation (then it is a single IEEE fp32 operation; build with
 * -ffp-contract=off and without -ffast-math).
 */
#include "w4a8_oracle.h"

#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define E4M3_MAX 448.0f /* Z_max of Eq. 3 for the +-448 variant of Sec. 4.1 */

/* ------------------------------------------------------------------ E4M3 grid, Sec. 2.2 */

/* 1 sign, 4 exponent (bias 7), 3 mantissa bits.  e=0: subnormal (m/8)*2^-6; e=15,m=7: NaN. */
float oracle_e4m3_decode(uint8_t code) {
    int sign = code >> 7;
    int e = (code >> 3) & 0xF;
    int m = code & 0x7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0)
        v = ldexp((double)m / 8.0, -6);
    else
        v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return (float)(sign ? -v : v);
}

/*
 * nearest_Z of Eq. 3: round the exact value to the nearest grid point, ties to the even
 * mantissa, magnitudes above the largest finite value clip to it (Sec. 3.3 "clipping").
 * The sign bit is kept even when the magnitude rounds to zero.
 */
uint8_t oracle_e4m3_encode(float v) {
    uint32_t bits;
    memcpy(&bits, &v, sizeof bits);
    uint8_t sign = (uint8_t)((bits >> 31) << 7);
    if (isnan(v)) return 0x7F;
    double a = fabs((double)v);
    if (a >= 448.0) return sign | 0x7E; /* includes +-inf; 464 is a tie that goes to even = 448 */
    if (a == 0.0) return sign;
    int ex;
    (void)frexp(a, &ex); /* a = f * 2^ex with f in [0.5,1)  ->  floor(log2 a) = ex-1 */
    int e = ex - 1;
    if (e < -6) {
        /* subnormal range: grid spacing 2^-9 */
        double q = ldexp(a, 9);   /* exact */
        int r = (int)nearbyint(q); /* default rounding mode: to nearest, ties to even */
        return sign | (uint8_t)r;  /* r == 8 is the smallest normal, code 0x08 */
    }
    double q = ldexp(a, 3 - e); /* in [8,16), exact */
    int r = (int)nearbyint(q);
    if (r == 16) {
        r = 8;
        e += 1;
    }
    int code = ((e + 7) << 3) | (r - 8);
    if (code > 0x7E) code = 0x7E;
    return sign | (uint8_t)code;
}

void oracle_e4m3_encode_n(const float* v, int64_t n, uint8_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_e4m3_encode(v[i]);
}

void oracle_e4m3_decode_n(const uint8_t* c, int64_t n, float* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_e4m3_decode(c[i]);
}

/* ------------------------------------------------------------------ BF16 bit patterns */

float oracle_bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

uint16_t oracle_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if (isnan(f)) return (uint16_t)((u >> 16) | 0x0040);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb; /* round to nearest, ties to even */
    return (uint16_t)(u >> 16);
}

/* round-to-nearest-integer operator of Eq. 1, ties to even (a choice; the paper only says "nearest") */
static float round_half_even(float x) { return nearbyintf(x); }

static float pow2_ceil(float s) {
    int e;
    float m = frexpf(s, &e); /* s = m*2^e, m in [0.5,1) */
    if (m == 0.5f) return s;
    return ldexpf(1.0f, e);
}

/* ------------------------------------------------------------------ offline RTN quantizer */

/*
 * Eq. 6: s_w = max|W| / Z_max.  Eq. 7: w8 = nearest_Z(w / s_w).
 * Eq. 8: per group, s = (max - min)/15, z = round(-min/s) (range widened to contain 0 so that
 * z stays in [0,15]); Eq. 9: u = round(w8/s + z) clipped to [0,15].
 * Symmetric variant of Eq. 1 (2^n - 2 levels): s = max|w8|/7, u = round(w8/s) + 8.
 * The group scale is rounded to BF16 first, so the codes agree with what is stored.
 * All steps here are single fp32 operations, so that a second implementation can match bit for bit.
 */
int oracle_quantize_weight_rtn(const float* W, int64_t N, int64_t K, int group, int symmetric,
                               int pow2, int per_channel, uint8_t* codes, uint16_t* gscale,
                               uint8_t* gzero, float* s_w) {
    if (!W || !codes || !gscale || !s_w || N <= 0 || K <= 0 || group <= 0 || (group & 1) ||
        K % group != 0)
        return -1;
    if (!symmetric && !gzero) return -1;
    int64_t G = K / group;
    float tmax = 0.0f;
    if (!per_channel) {
        for (int64_t i = 0; i < N * K; ++i) {
            float a = fabsf(W[i]);
            if (a > tmax) tmax = a;
        }
        s_w[0] = (tmax > 0.0f) ? tmax / E4M3_MAX : 1.0f;
    }
    float* w8 = (float*)malloc((size_t)group * sizeof(float));
    if (!w8) return -1;
    for (int64_t n = 0; n < N; ++n) {
        const float* row = W + n * K;
        float sw;
        if (per_channel) {
            float rmax = 0.0f;
            for (int64_t k = 0; k < K; ++k) {
                float a = fabsf(row[k]);
                if (a > rmax) rmax = a;
            }
            sw = (rmax > 0.0f) ? rmax / E4M3_MAX : 1.0f;
            s_w[n] = sw;
        } else {
            sw = s_w[0];
        }
        for (int64_t g = 0; g < G; ++g) {
            float lo = 0.0f, hi = 0.0f, amax = 0.0f;
            for (int j = 0; j < group; ++j) {
                float q = row[g * group + j] / sw;                       /* fp32 division */
                w8[j] = oracle_e4m3_decode(oracle_e4m3_encode(q));       /* Eq. 7 */
                if (w8[j] < lo) lo = w8[j];
                if (w8[j] > hi) hi = w8[j];
                if (fabsf(w8[j]) > amax) amax = fabsf(w8[j]);
            }
            float s;
            int z;
            if (symmetric) {
                s = (amax > 0.0f) ? amax / 7.0f : 1.0f;
                z = 8;
            } else {
                s = (hi > lo) ? (hi - lo) / 15.0f : 1.0f;               /* Eq. 8 */
                z = 0;
            }
            if (pow2) s = pow2_ceil(s);
            uint16_t sb = oracle_f32_to_bf16(s);
            s = oracle_bf16_to_f32(sb);
            if (!symmetric) {
                float zf = round_half_even(-lo / s);                    /* Eq. 8 */
                z = (int)fminf(fmaxf(zf, 0.0f), 15.0f);
            }
            gscale[n * G + g] = sb;
            if (gzero) gzero[n * G + g] = (uint8_t)z;
            for (int j = 0; j < group; ++j) {
                int u;
                if (symmetric) {
                    float q = round_half_even(w8[j] / s);
                    q = fminf(fmaxf(q, -7.0f), 7.0f);
                    u = (int)q + 8;
                } else {
                    float q = round_half_even(w8[j] / s + (float)z);   /* Eq. 9 */
                    u = (int)fminf(fmaxf(q, 0.0f), 15.0f);
                }
                int64_t k = g * group + j;
                uint8_t* byte = codes + n * (K / 2) + k / 2;
                if (k & 1)
                    *byte = (uint8_t)((*byte & 0x0F) | (u << 4));
                else
                    *byte = (uint8_t)((*byte & 0xF0) | u);
            }
        }
    }
    free(w8);
    return 0;
}

/* ------------------------------------------------------------------ Eq. 10 / Eq. 14 */

/*
 * w8_hat[n][k] = nearest_Z( (u - z_g) * s_g ).  The product of a small integer and a BF16
 * value is exact in fp32, so this is the real number (u-z)*s rounded once to E4M3; its
 * sign (also of a zero product) is that of the fp32 product.
 */
int oracle_dequant_weight(const uint8_t* codes, const uint16_t* gscale, const uint8_t* gzero,
                          int64_t N, int64_t K, int group, uint8_t* w8) {
    if (!codes || !gscale || !w8 || N <= 0 || K <= 0 || group <= 0 || (group & 1) || K % group != 0)
        return -1;
    int64_t G = K / group;
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t k = 0; k < K; ++k) {
            int64_t g = k / group;
            uint8_t byte = codes[n * (K / 2) + k / 2];
            int u = (k & 1) ? (byte >> 4) : (byte & 0x0F);
            int z = gzero ? gzero[n * G + g] : 8;
            float s = oracle_bf16_to_f32(gscale[n * G + g]);
            float prod = (float)(u - z) * s; /* exact */
            w8[n * K + k] = oracle_e4m3_encode(prod);
        }
    }
    return 0;
}

/*
 * Eq. 10 when the weights were quantized in an unconstrained activation order (the W4A8* rows
 * of Table 3; appendix "Activation Reordering"): after the codes are put back in their original
 * positions the scale and zero-point of column k are those of group g_idx[k] of the processing
 * order, no longer of k / group -- every weight needs its own look-up.
 */
int oracle_dequant_weight_gidx(const uint8_t* codes, const uint16_t* gscale, const uint8_t* gzero,
                               const int32_t* g_idx, int64_t N, int64_t K, int64_t G, uint8_t* w8) {
    if (!codes || !gscale || !g_idx || !w8 || N <= 0 || K <= 0 || G <= 0 || (K & 1)) return -1;
    for (int64_t k = 0; k < K; ++k)
        if (g_idx[k] < 0 || g_idx[k] >= G) return -1;
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t k = 0; k < K; ++k) {
            int64_t g = g_idx[k];
            uint8_t byte = codes[n * (K / 2) + k / 2];
            int u = (k & 1) ? (byte >> 4) : (byte & 0x0F);
            int z = gzero ? gzero[n * G + g] : 8;
            float s = oracle_bf16_to_f32(gscale[n * G + g]);
            w8[n * K + k] = oracle_e4m3_encode((float)(u - z) * s);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ Eq. 13 */

/*
 * Per token (row): amax = max_k |x|; s_x = amax / Z_max (fp32 division); the quotient x/s_x of
 * Eq. 13 is taken as the fp32 product x * inv with inv = Z_max / amax (fp32 division), then
 * rounded once to E4M3 with saturation.  An all-zero row takes s_x = 1.
 * Power-of-two mode (Sec. 2.2): s_x is rounded up to a power of two and x/s_x is exact.
 * Static mode (Sec. 3.1, "computed offline"): s_x is given; inv = 1/s_x (fp32 division).
 */
int oracle_quantize_act(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, uint8_t* x8,
                        int64_t ldx8, float* s_x, int scale_mode, const float* static_scale) {
    if (!x || !x8 || !s_x || M <= 0 || K <= 0 || ldx < K || ldx8 < K) return -1;
    if (scale_mode != 0 && scale_mode != 1) return -1;
    for (int64_t m = 0; m < M; ++m) {
        const uint16_t* row = x + m * ldx;
        float s, inv;
        if (static_scale) {
            s = *static_scale;
            inv = 1.0f / s;
        } else {
            float amax = 0.0f;
            for (int64_t k = 0; k < K; ++k) {
                float a = fabsf(oracle_bf16_to_f32(row[k]));
                if (a > amax) amax = a;
            }
            if (amax == 0.0f) {
                s = 1.0f;
                inv = 1.0f;
            } else if (scale_mode == 1) {
                s = pow2_ceil(amax / E4M3_MAX);
                inv = 1.0f / s; /* exact: s is a power of two */
            } else {
                s = amax / E4M3_MAX;
                inv = E4M3_MAX / amax;
            }
        }
        s_x[m] = s;
        for (int64_t k = 0; k < K; ++k) {
            float q = oracle_bf16_to_f32(row[k]) * inv; /* one fp32 multiply */
            x8[m * ldx8 + k] = oracle_e4m3_encode(q);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ FP8 matmul + Eq. 4 / Eq. 11 */

/*
 * acc[m][n] = sum_k x8[m][k] * w8[n][k] over the decoded FP8 values, in double.  Every product
 * is a multiple of 2^-18 below 2^18, so the double sum is exact for any K used here.
 * y = acc * s_x[m] * s_w[n]  (Eq. 4 undoes the activation scale, Eq. 11 the weight scale).
 */
int oracle_linear(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* w8,
                  const float* s_w, int sw_stride, int64_t N, int64_t K, const int64_t* cols,
                  int64_t ncols, double* y64, float* y32, uint16_t* ybf16, double* yabs) {
    if (!x8 || !s_x || !w8 || !s_w || M <= 0 || N <= 0 || K <= 0 || ldx8 < K) return -1;
    if (sw_stride != 0 && sw_stride != 1) return -1;
    double dec[256];
    for (int c = 0; c < 256; ++c) dec[c] = (double)oracle_e4m3_decode((uint8_t)c);
    int64_t NC = cols ? ncols : N;
    if (NC <= 0) return -1;
    for (int64_t j = 0; j < NC; ++j) {
        int64_t n = cols ? cols[j] : j;
        if (n < 0 || n >= N) return -1;
    }
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < NC; ++j) {
        int64_t n = cols ? cols[j] : j;
        const uint8_t* wr = w8 + n * K;
        for (int64_t m = 0; m < M; ++m) {
            const uint8_t* xr = x8 + m * ldx8;
            double acc = 0.0, aabs = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double p = dec[xr[k]] * dec[wr[k]];
                acc += p;
                aabs += fabs(p);
            }
            double scale = (double)s_x[m] * (double)s_w[n * sw_stride];
            double y = acc * scale;
            int64_t o = m * NC + j;
            if (y64) y64[o] = y;
            if (y32) y32[o] = (float)y;
            if (ybf16) ybf16[o] = oracle_f32_to_bf16((float)y);
            if (yabs) yabs[o] = aabs * fabs(scale);
        }
    }
    return 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
