/*
 * CPU oracle for the DPQ weight quantizer (Algorithm 1, Sec. 3.1-3.3 and the appendix on
 * Group-Aware Reordering).
 *
 * TEST INFRASTRUCTURE ONLY (see w4a8_oracle.h).  Scalar C, one weight at a time, in the order
 * and notation of Algorithm 1:
 *
 *   s_w = max|W| / Z_max                                   (Eq. 6)
 *   for each row, for each group g (in processing order):
 *       group scale s_g and zero-point z_g from the group's current weights  (Eq. 8; optional
 *                                                           search of the scale with least squared error, Sec. 3.3)
 *       for each weight w of the group (left to right in processing order):
 *           w8   = nearest_Z(w / s_w)                      (Eq. 7)
 *           u    = round(w8 / s_g + z_g) clipped to 0..15  (Eq. 9)
 *           w8^  = nearest_Z((u - z_g) * s_g)              (Eq. 10, as the inference path computes it)
 *           w16^ = w8^ * s_w                               (Eq. 11)
 *           e    = (w - w16^) / [H_F^-1]_qq
 *           w_v <- w_v - e * (H_F^-1)_qv  for every v to the right   (Eq. 12)
 *
 * The inverse Hessians of the shrinking sets F are not formed one by one: as in GPTQ (which
 * Sec. 3.3 follows) row q of the upper Cholesky factor U of H^-1 holds (H_F^-1)_qv / sqrt of
 * [H_F^-1]_qq, so that with e = (w - w16^) / U_qq the update is w_v <- w_v - e * U_qv.  U is an
 * INPUT here (it comes from a factorization routine, in processing order, after dampening).
 *
 * Group-Aware Reordering: `perm` gives the processing order; position p handles original column
 * perm[p].  A processing group (`group` consecutive positions) must hold exactly the columns of
 * one original group, so that scale and zero-point go back to that group when the codes are put
 * back in the original order.
 *
 * Precision.  The paper does not fix one.  Every step that decides an integer is a single fp32
 * operation written out below (division, multiply, fused multiply-add for the update), so that
 * a second implementation can take the same decisions; the squared errors of the scale search
 * are summed as exact integers (all terms are multiples of 2^-18).
 *
 * Readings of the paper taken here: the range of Eq. 8 is widened to contain 0; integer rounding
 * is half-to-even; the group scale is rounded to BF16 before it is used; w8^ is rounded to the
 * E4M3 grid because that is what inference multiplies with; the scale search tries
 * mse_steps shrink factors 1, 0.98, 0.96, ... of the range and keeps the first best.
 * "parity unpinned": these readings, the search grid, the dampening and dead-column handling done
 * by the caller.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "w4a8_oracle.h"

#define E4M3_MAX 448.0f

static float rhe(float x) { return nearbyintf(x); } /* round half to even (default rounding mode) */

/* Eq. 8 (asymmetric, range widened to 0) or the symmetric variant of Eq. 1, for the range shrunk
 * by p; the scale is rounded to BF16. */
static void group_params(float lo, float hi, float amax, float p, int symmetric, float* s_out, int* z_out) {
    float s;
    int z;
    if (symmetric) {
        float a = p * amax;
        s = (a > 0.0f) ? a / 7.0f : 1.0f;
        z = 8;
        s = oracle_bf16_to_f32(oracle_f32_to_bf16(s));
    } else {
        float l = p * lo, h = p * hi;
        s = (h > l) ? (h - l) / 15.0f : 1.0f;
        s = oracle_bf16_to_f32(oracle_f32_to_bf16(s));
        float zf = rhe(-l / s);
        z = (int)fminf(fmaxf(zf, 0.0f), 15.0f);
    }
    *s_out = s;
    *z_out = z;
}

/* Eq. 9 then Eq. 10 for one FP8-valued weight: returns the code, *w8hat = the value inference sees. */
static int quant_dequant(float w8, float s, int z, int symmetric, float* w8hat) {
    int u;
    if (symmetric) {
        float q = rhe(w8 / s);
        q = fminf(fmaxf(q, -7.0f), 7.0f);
        u = (int)q + 8;
    } else {
        float q = rhe(w8 / s + (float)z);
        u = (int)fminf(fmaxf(q, 0.0f), 15.0f);
    }
    *w8hat = oracle_e4m3_decode(oracle_e4m3_encode((float)(u - z) * s));
    return u;
}

int oracle_dpq_quantize(const float* W, int64_t N, int64_t K, int group, const float* U, const int32_t* perm,
                        int symmetric, int mse_steps, int per_channel, uint8_t* codes, uint16_t* gscale,
                        uint8_t* gzero, float* s_w, float* err_out, float* what_out) {
    if (!W || !U || !codes || !gscale || !s_w || N <= 0 || K <= 0 || group <= 0 || (group & 1) || K % group != 0)
        return -1;
    if (!symmetric && !gzero) return -1;
    if (mse_steps < 0 || mse_steps > 11) return -1;
    const int64_t G = K / group;
    /* the processing order must keep original groups together */
    for (int64_t g = 0; g < G; ++g) {
        int64_t og = perm ? perm[g * group] / group : g;
        for (int j = 0; j < group; ++j) {
            int64_t c = perm ? perm[g * group + j] : g * group + j;
            if (c < 0 || c >= K || c / group != og) return -1;
        }
    }
    if (!per_channel) {
        float tmax = 0.0f;
        for (int64_t i = 0; i < N * K; ++i) {
            float a = fabsf(W[i]);
            if (a > tmax) tmax = a;
        }
        s_w[0] = (tmax > 0.0f) ? tmax / E4M3_MAX : 1.0f; /* Eq. 6 */
    }
    memset(codes, 0, (size_t)N * (size_t)(K / 2));
    int failed = 0;
    /* rows are independent (Algorithm 1 loops over them); they may run on several cores */
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t n = 0; n < N; ++n) {
        float* w = (float*)malloc((size_t)K * sizeof(float)); /* the row in processing order, updated in place */
        float* w8 = (float*)malloc((size_t)group * sizeof(float));
        if (!w || !w8) {
            free(w);
            free(w8);
#pragma omp atomic write
            failed = 1;
            continue;
        }
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
        for (int64_t p = 0; p < K; ++p) w[p] = row[perm ? perm[p] : p];
        for (int64_t g = 0; g < G; ++g) {
            const int64_t p0 = g * group;
            const int64_t og = perm ? perm[p0] / group : g;
            /* scale and zero-point of the group, once, from its current (compensated) weights */
            float lo = 0.0f, hi = 0.0f, amax = 0.0f;
            for (int j = 0; j < group; ++j) {
                w8[j] = oracle_e4m3_decode(oracle_e4m3_encode(w[p0 + j] / sw)); /* Eq. 7 */
                if (w8[j] < lo) lo = w8[j];
                if (w8[j] > hi) hi = w8[j];
                if (fabsf(w8[j]) > amax) amax = fabsf(w8[j]);
            }
            float s;
            int z;
            group_params(lo, hi, amax, 1.0f, symmetric, &s, &z);
            if (mse_steps > 1) {
                /* Sec. 3.3: the scale with the least squared error over the group, among shrunk ranges */
                int64_t best = -1;
                for (int t = 0; t < mse_steps; ++t) {
                    float pt = 1.0f - (float)t * 0.02f;
                    float st;
                    int zt;
                    group_params(lo, hi, amax, pt, symmetric, &st, &zt);
                    int64_t e2 = 0;
                    for (int j = 0; j < group; ++j) {
                        float h;
                        (void)quant_dequant(w8[j], st, zt, symmetric, &h);
                        int64_t d = (int64_t)((w8[j] - h) * 512.0f); /* exact: both on the 2^-9 grid */
                        e2 += d * d;
                    }
                    if (best < 0 || e2 < best) {
                        best = e2;
                        s = st;
                        z = zt;
                    }
                }
            }
            gscale[n * G + og] = oracle_f32_to_bf16(s);
            if (gzero) gzero[n * G + og] = (uint8_t)z;
            for (int j = 0; j < group; ++j) {
                const int64_t q = p0 + j;
                float wq8 = oracle_e4m3_decode(oracle_e4m3_encode(w[q] / sw)); /* Eq. 7 on the compensated weight */
                float h8;
                int u = quant_dequant(wq8, s, z, symmetric, &h8); /* Eq. 9, Eq. 10 */
                float h16 = h8 * sw;                              /* Eq. 11 */
                float e = (w[q] - h16) / U[q * K + q];
                if (err_out) err_out[n * K + q] = e;
                if (what_out) what_out[n * K + q] = h16;
                for (int64_t v = q + 1; v < K; ++v) w[v] = fmaf(-e, U[q * K + v], w[v]); /* Eq. 12 */
                const int64_t c = perm ? perm[q] : q;
                uint8_t* byte = codes + n * (K / 2) + c / 2;
                if (c & 1)
                    *byte = (uint8_t)((*byte & 0x0F) | (u << 4));
                else
                    *byte = (uint8_t)((*byte & 0xF0) | u);
            }
        }
        free(w);
        free(w8);
    }
    return failed ? -1 : 0;
}
