/*
 * CPU oracle for the W4A8 linear layer of "Dual Precision Quantization" (DPQ).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, scalar C written from the paper's
 * equations.  It shares no code with the CUDA library and must never be on a
 * product path: only the test-suite, the smoke check and the benchmark's
 * CPU-baseline leg may load it.
 *
 * Conventions (the paper is silent on storage details; these are decisions):
 *   - E4M3 is the OCP "fn" variant: bias 7, no infinities, 0x7F/0xFF = NaN,
 *     max finite 448 (the +-448 range of Sec. 4.1).
 *   - INT4 codes u in [0,15] are packed two per byte along K, even k in the
 *     low nibble.  Groups of `group` consecutive k share one scale (BF16 bit
 *     pattern, uint16) and one integer zero-point (uint8 in [0,15]).
 *     gzero == NULL means symmetric storage, z = 8 for every group.
 *   - BF16 tensors travel as uint16 bit patterns.
 *
 * "parity unpinned" items: the storage conventions above (scale dtype, nibble
 * order, matrix orientation), the tie-break of the integer rounding operator
 * in Eq. 1/8/9 (half-to-even here) and the operational fp32 definition of the
 * activation quotient of Eq. 13 are choices the paper does not fix; no value
 * printed in the paper pins them.
 */
#ifndef W4A8_ORACLE_H
#define W4A8_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Sec. 2.2 (E4M3 grid Z, "nearest_Z"): decode one code to its real value. NaN codes give NaN. */
float oracle_e4m3_decode(uint8_t code);
/* Sec. 2.2, Eq. 3 "nearest_Z" with ties-to-even and saturation to +-448 (the clipping of Sec. 3.3). */
uint8_t oracle_e4m3_encode(float v);
/* The scalar encoder / decoder applied to n elements. */
void oracle_e4m3_encode_n(const float* v, int64_t n, uint8_t* out);
void oracle_e4m3_decode_n(const uint8_t* c, int64_t n, float* out);

/* BF16 helpers (bit patterns). */
float oracle_bf16_to_f32(uint16_t b);
uint16_t oracle_f32_to_bf16(float f); /* round-to-nearest-even */

/*
 * Offline round-to-nearest weight quantizer: Eq. 6 -> Eq. 7 -> Eq. 8 -> Eq. 9 with no
 * error compensation (the "RTN" row of Table 2).
 *   W        [N][K] fp32 (row = output channel)
 *   symmetric!=0: Eq. 1 symmetric variant (z = 8, codes 1..15); else asymmetric Eq. 8/9.
 *   pow2     !=0: group scales rounded up to a power of two.
 *   per_channel!=0: s_w per row (Eq. 6 "per channel"), else one per tensor.
 * Outputs: codes [N][K/2], gscale [N][K/group] (BF16 bits), gzero [N][K/group], s_w [N or 1].
 * Returns 0, or -1 on bad arguments.
 */
int oracle_quantize_weight_rtn(const float* W, int64_t N, int64_t K, int group, int symmetric,
                               int pow2, int per_channel, uint8_t* codes, uint16_t* gscale,
                               uint8_t* gzero, float* s_w);

/* Eq. 10 / Eq. 14: w8_hat = nearest_Z((u - z_g) * s_g), one rounding.  w8 is [N][K] E4M3 bytes. */
int oracle_dequant_weight(const uint8_t* codes, const uint16_t* gscale, const uint8_t* gzero,
                          int64_t N, int64_t K, int group, uint8_t* w8);

/*
 * Eq. 13 (with Eq. 3): activation FP8 quantization, one scale per token (row).
 *   scale_mode 0: s_x = amax/448 ; 1: s_x = 2^ceil(log2(amax/448)) (power-of-two scales, Sec. 2.2).
 *   static_scale != NULL: the paper's static per-tensor scale is used for every row instead.
 * x is BF16 bits [M][ldx]; outputs x8 [M][ldx8] E4M3 bytes and s_x [M].
 */
int oracle_quantize_act(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, uint8_t* x8,
                        int64_t ldx8, float* s_x, int scale_mode, const float* static_scale);

/*
 * FP8 matmul with the two FP8 dequantization scales (Eq. 4 for activations, Eq. 11 for
 * weights): y[m][n] = s_x[m] * s_w[n*sw_stride] * sum_k x8[m][k] * w8[n][k], in double.
 * cols == NULL: all N columns, outputs are [M][N]; else only the listed columns, outputs
 * are [M][ncols].  Any output pointer may be NULL.
 *   y64  double result; y32 its fp32 rounding; ybf16 BF16(RNE) of y32;
 *   yabs s_x*s_w*sum_k |x8*w8| (for error normalisation).
 */
int oracle_linear(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* w8,
                  const float* s_w, int sw_stride, int64_t N, int64_t K, const int64_t* cols,
                  int64_t ncols, double* y64, float* y32, uint16_t* ybf16, double* yabs);

/* Number of OpenMP threads the linear will use. */
int oracle_num_threads(void);

/* Eq. 10 with a per-column group index (activation-ordered quantization, Table 3 '*' rows):
 * column k takes scale / zero-point of group g_idx[k]; gscale and gzero are [N][G]. */
int oracle_dequant_weight_gidx(const uint8_t* codes, const uint16_t* gscale, const uint8_t* gzero,
                               const int32_t* g_idx, int64_t N, int64_t K, int64_t G, uint8_t* w8);

/*
 * DPQ weight quantizer, Algorithm 1 (Sec. 3.1-3.3, Eq. 6-12) with the Cholesky formulation of the
 * update and Group-Aware Reordering (Sec. 3.2, appendix); see w4a8_dpq_oracle.c for the steps.
 *   W     [N][K] fp32, original column order.
 *   U     [K][K] fp32, upper Cholesky factor of the inverse of the dampened Hessian, rows and
 *         columns in PROCESSING order (only the upper triangle is read).
 *   perm  [K]: processing position p handles original column perm[p] (NULL = identity); every
 *         run of `group` positions must be a permutation of one original group.
 *   mse_steps  0 or 1: Eq. 8 as is; t in 2..11: least-squared-error search over t shrink factors.
 * Outputs in ORIGINAL order: codes [N][K/2], gscale [N][K/group], gzero (asymmetric), s_w.
 * err_out / what_out (optional, [N][K], processing order): the scaled errors e_q and the
 * dequantized weights of Eq. 11, for checks.  Returns 0, or -1 on bad arguments.
 */
int oracle_dpq_quantize(const float* W, int64_t N, int64_t K, int group, const float* U, const int32_t* perm,
                        int symmetric, int mse_steps, int per_channel, uint8_t* codes, uint16_t* gscale,
                        uint8_t* gzero, float* s_w, float* err_out, float* what_out);

#ifdef __cplusplus
}
#endif
#endif
