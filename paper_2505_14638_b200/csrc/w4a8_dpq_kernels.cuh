// DPQ weight quantizer on the GPU: Algorithm 1 (Sec. 3.1-3.3, Eq. 6-12) with the Cholesky form of
// the update that Sec. 3.3 takes from GPTQ, the least-squared-error search of the group scale,
// and Group-Aware Reordering (Sec. 3.2 and its appendix).
//
// The rows of W are independent; the columns of a row are quantized one after the other, each
// sending its scaled error e to the columns on its right (Eq. 12): w_v <- fma(-e, U_qv, w_v),
// U = upper Cholesky factor of the inverse Hessian in processing order.  Work is cut the way
// GPTQ cuts it, in blocks of one group (128 columns):
//   dpq_block_kernel     half a warp per row: group scale / zero-point (Eq. 8, optional search),
//                        then the 128 columns in sequence with the updates inside the block;
//                        writes the codes, the group's scale and zero-point and the 128 errors;
//   dpq_trailing_kernel  applies the block's 128 errors to every column to the right of the
//                        block, q ascending -- the same chain of fused multiply-adds, in the same
//                        order, that the column-by-column algorithm performs for that element.
// Every floating-point step that decides an integer is one explicitly rounded fp32 operation
// (__fdiv_rn, __fmul_rn, __fmaf_rn ...: never contracted), and the search compares exact integer
// sums, so the codes do not depend on how the work is spread over threads.
#pragma once

#include <cuda_bf16.h>

#include "w4a8_common.cuh"
#include "w4a8_simple_kernels.cuh"

namespace w4a8 {

// ---- Group-Aware Reordering -----------------------------------------------------------------
// Inside each group the columns go by descending Hessian diagonal, the groups by descending
// maximum diagonal; ties keep the original order.  Ranks are found by counting (exact compares).
__global__ void __launch_bounds__(128)
gar_within_kernel(const float* __restrict__ hdiag, int32_t* __restrict__ within, float* __restrict__ gmax) {
    __shared__ float d[128];
    __shared__ float red[4];
    const int g = blockIdx.x, i = threadIdx.x;
    const float di = hdiag[(int64_t)g * 128 + i];
    d[i] = di;
    __syncthreads();
    int rank = 0;
    for (int j = 0; j < 128; ++j) rank += (d[j] > di || (d[j] == di && j < i)) ? 1 : 0;
    within[(int64_t)g * 128 + rank] = g * 128 + i;
    float m = warp_max(di);
    if ((i & 31) == 0) red[i >> 5] = m;
    __syncthreads();
    if (i == 0) gmax[g] = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
}

__global__ void __launch_bounds__(128)
gar_order_kernel(const int32_t* __restrict__ within, const float* __restrict__ gmax, int G,
                 int32_t* __restrict__ perm) {
    const int g = blockIdx.x;
    const float mg = gmax[g];
    int rank = 0;
    for (int j = 0; j < G; ++j) {
        const float mj = gmax[j];
        rank += (mj > mg || (mj == mg && j < g)) ? 1 : 0;
    }
    perm[(int64_t)rank * 128 + threadIdx.x] = within[(int64_t)g * 128 + threadIdx.x];
}

// work[n][p] = W[n][perm[p]]: the rows in processing order.
__global__ void __launch_bounds__(256)
dpq_gather_kernel(const float* __restrict__ W, const int32_t* __restrict__ perm, int64_t N, int64_t K,
                  float* __restrict__ work) {
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= N * K) return;
    const int64_t n = i / K, p = i - n * K;
    work[i] = W[n * K + (perm ? perm[p] : (int32_t)p)];
}

// ---- Eq. 8 / Eq. 9 / Eq. 10 on one FP8-valued weight ------------------------------------------
struct DpqGroup {
    float s;  // group scale (a BF16 value)
    int z;    // zero-point
};

__device__ __forceinline__ DpqGroup dpq_group_params(float lo, float hi, float amax, float p, int symmetric) {
    DpqGroup g;
    if (symmetric) {
        const float a = __fmul_rn(p, amax);
        g.s = (a > 0.0f) ? __fdiv_rn(a, 7.0f) : 1.0f;
        g.z = 8;
        g.s = __bfloat162float(__float2bfloat16_rn(g.s));
    } else {
        const float l = __fmul_rn(p, lo), h = __fmul_rn(p, hi);
        g.s = (h > l) ? __fdiv_rn(__fsub_rn(h, l), 15.0f) : 1.0f;  // Eq. 8
        g.s = __bfloat162float(__float2bfloat16_rn(g.s));
        const float zf = rintf(__fdiv_rn(-l, g.s));
        g.z = (int)fminf(fmaxf(zf, 0.0f), 15.0f);
    }
    return g;
}

// Returns the code u (Eq. 9); w8hat = nearest_Z((u - z) s), the value inference multiplies with (Eq. 10).
__device__ __forceinline__ int dpq_quant_dequant(float w8, const DpqGroup& g, int symmetric, float& w8hat) {
    int u;
    if (symmetric) {
        const float q = rintf(__fdiv_rn(w8, g.s));
        u = (int)fminf(fmaxf(q, -7.0f), 7.0f) + 8;
    } else {
        const float q = rintf(__fadd_rn(__fdiv_rn(w8, g.s), (float)g.z));
        u = (int)fminf(fmaxf(q, 0.0f), 15.0f);
    }
    w8hat = e4m3_roundtrip(__fmul_rn((float)(u - g.z), g.s));
    return u;
}

__device__ __forceinline__ long long warp_sum_ll(long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Half a warp per row, 32 rows per CTA; block `b` = processing positions [128 b, 128 b + 128).
// The chain of one column (three IEEE divisions, two FP8 conversions) is some seventy dependent
// instructions that every lane executes and only the column's owner needs: with two rows per warp a
// warp instruction carries two of those chains (a warp per row spent its issue slots on them: with
// 28 warps per SM the kernel was bound by issue, not by latency).  Lane l of a half owns positions
// l, l + 16, ..., l + 112 of the block.  The block of U (128 x 128) is staged in shared memory for
// the whole CTA.
constexpr int kDpqRowsPerCta = 32;

__device__ __forceinline__ float half_warp_min(float v) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ float half_warp_max(float v) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ long long half_warp_sum_ll(long long v) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__global__ void __launch_bounds__(16 * kDpqRowsPerCta)
dpq_block_kernel(float* __restrict__ work, const float* __restrict__ U, const int32_t* __restrict__ perm,
                 int64_t N, int64_t K, int b, int symmetric, int mse_steps, int per_channel,
                 const float* __restrict__ s_w, uint8_t* __restrict__ codes, uint16_t* __restrict__ gscale,
                 uint8_t* __restrict__ gzero, float* __restrict__ err) {
    extern __shared__ float u_s[];  // [128][128] block of U, then kDpqRowsPerCta x 128 bytes of code staging
    uint8_t* code_s = reinterpret_cast<uint8_t*>(u_s + 128 * 128);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int half = lane >> 4, sl = lane & 15;
    const int64_t p0 = (int64_t)b * 128;
    for (int i = threadIdx.x; i < 128 * 128; i += 16 * kDpqRowsPerCta) {
        const int q = i >> 7, v = i & 127;
        u_s[i] = (v >= q) ? U[(p0 + q) * K + p0 + v] : 0.0f;
    }
    __syncthreads();
    const int rl = 2 * warp + half;                               // row within the CTA
    const int64_t n_raw = (int64_t)blockIdx.x * kDpqRowsPerCta + rl;
    if ((int64_t)blockIdx.x * kDpqRowsPerCta + 2 * warp >= N) return;   // neither row of the warp exists
    const bool valid = n_raw < N;                                 // (a half without a row repeats the last one and stores nothing)
    const int64_t n = valid ? n_raw : N - 1;
    const int64_t G = K >> 7;
    const float sw = per_channel ? s_w[n] : s_w[0];
    float* wrow = work + n * K + p0;
    float w[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = wrow[sl + 16 * i];

    // Eq. 7 on the group's current weights, then Eq. 8 (once per group)
    float w8[8];
    float lo = 0.0f, hi = 0.0f, amax = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        w8[i] = e4m3_roundtrip(__fdiv_rn(w[i], sw));
        lo = fminf(lo, w8[i]);
        hi = fmaxf(hi, w8[i]);
        amax = fmaxf(amax, fabsf(w8[i]));
    }
    lo = half_warp_min(lo);
    hi = half_warp_max(hi);
    amax = half_warp_max(amax);
    DpqGroup grp = dpq_group_params(lo, hi, amax, 1.0f, symmetric);
    if (mse_steps > 1) {
        // Sec. 3.3: least squared error over the group among shrunk ranges; exact integer sums
        long long best = -1;
        for (int t = 0; t < mse_steps; ++t) {
            const float pt = __fsub_rn(1.0f, __fmul_rn((float)t, 0.02f));
            const DpqGroup gt = dpq_group_params(lo, hi, amax, pt, symmetric);
            long long e2 = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float h;
                (void)dpq_quant_dequant(w8[i], gt, symmetric, h);
                const long long d = (long long)__fmul_rn(__fsub_rn(w8[i], h), 512.0f);
                e2 += d * d;
            }
            e2 = half_warp_sum_ll(e2);
            if (best < 0 || e2 < best) {
                best = e2;
                grp = gt;
            }
        }
    }

    // the 128 columns in sequence; every lane of a half follows the same scalar computation
    const int64_t og = perm ? (int64_t)(perm[p0] >> 7) : (int64_t)b;
    float* erow = err + n * 128;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll 4
        for (int o = 0; o < 16; ++o) {
            const int q = 16 * i + o;
            const float wq = __shfl_sync(0xFFFFFFFFu, w[i], (lane & 16) | o);
            const float wq8 = e4m3_roundtrip(__fdiv_rn(wq, sw));         // Eq. 7
            float h8;
            const int u = dpq_quant_dequant(wq8, grp, symmetric, h8);    // Eq. 9, Eq. 10
            const float h16 = __fmul_rn(h8, sw);                         // Eq. 11
            const float e = __fdiv_rn(__fsub_rn(wq, h16), u_s[q * 128 + q]);
            const float* urow = u_s + q * 128;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int v = sl + 16 * k;
                if (v > q) w[k] = __fmaf_rn(-e, urow[v], w[k]);          // Eq. 12
            }
            if (sl == o && valid) {
                erow[q] = e;
                const int c = perm ? (perm[p0 + q] & 127) : q;  // column inside its original group
                code_s[rl * 128 + c] = (uint8_t)u;
            }
        }
    }
    __syncwarp();
    if (!valid) return;
    // codes of the group, original order, two per byte (even column in the low nibble)
    {
        const uint8_t* cs = code_s + rl * 128 + sl * 8;
        const uint32_t packed = (uint32_t)cs[0] | ((uint32_t)cs[1] << 4) | ((uint32_t)cs[2] << 8) | ((uint32_t)cs[3] << 12) |
                                ((uint32_t)cs[4] << 16) | ((uint32_t)cs[5] << 20) | ((uint32_t)cs[6] << 24) | ((uint32_t)cs[7] << 28);
        *reinterpret_cast<uint32_t*>(codes + n * (K >> 1) + og * 64 + sl * 4) = packed;
    }
    if (sl == 0) {
        gscale[n * G + og] = __bfloat16_as_ushort(__float2bfloat16_rn(grp.s));
        if (gzero) gzero[n * G + og] = (uint8_t)grp.z;
    }
}

// Columns to the right of block b: w[n][v] <- fma(-e[n][q], U[128 b + q][v], w[n][v]), q = 0..127
// in order.  A CTA takes 128 rows x 128 columns, a thread 8 rows x 8 columns (two runs of four
// columns, 64 apart) which it keeps in registers; the errors and the rows of U come through shared
// memory in chunks of 32 values of q, so that one q costs a thread four 16-byte shared loads and 64
// FMAs and a tile of U is fetched once per 128 rows.  (First version: 16 rows x 512 columns per CTA,
// U straight from L2 -- every 16 rows fetched it again, and the L2 traffic, not the FMA pipe, set
// the pace: a fifth to a third of the FMA peak.)  The chain of one element is unchanged: the same
// fused multiply-adds, q ascending.
__global__ void __launch_bounds__(256, 2)
dpq_trailing_kernel(float* __restrict__ work, const float* __restrict__ U, const float* __restrict__ err,
                    int64_t N, int64_t K, int b) {
    __shared__ __align__(16) float e_s[32][132];  // [q][row] = -e (the padding spreads the transposing stores over the banks)
    __shared__ __align__(16) float u_s[32][128];  // [q][column]
    const int64_t p0 = (int64_t)b * 128;
    const int64_t v0 = p0 + 128 + (int64_t)blockIdx.x * 128;   // K is a multiple of 128: the column tile is whole
    const int64_t n0 = (int64_t)blockIdx.y * 128;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t n = n0 + ty * 8 + i;
        float4 a = make_float4(0.0f, 0.0f, 0.0f, 0.0f), c = a;
        if (n < N) {
            a = *reinterpret_cast<const float4*>(work + n * K + v0 + tx * 4);
            c = *reinterpret_cast<const float4*>(work + n * K + v0 + 64 + tx * 4);
        }
        acc[i][0] = a.x; acc[i][1] = a.y; acc[i][2] = a.z; acc[i][3] = a.w;
        acc[i][4] = c.x; acc[i][5] = c.y; acc[i][6] = c.z; acc[i][7] = c.w;
    }
    const float* up = U + p0 * K + v0;
#pragma unroll 1
    for (int qc = 0; qc < 128; qc += 32) {
        if (qc > 0) __syncthreads();   // the previous chunk has been consumed
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int idx = i * 256 + tid;
            const int q = idx & 31, row = idx >> 5;
            e_s[q][row] = (n0 + row < N) ? -err[(n0 + row) * 128 + qc + q] : 0.0f;   // -e, exact
            const int c = idx & 127, qu = idx >> 7;
            u_s[qu][c] = __ldg(up + (int64_t)(qc + qu) * K + c);
        }
        __syncthreads();
#pragma unroll 2
        for (int q = 0; q < 32; ++q) {
            const float4 ea = *reinterpret_cast<const float4*>(&e_s[q][ty * 8]);
            const float4 eb = *reinterpret_cast<const float4*>(&e_s[q][ty * 8 + 4]);
            const float4 ua = *reinterpret_cast<const float4*>(&u_s[q][tx * 4]);
            const float4 ub = *reinterpret_cast<const float4*>(&u_s[q][64 + tx * 4]);
            const float e[8] = {ea.x, ea.y, ea.z, ea.w, eb.x, eb.y, eb.z, eb.w};
            const float u[8] = {ua.x, ua.y, ua.z, ua.w, ub.x, ub.y, ub.z, ub.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = __fmaf_rn(e[i], u[j], acc[i][j]);   // Eq. 12
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t n = n0 + ty * 8 + i;
        if (n < N) {
            *reinterpret_cast<float4*>(work + n * K + v0 + tx * 4) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
            *reinterpret_cast<float4*>(work + n * K + v0 + 64 + tx * 4) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
        }
    }
}


// ---------------------------------------------------------------------------------------------
// The layer Hessian of the quantizer (Sec. 3.1; Sec. 3.3 for its preparation): H = X^T X over the
// calibration tokens.  A plain FP32 contraction on the FMA pipes -- an offline step whose sums
// decide nothing bit-exactly (the factorization that follows is a library matter in float64).
// One CTA per 64 x 64 tile of the upper triangle (tiles below the diagonal are mirrored on the
// way out); 256 threads, 4 x 4 outputs each; the token dimension in slabs of 32 rows staged in
// shared memory as fp32.
// ---------------------------------------------------------------------------------------------
constexpr int kHessTile = 64, kHessSlab = 32;
__global__ void __launch_bounds__(256)
hessian_xtx_kernel(const uint16_t* __restrict__ x, int64_t T, int64_t K, int64_t ldx, float* __restrict__ H,
                   float beta) {
    // tile (bi, bj) with bj >= bi, enumerated row by row of the upper triangle
    const int nb = (int)((K + kHessTile - 1) / kHessTile);
    int bi = 0, rem = (int)blockIdx.x;
    while (rem >= nb - bi) {
        rem -= nb - bi;
        ++bi;
    }
    const int bj = bi + rem;
    __shared__ float a_s[kHessSlab][kHessTile + 1], b_s[kHessSlab][kHessTile + 1];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;   // 16 x 16 threads, 4 x 4 outputs each
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
    for (int64_t t0 = 0; t0 < T; t0 += kHessSlab) {
        // 32 x 64 BF16 values per operand: 2048 values, 8 per thread
        for (int e = (int)threadIdx.x; e < kHessSlab * kHessTile; e += 256) {
            const int r = e / kHessTile, c = e - r * kHessTile;
            const int64_t t = t0 + r;
            const int64_t ca = (int64_t)bi * kHessTile + c, cb = (int64_t)bj * kHessTile + c;
            a_s[r][c] = (t < T && ca < K) ? bf16_bits_to_float((uint32_t)__ldg(x + t * ldx + ca)) : 0.0f;
            b_s[r][c] = (t < T && cb < K) ? bf16_bits_to_float((uint32_t)__ldg(x + t * ldx + cb)) : 0.0f;
        }
        __syncthreads();
#pragma unroll 4
        for (int r = 0; r < kHessSlab; ++r) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) av[i] = a_s[r][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) bv[j] = b_s[r][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t gi = (int64_t)bi * kHessTile + ty * 4 + i, gj = (int64_t)bj * kHessTile + tx * 4 + j;
            if (gi < K && gj < K) {
                const float v = acc[i][j] + (beta != 0.0f ? beta * H[gi * K + gj] : 0.0f);
                H[gi * K + gj] = v;
                if (bi != bj) H[gj * K + gi] = v;   // (a diagonal tile computes both halves itself)
            }
        }
}

// Sec. 3.3 (as in GPTQ): the Hessian in processing order, a unit diagonal for input features that
// never fired, damp * mean(diag) added to the diagonal.  Pass 1: the mean of the diagonal after the
// dead-feature rule (one CTA); pass 2: the permuted copy.
__global__ void __launch_bounds__(256)
hessian_diag_mean_kernel(const float* __restrict__ H, int64_t K, float* __restrict__ mean_out) {
    __shared__ double red[256];
    double s = 0.0;
    for (int64_t k = threadIdx.x; k < K; k += 256) {
        const float d = H[k * K + k];
        s += d == 0.0f ? 1.0 : (double)d;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *mean_out = (float)(red[0] / (double)K);
}
__global__ void __launch_bounds__(256)
hessian_prepare_kernel(const float* __restrict__ H, int64_t K, const int32_t* __restrict__ perm, float damp,
                       const float* __restrict__ mean_diag, float* __restrict__ Hp) {
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (idx >= K * K) return;
    const int64_t i = idx / K, j = idx - i * K;
    const int64_t si = perm ? perm[i] : i, sj = perm ? perm[j] : j;
    float v = H[si * K + sj];
    if (i == j) {
        if (v == 0.0f) v = 1.0f;
        v = __fadd_rn(v, __fmul_rn(damp, *mean_diag));
    }
    Hp[idx] = v;
}

}  // namespace w4a8
