// Fused W4A8 linear for sm_100a (Sec. 3 inference flow): packed INT4 weight tiles and FP8
// activation tiles arrive by TMA, the weight tile is expanded to E4M3 in shared memory (Eq. 10),
// tcgen05 kind::f8f6f4 MMAs accumulate in tensor memory, and the epilogue applies the Eq. 4 /
// Eq. 11 scales and the BF16 cast (or stores fp32 split-K partials).
//
// Operand roles are swapped with respect to Y = X W^T: the 128 weight rows of a tile are the
// M side of the MMA (one tensor-memory lane per output channel n) and the tokens are its N side
// (BNX columns), so that decode-sized token counts use a narrow MMA instead of a padded one.
//
// CTA = 6 warps: warp 0 issues TMA, warp 1 owns tensor memory and issues the MMAs, warps 2..5
// (one thread per weight row) dequantize and later run the epilogue.
#pragma once

#include <cuda_bf16.h>

#include "w4a8_ptx.cuh"

namespace w4a8 {

// W8_ = true: the weights are FP8 E4M3 bytes already (the W8A8 comparison scheme of Sec. 4.3): the
// TMA tile of 128 rows x 128 bytes lands directly in the swizzled MMA operand, nothing is expanded.
// W16_ = true: the W4A16 comparison scheme of Sec. 4.3: activations stay BF16, the INT4 codes are
// expanded to BF16 (u - z) * s_g, rounded once, and multiplied with kind::f16 MMAs (K = 16 each);
// a k-block of 128 is then two swizzled 128-byte panels of 64 elements per operand.
// GIDX_ = true: weights quantized in an unconstrained activation order (the W4A8* rows of Table 3,
// appendix "Activation Reordering"): column k takes the scale and zero-point of group g_idx[k], so
// no look-up table can be shared by the 128 columns of a k-block -- every weight is expanded by its
// own multiplication and conversion (Eq. 10 element by element), inside the same kernel.
template <int BNX_, int STAGES_, bool W8_ = false, bool W16_ = false, bool GIDX_ = false>
struct UmmaCfg {
    static constexpr bool W8 = W8_;
    static constexpr bool W16 = W16_;
    static constexpr bool GIDX = GIDX_;
    static constexpr int BNX = BNX_;        // tokens per tile (MMA N)
    static constexpr int STAGES = STAGES_;
    static constexpr int BW = 128;          // weight rows per tile (MMA M)
    static constexpr int BK = 128;          // K per pipeline stage = one quantization group
    static constexpr int kWpBytes = BW * BK / 2;   // packed codes
    static constexpr int kW8Bytes = BW * BK * (W16_ ? 2 : 1);   // dequantized E4M3 (BF16)
    static constexpr int kXBytes = BNX * BK * (W16_ ? 2 : 1);   // FP8 (BF16) activations
    static constexpr int kStageBytes = kWpBytes + kW8Bytes + kXBytes;
    static constexpr int kBarBytes = 256;
    static constexpr int kSmemBytes = STAGES * kStageBytes + kBarBytes + 1024;  // + alignment slack
    static constexpr int kTmemCols = BNX < 32 ? 32 : BNX;
    static constexpr int kThreads = 192;
    static_assert(BNX % 16 == 0 && BNX >= 16 && BNX <= 256, "MMA N for M=128");
    static_assert(kStageBytes % 1024 == 0, "stage buffers must stay 1024-byte aligned");
    static_assert((3 * STAGES + 2) * 8 + 8 <= kBarBytes, "barrier area");
};

// p[j] with a run-time j without turning the register array into local memory: a chain of selects.
__device__ __forceinline__ uint32_t p_word(const uint32_t (&p)[16], int j) {
    uint32_t v = p[0];
#pragma unroll
    for (int i = 1; i < 16; ++i) v = (j == i) ? p[i] : v;
    return v;
}

template <class Cfg>
__global__ void __launch_bounds__(Cfg::kThreads)
linear_umma_kernel(const __grid_constant__ CUtensorMap tmap_w,   // codes  u8 [N][K/2], box 64 x 128, 64B swizzle (W8: FP8 u8 [N][K], box 128 x 128, 128B swizzle)
                   const __grid_constant__ CUtensorMap tmap_x,   // X8     u8 [M][K],   box 128 x BNX, 128B swizzle
                   const uint16_t* __restrict__ gscale, const uint8_t* __restrict__ gzero,
                   const int32_t* __restrict__ g_idx,   // GIDX: group of every input column, int32 [K]
                   const float* __restrict__ s_x, const float* __restrict__ s_w, int sw_stride,
                   void* __restrict__ y, int64_t ldy, int out_dtype, float* __restrict__ partial,
                   int M, int N, int K, int kb_per_split, unsigned int* status_word) {
    constexpr int BNX = Cfg::BNX, STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw_addr);

    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + STAGES * Cfg::kStageBytes);
    const uint32_t bars_addr = base + STAGES * Cfg::kStageBytes;
    auto bar_full_tma = [&](int s) { return bars_addr + 8u * (uint32_t)s; };
    auto bar_w8_full = [&](int s) { return bars_addr + 8u * (uint32_t)(STAGES + s); };
    auto bar_mma_done = [&](int s) { return bars_addr + 8u * (uint32_t)(2 * STAGES + s); };
    const uint32_t bar_acc_full = bars_addr + 8u * (uint32_t)(3 * STAGES);
    const uint32_t bar_drain = bars_addr + 8u * (uint32_t)(3 * STAGES + 1);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 3 * STAGES + 2);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    auto stage_wp = [&](int s) { return base + (uint32_t)(s * Cfg::kStageBytes); };
    auto stage_w8 = [&](int s) { return base + (uint32_t)(s * Cfg::kStageBytes + Cfg::kWpBytes); };
    auto stage_x = [&](int s) {
        return base + (uint32_t)(s * Cfg::kStageBytes + Cfg::kWpBytes + Cfg::kW8Bytes);
    };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * Cfg::BW;
    const int m0 = blockIdx.y * BNX;
    const int kb0 = blockIdx.z * kb_per_split;
    const int nkb = kb_per_split;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(bar_full_tma(s), 1);
            ptx::mbar_init(bar_w8_full(s), 128);
            ptx::mbar_init(bar_mma_done(s), 1);
        }
        ptx::mbar_init(bar_acc_full, 1);
        ptx::mbar_init(bar_drain, 1);
        *abort_flag = 0u;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_w);
        ptx::prefetch_tensormap(&tmap_x);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), Cfg::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            for (int it = 0; it < nkb && ok; ++it) {
                const int s = it % STAGES;
                if (it >= STAGES)
                    ok = ptx::mbar_wait(bar_mma_done(s), (uint32_t)((it / STAGES - 1) & 1), abort_flag,
                                        status_word);
                if (!ok) break;
                if (Cfg::W8) {
                    ptx::mbar_arrive_expect_tx(bar_full_tma(s), (uint32_t)(Cfg::kW8Bytes + Cfg::kXBytes));
                    ptx::tma_load_2d(stage_w8(s), &tmap_w, (kb0 + it) * 128, n0, bar_full_tma(s));
                } else {
                    ptx::mbar_arrive_expect_tx(bar_full_tma(s), (uint32_t)(Cfg::kWpBytes + Cfg::kXBytes));
                    ptx::tma_load_2d(stage_wp(s), &tmap_w, (kb0 + it) * 64, n0, bar_full_tma(s));
                }
                if (Cfg::W16) {  // X as bytes: two panels of 64 BF16 values per k-block
                    ptx::tma_load_2d(stage_x(s), &tmap_x, (kb0 + it) * 256, m0, bar_full_tma(s));
                    ptx::tma_load_2d(stage_x(s) + (uint32_t)(BNX * 128), &tmap_x, (kb0 + it) * 256 + 128, m0,
                                     bar_full_tma(s));
                } else {
                    ptx::tma_load_2d(stage_x(s), &tmap_x, (kb0 + it) * 128, m0, bar_full_tma(s));
                }
                issued = it + 1;
            }
            if (!ok) {
                // Gave up: let the copies already in flight land before the CTA goes away.
                for (int it = (issued > STAGES ? issued - STAGES : 0); it < issued; ++it) {
                    uint64_t t0 = ptx::globaltimer_ns();
                    while (!ptx::mbar_try_wait(bar_full_tma(it % STAGES), (uint32_t)((it / STAGES) & 1)) &&
                           ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc =
                Cfg::W16 ? ptx::umma_idesc_bf16_f32(128, BNX) : ptx::umma_idesc_e4m3_f32(128, BNX);
            bool ok = true;
            for (int it = 0; it < nkb && ok; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)((it / STAGES) & 1);
                ok = ptx::mbar_wait(bar_full_tma(s), ph, abort_flag, status_word) &&
                     (Cfg::W8 || ptx::mbar_wait(bar_w8_full(s), ph, abort_flag, status_word));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                if (Cfg::W16) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {  // panel k / 4, K = 16 slice k % 4 (32 bytes each)
                        const uint32_t pa = (uint32_t)((k >> 2) * 128 * 128 + (k & 3) * 32);
                        const uint32_t pb = (uint32_t)((k >> 2) * BNX * 128 + (k & 3) * 32);
                        const uint64_t adesc = ptx::umma_desc_k_sw128(stage_w8(s) + pa);
                        const uint64_t bdesc = ptx::umma_desc_k_sw128(stage_x(s) + pb);
                        ptx::umma_bf16(tmem_base, adesc, bdesc, idesc, (it > 0 || k > 0) ? 1u : 0u);
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t adesc = ptx::umma_desc_k_sw128(stage_w8(s) + 32u * k);
                        const uint64_t bdesc = ptx::umma_desc_k_sw128(stage_x(s) + 32u * k);
                        ptx::umma_f8(tmem_base, adesc, bdesc, idesc, (it > 0 || k > 0) ? 1u : 0u);
                    }
                }
                ptx::umma_commit(bar_mma_done(s));
            }
            if (ok) {
                ptx::umma_commit(bar_acc_full);
            } else {
                // Gave up: wait (bounded) for the MMAs already issued before tensor memory is freed.
                ptx::umma_commit(bar_drain);
                uint64_t t0 = ptx::globaltimer_ns();
                while (!ptx::mbar_try_wait(bar_drain, 0u) && ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ dequant, then epilogue
        const int q = warp & 3;          // tensor-memory lane quarter this warp may access
        const int r = q * 32 + lane;     // weight row within the tile
        const int n = n0 + r;
        const bool row_ok = n < N;
        const int G = K >> 7;
        const uint16_t* sc_ptr = gscale + (int64_t)(row_ok ? n : 0) * G + kb0;
        const uint8_t* z_ptr = gzero ? gzero + (int64_t)(row_ok ? n : 0) * G + kb0 : nullptr;
        const uint32_t sw64 = (uint32_t)((r >> 1) & 3);
        const uint32_t sw128 = (uint32_t)(r & 7);
        uint32_t sc_next = (row_ok && !Cfg::W8 && !Cfg::GIDX) ? (uint32_t)__ldg(sc_ptr) : 0u;
        int z_next = (z_ptr && row_ok && !Cfg::W8 && !Cfg::GIDX) ? (int)__ldg(z_ptr) : 8;
        // GIDX: this row's scales and zero-points of ALL groups (the look-ups below stay in L1)
        const uint16_t* sc_row = gscale + (int64_t)(row_ok ? n : 0) * G;
        const uint8_t* z_row = gzero ? gzero + (int64_t)(row_ok ? n : 0) * G : nullptr;
        bool ok = true;
        for (int it = 0; it < (Cfg::W8 ? 0 : nkb); ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (uint32_t)((it / STAGES) & 1);
            const uint32_t sc_bits = sc_next;
            const float sc = bf16_bits_to_float(sc_next);
            const int z = z_next;
            if (!Cfg::GIDX && it + 1 < nkb && row_ok) {
                sc_next = (uint32_t)__ldg(sc_ptr + it + 1);
                if (z_ptr) z_next = (int)__ldg(z_ptr + it + 1);
            }
            DequantLut lut;
            if (!Cfg::W16 && !Cfg::GIDX) lut.build(sc, z);
            ok = ptx::mbar_wait(bar_full_tma(s), ph, abort_flag, status_word);
            if (!ok) break;
            const uint32_t src = stage_wp(s) + (uint32_t)r * 64u;
            uint32_t p[16];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(p[4 * j]), "=r"(p[4 * j + 1]), "=r"(p[4 * j + 2]), "=r"(p[4 * j + 3])
                             : "r"(src + (((uint32_t)j ^ sw64) << 4)));
            }
            const uint32_t dst = stage_w8(s) + (uint32_t)r * 128u;
            if (Cfg::W16) {
                // BF16 (128 + u) has the bit pattern 0x4300 | u: subtract 128 + z (exact), multiply by the
                // group scale (one rounding).  Word j holds elements 8j .. 8j+7 = one 16-byte chunk.
                const uint32_t off2 = (uint32_t)(0x4300 | z) * 0x00010001u;  // BF16 pair (128 + z, 128 + z)
                const uint32_t sc2 = (sc_bits & 0xFFFFu) * 0x00010001u;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    uint32_t a = (p[j] & 0x000F000Fu) | 0x43004300u;           // elements 0, 4
                    uint32_t b = ((p[j] >> 4) & 0x000F000Fu) | 0x43004300u;    // elements 1, 5
                    uint32_t c = ((p[j] >> 8) & 0x000F000Fu) | 0x43004300u;    // elements 2, 6
                    uint32_t d = ((p[j] >> 12) & 0x000F000Fu) | 0x43004300u;   // elements 3, 7
                    a = bf16x2_sub_mul(a, off2, sc2);
                    b = bf16x2_sub_mul(b, off2, sc2);
                    c = bf16x2_sub_mul(c, off2, sc2);
                    d = bf16x2_sub_mul(d, off2, sc2);
                    const uint32_t o0 = prmt(a, b, 0x5410u), o1 = prmt(c, d, 0x5410u);
                    const uint32_t o2 = prmt(a, b, 0x7632u), o3 = prmt(c, d, 0x7632u);
                    const uint32_t panel = dst + (uint32_t)((j >> 3) * 128 * 128);
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(
                                     panel + ((((uint32_t)j & 7u) ^ sw128) << 4)),
                                 "r"(o0), "r"(o1), "r"(o2), "r"(o3)
                                 : "memory");
                }
            } else if (Cfg::GIDX) {
                // Eq. 10 with the scale and zero-point of group g_idx[k], one weight at a time:
                // word w holds the nibbles of columns 8w .. 8w+7 (even column in the low nibble)
                const int32_t* gi = g_idx + (int64_t)(kb0 + it) * 128;
#pragma unroll 1
                for (int c = 0; c < 8; ++c) {
                    uint32_t o[4];
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const uint32_t word = p_word(p, 2 * c + (h >> 1));
                        uint32_t out = 0;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int col = 16 * c + 4 * h + e;
                            const int g = __ldg(gi + col);
                            const int u = (int)((word >> (4 * ((h & 1) * 4 + e))) & 15u);
                            const int zz = z_row ? (int)__ldg(z_row + g) : 8;
                            const float ss = bf16_bits_to_float((uint32_t)__ldg(sc_row + g));
                            out |= (cvt_e4m3x2(0.0f, __fmul_rn((float)(u - zz), ss)) & 0xFFu) << (8 * e);
                        }
                        o[h] = out;
                    }
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (((uint32_t)c ^ sw128) << 4)),
                                 "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3])
                                 : "memory");
                }
            } else {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint32_t o0, o1, o2, o3;
                    lut.dequant8(p[2 * c], o0, o1);
                    lut.dequant8(p[2 * c + 1], o2, o3);
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (((uint32_t)c ^ sw128) << 4)),
                                 "r"(o0), "r"(o1), "r"(o2), "r"(o3)
                                 : "memory");
                }
            }
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(bar_w8_full(s));
        }
        // Epilogue: accumulator lane = output channel n, column = token.
        if (ok) ok = ptx::mbar_wait(bar_acc_full, 0u, abort_flag, status_word);
        if (ok) {
            ptx::tc_fence_after_sync();
            const float swn = row_ok ? __ldg(s_w + (int64_t)n * sw_stride) : 0.0f;
            const int64_t MN = (int64_t)M * N;
#pragma unroll 1
            for (int c0 = 0; c0 < BNX; c0 += 16) {
                uint32_t v[16];
                ptx::tmem_ld_32x32b_x16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
                ptx::tmem_ld_wait();
                if (m0 + c0 >= M) continue;  // uniform across the warp
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int m = m0 + c0 + j;
                    if (m < M && row_ok) {
                        const float acc = __uint_as_float(v[j]);
                        if (partial != nullptr) {
                            partial[(int64_t)blockIdx.z * MN + (int64_t)m * N + n] = acc;
                        } else {
                            const float res = acc * ((s_x != nullptr ? __ldg(s_x + m) : 1.0f) * swn);  // Eq. 4, Eq. 11
                            if (out_dtype == W4A8_OUT_FP32)
                                reinterpret_cast<float*>(y)[(int64_t)m * ldy + n] = res;
                            else
                                reinterpret_cast<__nv_bfloat16*>(y)[(int64_t)m * ldy + n] =
                                    __float2bfloat16_rn(res);
                        }
                    }
                }
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

}  // namespace w4a8
