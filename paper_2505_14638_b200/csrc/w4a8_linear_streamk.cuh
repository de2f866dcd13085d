// Persistent, load-balanced W4A8 linear for sm_100a on the tiled ("prepacked") weight layout.
//
// Work is the flattened space (weight tile of 128 rows, token tile of BNX rows, k-block of 128):
// every CTA takes an equal, contiguous share of it, so the SMs stay evenly loaded whatever the
// layer shape (decode-sized problems have fewer tiles than SMs).  A CTA whose share covers only
// part of a tile's K range stores an fp32 partial tile; the CTA that arrives last at a tile adds
// the partials in a fixed order and applies the Eq. 4 / Eq. 11 scales -- no second kernel, and
// bit-identical results from run to run.
//
// Per k-block one bulk copy brings the tile's packed INT4 codes, BF16 group scales (and
// zero-points) and one TMA tile load brings the FP8 activations.  G groups of four warps expand
// the codes to E4M3 (Eq. 10) into a ring of swizzled shared-memory tiles; one thread issues the
// tcgen05 kind::f8f6f4 MMAs (weights on the M side, tokens on the N side); accumulators are
// double-buffered in tensor memory so the epilogue warps overlap the next tile's main loop.
#pragma once

#include <cuda_bf16.h>

#include "w4a8_ptx.cuh"
#include "w4a8_tiled_format.cuh"

namespace w4a8 {

#ifdef W4A8_TIMING
#define DBG_STAMP(slot) g_dbg[blockIdx.x * 16 + (slot)] = clock64()
#define DBG_ADD(slot, v) g_dbg[blockIdx.x * 16 + (slot)] += (v)
#define DBG_SET(slot, v) g_dbg[blockIdx.x * 16 + (slot)] = (v)
#else
#define DBG_STAMP(slot)
#define DBG_ADD(slot, v)
#define DBG_SET(slot, v)
#endif

template <int BNX_, int G_, int S1_, int S2_, int FMT_>
struct SkCfg {
    static constexpr int BNX = BNX_;   // tokens per tile (MMA N)
    static constexpr int G = G_;       // dequantization groups of 4 warps
    static constexpr int S1 = S1_;     // ring of TMA stages (packed chunk + activation tile)
    static constexpr int S2 = S2_;     // ring of dequantized E4M3 weight tiles
    static constexpr int FMT = FMT_;
    static constexpr int kMeta = meta_bytes(FMT);
    static constexpr int kWStage = 9216;  // 128 rows x (64 code bytes + meta), padded to keep the activation tile 1024-aligned
    static constexpr int kXBytes = BNX * 128;
    static constexpr int kStage1 = kWStage + kXBytes;
    static constexpr int kW8Bytes = 128 * 128;
    static constexpr int kBarBytes = 512;
    static constexpr int kSmemBytes = S1 * kStage1 + S2 * kW8Bytes + kBarBytes + 1024;
    static constexpr int kTmemCols = 2 * BNX < 32 ? 32 : 2 * BNX;
    static constexpr int kThreads = 32 * (6 + 4 * G);
    static constexpr int kSlotFloats = BNX * 128;
    static_assert(BNX == 16 || BNX == 32 || BNX == 64 || BNX == 128 || BNX == 256, "token tile");
    static_assert(kStage1 % 1024 == 0, "alignment of the swizzled tiles");
    static_assert((2 * S1 + 2 * S2 + 5) * 8 + 16 <= kBarBytes, "barrier area");
    static_assert(kSmemBytes <= 232448, "shared memory per CTA");
};

template <class Cfg>
__global__ void __launch_bounds__(Cfg::kThreads)
linear_streamk_kernel(const __grid_constant__ CUtensorMap tmap_x,  // X8 u8 [M][K], box 128 x BNX, 128B swizzle
                      const uint8_t* __restrict__ wpp,             // tiled weights (panels, k-block major)
                      const float* __restrict__ s_x, const float* __restrict__ s_w, int sw_stride,
                      void* __restrict__ y, int64_t ldy, int out_dtype, unsigned int* counters,
                      float* slots, int M, int N, int K, int TM, int TN, unsigned int* status_word) {
    constexpr int BNX = Cfg::BNX, G = Cfg::G, S1 = Cfg::S1, S2 = Cfg::S2;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw_addr);

    constexpr int kRing1 = S1 * Cfg::kStage1;
    constexpr int kRing2 = S2 * Cfg::kW8Bytes;
    const uint32_t bars_addr = base + kRing1 + kRing2;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + kRing1 + kRing2);
    auto bar_full = [&](int s) { return bars_addr + 8u * (uint32_t)s; };
    auto bar_free1 = [&](int s) { return bars_addr + 8u * (uint32_t)(S1 + s); };
    auto bar_w8_full = [&](int s) { return bars_addr + 8u * (uint32_t)(2 * S1 + s); };
    auto bar_free2 = [&](int s) { return bars_addr + 8u * (uint32_t)(2 * S1 + S2 + s); };
    auto bar_acc_full = [&](int b) { return bars_addr + 8u * (uint32_t)(2 * S1 + 2 * S2 + b); };
    auto bar_acc_empty = [&](int b) { return bars_addr + 8u * (uint32_t)(2 * S1 + 2 * S2 + 2 + b); };
    const uint32_t bar_drain = bars_addr + 8u * (uint32_t)(2 * S1 + 2 * S2 + 4);
    constexpr int kNumBars = 2 * S1 + 2 * S2 + 5;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + kNumBars);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile uint32_t* ticket_slot = tmem_slot + 2;

    auto stage_w = [&](int s) { return base + (uint32_t)(s * Cfg::kStage1); };
    auto stage_x = [&](int s) { return base + (uint32_t)(s * Cfg::kStage1 + Cfg::kWStage); };
    auto stage_w8 = [&](int s) { return base + (uint32_t)(kRing1 + s * Cfg::kW8Bytes); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = K >> 7;
    const uint8_t* meta_base = wpp + (int64_t)KB * N * kRowCodeBytes;
    const int64_t U = (int64_t)TM * TN * KB;
    const int64_t P = gridDim.x, p = blockIdx.x;
    const int64_t u_begin = p * U / P, u_end = (p + 1) * U / P;
    const int n_it = (int)(u_end - u_begin);

    if (threadIdx.x == 0) {
        DBG_STAMP(0);
        DBG_SET(15, (long long)ptx::globaltimer_ns());
        for (int s = 0; s < S1; ++s) {
            ptx::mbar_init(bar_full(s), 1);
            ptx::mbar_init(bar_free1(s), 1);
        }
        for (int s = 0; s < S2; ++s) {
            ptx::mbar_init(bar_w8_full(s), 128);
            ptx::mbar_init(bar_free2(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(bar_acc_full(b), 1);
            ptx::mbar_init(bar_acc_empty(b), 128);
        }
        ptx::mbar_init(bar_drain, 1);
        *abort_flag = 0u;
        ptx::fence_mbar_init();
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
    if (threadIdx.x == 0) DBG_STAMP(1);

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            bool ok = true;
            int it = 0, issued = 0;
            int64_t tile = u_begin / KB;
            int kb = (int)(u_begin - tile * KB);
            for (; it < n_it; ++it) {
                const int s = it % S1;
                if (it >= S1) {
                    ok = ptx::mbar_wait(bar_free1(s), (uint32_t)((it / S1 - 1) & 1), abort_flag, status_word);
                    if (!ok) break;
                }
                const int nt = (int)(tile / TM), mt = (int)(tile - (int64_t)nt * TM);
                const int rows = (N - nt * 128) < 128 ? (N - nt * 128) : 128;  // ragged last tile
                const int64_t row0 = (int64_t)kb * N + (int64_t)nt * 128;
                ptx::mbar_arrive_expect_tx(bar_full(s),
                                           (uint32_t)(rows * (kRowCodeBytes + Cfg::kMeta) + Cfg::kXBytes));
                ptx::bulk_load(stage_w(s), wpp + row0 * kRowCodeBytes, (uint32_t)(rows * kRowCodeBytes), bar_full(s));
                ptx::bulk_load(stage_w(s) + 8192u, meta_base + row0 * Cfg::kMeta, (uint32_t)(rows * Cfg::kMeta),
                               bar_full(s));
                ptx::tma_load_2d(stage_x(s), &tmap_x, kb * 128, mt * BNX, bar_full(s));
                issued = it + 1;
                if (++kb == KB) {
                    kb = 0;
                    ++tile;
                }
            }
            if (!ok) {
                for (int i = (issued > S1 ? issued - S1 : 0); i < issued; ++i) {
                    uint64_t t0 = ptx::globaltimer_ns();
                    while (!ptx::mbar_try_wait(bar_full(i % S1), (uint32_t)((i / S1) & 1)) &&
                           ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_e4m3_f32(128, BNX);
            bool ok = true;
            int it = 0, j = 0;
            int64_t u = u_begin;
            while (u < u_end && ok) {
                const int64_t tile = u / KB;
                const int kb0 = (int)(u - tile * KB);
                const int len = (int)((u_end - u) < (int64_t)(KB - kb0) ? (u_end - u) : (int64_t)(KB - kb0));
                const int buf = j & 1;
                if (j >= 2) {
                    ok = ptx::mbar_wait(bar_acc_empty(buf), (uint32_t)(((j >> 1) - 1) & 1), abort_flag, status_word);
                    if (!ok) break;
                }
                const uint32_t tmem_acc = tmem_base + (uint32_t)(buf * BNX);
                for (int i = 0; i < len; ++i, ++it) {
                    const int s1 = it % S1, s2 = it % S2;
                    ok = ptx::mbar_wait(bar_full(s1), (uint32_t)((it / S1) & 1), abort_flag, status_word) &&
                         ptx::mbar_wait(bar_w8_full(s2), (uint32_t)((it / S2) & 1), abort_flag, status_word);
                    if (!ok) break;
                    if (it == 0) DBG_STAMP(2);
                    ptx::tc_fence_after_sync();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t adesc = ptx::umma_desc_k_sw128(stage_w8(s2) + 32u * k);
                        const uint64_t bdesc = ptx::umma_desc_k_sw128(stage_x(s1) + 32u * k);
                        ptx::umma_f8(tmem_acc, adesc, bdesc, idesc, (i > 0 || k > 0) ? 1u : 0u);
                    }
                    ptx::umma_commit(bar_free1(s1));
                    ptx::umma_commit(bar_free2(s2));
                }
                if (!ok) break;
                ptx::umma_commit(bar_acc_full(buf));
                DBG_STAMP(3);
                u += len;
                ++j;
            }
            if (!ok) {
                // Gave up: let the MMAs already issued finish before tensor memory is freed.
                ptx::umma_commit(bar_drain);
                uint64_t t0 = ptx::globaltimer_ns();
                while (!ptx::mbar_try_wait(bar_drain, 0u) && ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                }
            }
        }
        __syncwarp();
    } else if (warp < 6) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;
        const int r = q * 32 + lane;
        bool ok = true;
        int j = 0;
        int64_t u = u_begin;
        while (u < u_end && ok) {
            const int64_t tile = u / KB;
            const int kb0 = (int)(u - tile * KB);
            const int len = (int)((u_end - u) < (int64_t)(KB - kb0) ? (u_end - u) : (int64_t)(KB - kb0));
            const int nt = (int)(tile / TM), mt = (int)(tile - (int64_t)nt * TM);
            const int n = nt * 128 + r, m0 = mt * BNX;
            const bool row_ok = n < N;
            const int buf = j & 1;
            const bool whole = (len == KB);
            const float swn = row_ok ? __ldg(s_w + (int64_t)n * sw_stride) : 0.0f;
            ok = ptx::mbar_wait(bar_acc_full(buf), (uint32_t)((j >> 1) & 1), abort_flag, status_word);
            if (!ok) break;
            if (r == 0) DBG_STAMP(4);
            ptx::tc_fence_after_sync();
            const uint32_t tmem_acc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BNX);
            // The CTA's first segment uses slot 0, a later (necessarily last) one slot 1.
            float* my_slot = slots + ((int64_t)p * 2 + (j == 0 ? 0 : 1)) * Cfg::kSlotFloats;
#pragma unroll 1
            for (int c0 = 0; c0 < BNX; c0 += 16) {
                uint32_t v[16];
                ptx::tmem_ld_32x32b_x16(tmem_acc + (uint32_t)c0, v);
                ptx::tmem_ld_wait();
                if (m0 + c0 >= M) continue;  // warp-uniform
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) {
                    const int m = m0 + c0 + jj;
                    if (m < M && row_ok) {
                        const float acc = __uint_as_float(v[jj]);
                        if (whole) {
                            const float res = acc * (__ldg(s_x + m) * swn);  // Eq. 4, Eq. 11
                            if (out_dtype == W4A8_OUT_FP32)
                                reinterpret_cast<float*>(y)[(int64_t)m * ldy + n] = res;
                            else
                                reinterpret_cast<__nv_bfloat16*>(y)[(int64_t)m * ldy + n] = __float2bfloat16_rn(res);
                        } else {
                            my_slot[(c0 + jj) * 128 + r] = acc;
                        }
                    }
                }
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(bar_acc_empty(buf));
            if (!whole) {
                // Publish the partial tile, then take a ticket; the last of the tile's segments
                // to arrive reduces all of them in ascending CTA order.
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (r == 0) *ticket_slot = atomicAdd(counters + tile, 1u);
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const uint32_t ticket = *ticket_slot;
                const int64_t p_lo = ((tile * KB + 1) * P - 1) / U;
                const int64_t p_hi = (((tile + 1) * KB) * P - 1) / U;
                if (ticket == (uint32_t)(p_hi - p_lo)) {
                    __threadfence();
#pragma unroll 1
                    for (int c0 = 0; c0 < BNX && m0 + c0 < M; c0 += 16) {
                        float acc[16];
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) acc[jj] = 0.0f;
                        for (int64_t qq = p_lo; qq <= p_hi; ++qq) {
                            const int64_t first_tile = (qq * U / P) / KB;
                            const float* sl = slots + (qq * 2 + (tile == first_tile ? 0 : 1)) * Cfg::kSlotFloats;
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj)
                                if (m0 + c0 + jj < M && row_ok) acc[jj] += __ldcg(sl + (c0 + jj) * 128 + r);
                        }
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            const int m = m0 + c0 + jj;
                            if (m < M && row_ok) {
                                const float res = acc[jj] * (__ldg(s_x + m) * swn);  // Eq. 4, Eq. 11
                                if (out_dtype == W4A8_OUT_FP32)
                                    reinterpret_cast<float*>(y)[(int64_t)m * ldy + n] = res;
                                else
                                    reinterpret_cast<__nv_bfloat16*>(y)[(int64_t)m * ldy + n] =
                                        __float2bfloat16_rn(res);
                            }
                        }
                    }
                    if (r == 0) counters[tile] = 0u;  // ready for the next launch
                }
            }
            u += len;
            ++j;
            if (r == 0) DBG_STAMP(5);
        }
    } else {
        // ------------------------------------------------------------------ dequantization groups
        const int dw = warp - 6;
        const int g = dw >> 2;
        const int r = (dw & 3) * 32 + lane;
        for (int it = g; it < n_it; it += G) {
            const int s1 = it % S1, s2 = it % S2;
#ifdef W4A8_TIMING
            long long tq0 = clock64();
#endif
            if (!ptx::mbar_wait(bar_full(s1), (uint32_t)((it / S1) & 1), abort_flag, status_word)) break;
#ifdef W4A8_TIMING
            long long tq1 = clock64();
            if (dw == 0 && lane == 0) DBG_ADD(8, tq1 - tq0);
#endif
#ifdef W4A8_TIMING
            long long tq2 = clock64();
#endif
            if (it >= S2) {
                if (!ptx::mbar_wait(bar_free2(s2), (uint32_t)((it / S2 - 1) & 1), abort_flag, status_word)) break;
            }
#ifdef W4A8_TIMING
            long long tq3 = clock64();
            if (dw == 0 && lane == 0) { DBG_ADD(9, tq2 - tq1); DBG_ADD(10, tq3 - tq2); }
#endif
            dequant_row_to_smem<Cfg::FMT>(stage_w(s1) + (uint32_t)r * 64u,
                                          stage_w(s1) + 8192u + (uint32_t)(r * Cfg::kMeta), r,
                                          stage_w8(s2) + (uint32_t)r * 128u);
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(bar_w8_full(s2));
#ifdef W4A8_TIMING
            if (dw == 0 && lane == 0) DBG_ADD(11, clock64() - tq3);
#endif
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) DBG_STAMP(6);
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
    if (threadIdx.x == 32) { DBG_STAMP(7); DBG_SET(14, (long long)ptx::globaltimer_ns()); }
}

}  // namespace w4a8
