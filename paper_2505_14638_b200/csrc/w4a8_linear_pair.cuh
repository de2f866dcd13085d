// W4A8 linear for many tokens on CTA pairs: a thread-block cluster of two CTAs works on one tile
// of 256 output channels x 256 tokens with two-CTA MMAs (tcgen05 cta_group::2).
//
// Why: in the one-CTA persistent kernel every 128 x 256 x 128 step brings 8.4 KB of packed
// weights and 32 KB of FP8 activations into the SM, 640 cycles at the 64 B/clock an SM takes
// from L2 against 512 cycles for its four MMAs, and the 227 KB of shared memory hold only four
// such stages.  In a pair each CTA expands its own 128 weight rows (the A operand and the
// accumulator rows of a two-CTA MMA are split by rows) and loads only HALF of the activation
// tile (the B operand is split by its rows, i.e. tokens): 24.6 KB per step and SM, six stages.
//
// Roles per CTA (26 warps): warp 0 producer (bulk copies of packed weights, TMA tile of this CTA's
// 128 tokens), warp 1 MMA issuer (works in the pair's leader only; both CTAs' warp 1 allocate and
// free tensor memory), warps 2-9 epilogue (this CTA's 128 accumulator rows x 256 tokens), warps
// 10-25 four dequantization groups (Eq. 10 into swizzled shared memory).  Barriers that the
// issuer waits on live in the leader and are arrived on from both CTAs (remote mbarrier arrive,
// TMA completion routed to the leader's barrier); barriers that free ring slots and publish
// accumulators are arrived on in both CTAs by multicast commits.  No load uses cluster multicast.
// Whole tiles only (no split tiles): N % 256 == 0; any M.  Every wait is bounded.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>

#include "w4a8_common.cuh"
#include "w4a8_ptx.cuh"
#include "w4a8_tiled_format.cuh"

namespace w4a8 {

template <int G_, int S1_, int S2_, int FMT_>
struct PairCfg {
    static constexpr int BNX = 256;   // tokens per tile (MMA N); each CTA loads 128 of them
    static constexpr int G = G_;      // dequantization groups of 4 warps
    static constexpr int S1 = S1_;    // ring of TMA stages (packed chunk + activation half tile)
    static constexpr int S2 = S2_;    // ring of dequantized E4M3 weight tiles
    static constexpr int FMT = FMT_;
    static constexpr int kMeta = meta_bytes(FMT);
    static constexpr int kWStage = 9216;
    static constexpr int kXBytes = 128 * 128;
    static constexpr int kStage1 = kWStage + kXBytes;
    static constexpr int kW8Bytes = 128 * 128;
    static constexpr int kBarBytes = 512;
    static constexpr int kSmemBytes = S1 * kStage1 + S2 * kW8Bytes + kBarBytes + 1024;
    static constexpr int kTmemCols = 512;  // two accumulators of 256 columns
    static constexpr int kThreads = 32 * (10 + 4 * G);
    // same ring-depth rule as the one-CTA persistent kernel (barrier parity, skipped phases)
    static_assert(S1 <= 2 * S2, "ring depths");
    // (a group's next "weights landed" wait must find the slot's previous use among the group's own
    // earlier stages: see the persistent one-CTA kernel)
    static_assert(S1_ % G_ == 0, "the ring depth must be a multiple of the number of expansion groups");
    static_assert(kStage1 % 1024 == 0, "alignment of the swizzled tiles");
    static_assert((3 * S1 + 2 * S2 + 5) * 8 + 32 <= kBarBytes, "barrier area");
    static_assert(kSmemBytes <= 232448, "shared memory per CTA");
};

template <class Cfg>
__global__ void __launch_bounds__(Cfg::kThreads)
linear_pair_kernel(const __grid_constant__ CUtensorMap tmap_x,  // X8 u8 [M][K], box 128 x 128, 128B swizzle
                   const uint8_t* __restrict__ wpp, const float* __restrict__ s_x,
                   const float* __restrict__ s_w, int sw_stride, void* __restrict__ y, int64_t ldy, int out_dtype,
                   int M, int N, int K, int TM, int TN2, unsigned int* status_word) {
    constexpr int BNX = Cfg::BNX, G = Cfg::G, S1 = Cfg::S1, S2 = Cfg::S2;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw_addr);

    constexpr int kRing1 = S1 * Cfg::kStage1;
    constexpr int kRing2 = S2 * Cfg::kW8Bytes;
    const uint32_t bars_addr = base + kRing1 + kRing2;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + kRing1 + kRing2);
    auto bar_full = [&](int s) { return bars_addr + 8u * (uint32_t)s; };                      // local: packed weights landed
    auto bar_free1 = [&](int s) { return bars_addr + 8u * (uint32_t)(S1 + s); };               // both: stage consumed
    auto bar_w8_full = [&](int s) { return bars_addr + 8u * (uint32_t)(2 * S1 + s); };         // leader: expanded in both CTAs
    auto bar_free2 = [&](int s) { return bars_addr + 8u * (uint32_t)(2 * S1 + S2 + s); };      // both: expanded tile consumed
    auto bar_acc_full = [&](int b) { return bars_addr + 8u * (uint32_t)(2 * S1 + 2 * S2 + b); };       // both
    auto bar_acc_empty = [&](int b) { return bars_addr + 8u * (uint32_t)(2 * S1 + 2 * S2 + 2 + b); };  // leader
    const uint32_t bar_drain = bars_addr + 8u * (uint32_t)(2 * S1 + 2 * S2 + 4);
    auto bar_xfull = [&](int s) { return bars_addr + 8u * (uint32_t)(2 * S1 + 2 * S2 + 5 + s); };  // leader: both halves landed
    constexpr int kNumBars = 3 * S1 + 2 * S2 + 5;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + kNumBars);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    auto stage_w = [&](int s) { return base + (uint32_t)(s * Cfg::kStage1); };
    auto stage_x = [&](int s) { return base + (uint32_t)(s * Cfg::kStage1 + Cfg::kWStage); };
    auto stage_w8 = [&](int s) { return base + (uint32_t)(kRing1 + s * Cfg::kW8Bytes); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const bool leader = rank == 0;
    const int KB = K >> 7;
    const uint8_t* meta_base = wpp + (int64_t)KB * N * kRowCodeBytes;
    const int C = (int)(gridDim.x >> 1), c = (int)(blockIdx.x >> 1);
    const int Tt = TM * TN2;
    const int n_tiles = c < Tt ? (Tt - c + C - 1) / C : 0;  // tiles c, c + C, ...
    const int n_it = n_tiles * KB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S1; ++s) {
            ptx::mbar_init(bar_full(s), 1);
            ptx::mbar_init(bar_xfull(s), 1);
            ptx::mbar_init(bar_free1(s), 1);
        }
        for (int s = 0; s < S2; ++s) {
            ptx::mbar_init(bar_w8_full(s), 256);
            ptx::mbar_init(bar_free2(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(bar_acc_full(b), 1);
            ptx::mbar_init(bar_acc_empty(b), 512);
        }
        ptx::mbar_init(bar_drain, 1);
        *abort_flag = 0u;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_x);
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), Cfg::kTmemCols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();  // the peer's barriers exist before anything arrives on them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    ptx::griddep_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        bool ok = true;
        ptx::Ring r1, rx;
        int tile = c, kb = 0;
        int xtile = c, xkb = 0;
        const int ahead = n_it < S1 ? n_it : S1;
        int it_x = 0;
        for (int it = 0; it < n_it; ++it) {
            ok = ptx::mbar_wait(bar_free1(r1.idx), r1.phase ^ 1u, abort_flag, status_word);
            if (!ok) break;
            const int nt = (tile / TM) * 2 + (int)rank;  // this CTA's 128-row block
            const int64_t row0 = (int64_t)kb * N + (int64_t)nt * 128;
            const uint32_t full = bar_full(r1.idx), wdst = stage_w(r1.idx);
            const uint8_t* csrc = wpp + row0 * kRowCodeBytes;
            const uint8_t* msrc = meta_base + row0 * Cfg::kMeta;
            constexpr uint32_t cbytes = 128u * kRowCodeBytes, mbytes = 128u * Cfg::kMeta;
            if (ptx::elect_one()) {
                ptx::mbar_arrive_expect_tx(full, cbytes + mbytes);
                ptx::bulk_load(wdst, csrc, cbytes, full);
                ptx::bulk_load(wdst + 8192u, msrc, mbytes, full);
            }
            r1.advance(S1);
            if (++kb == KB) {
                kb = 0;
                tile += C;
            }
            if (it + 1 < ahead) continue;  // still inside the weight-only prologue
            if (it + 1 == ahead) ptx::griddep_wait();
            for (; it_x <= it; ++it_x) {
                const uint32_t xfull_local = bar_xfull(rx.idx), xdst = stage_x(rx.idx);
                const uint32_t xfull_leader = ptx::map_to_cta(xfull_local, 0u);
                const int x0 = xkb * 128, y0 = (xtile % TM) * BNX + (int)rank * 128;
                if (ptx::elect_one()) {
                    if (leader) ptx::mbar_arrive_expect_tx(xfull_local, 2u * (uint32_t)Cfg::kXBytes);
                    ptx::tma_load_2d_pair(xdst, &tmap_x, x0, y0, xfull_leader);
                }
                rx.advance(S1);
                if (++xkb == KB) {
                    xkb = 0;
                    xtile += C;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader only)
        if (leader) {
            constexpr uint32_t idesc = ptx::umma_idesc_e4m3_f32(256, BNX);
            bool ok = true;
            ptx::Ring r1, r2;
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int buf = j & 1;
                if (j >= 2) {
                    ok = ptx::mbar_wait(bar_acc_empty(buf), (uint32_t)(((j >> 1) - 1) & 1), abort_flag, status_word);
                    if (!ok) break;
                }
                const uint32_t tmem_acc = tmem_base + (uint32_t)(buf * BNX);
                uint32_t accumulate = 0;
                for (int i = 0; i < KB; ++i) {
                    ok = ptx::mbar_wait(bar_xfull(r1.idx), r1.phase, abort_flag, status_word);
                    ok = ok && ptx::mbar_wait(bar_w8_full(r2.idx), r2.phase, abort_flag, status_word);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_lo = ptx::umma_desc_lo(stage_w8(r2.idx));
                    const uint32_t b_lo = ptx::umma_desc_lo(stage_x(r1.idx));
                    const uint32_t f1 = bar_free1(r1.idx), f2 = bar_free2(r2.idx);
                    if (ptx::elect_one()) {
                        ptx::umma_f8_kblock_pair(tmem_acc, a_lo, b_lo, idesc, accumulate);
                        ptx::umma_commit_pair(f1);
                        ptx::umma_commit_pair(f2);
                    }
                    accumulate = 1u;
                    r1.advance(S1);
                    r2.advance(S2);
                }
                if (!ok) break;
                if (ptx::elect_one()) ptx::umma_commit_pair(bar_acc_full(buf));
            }
            if (!ok && lane == 0) {
                ptx::umma_commit(bar_drain);
                uint64_t t0 = ptx::globaltimer_ns();
                while (!ptx::mbar_try_wait(bar_drain, 0u) && ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                }
            }
        }
        __syncwarp();
    } else if (warp < 10) {
        // ------------------------------------------------------------------ epilogue (8 warps)
        // This CTA's accumulator rows: lane = output channel, column = token of the 256-token tile.
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        const int r = q * 32 + lane;
        constexpr int kHalfCols = BNX / 2;
        bool ok = true;
        ptx::griddep_wait();  // scales come from, outputs may still be in use by, earlier kernels
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int tile = c + j * C;
            const int nt = (tile / TM) * 2 + (int)rank, mt = tile % TM;
            const int n = nt * 128 + r, m0 = mt * BNX + half * kHalfCols;
            const int buf = j & 1;
            const float swn = __ldg(s_w + (int64_t)n * sw_stride);
            float sx_pre[kHalfCols / 32];
#pragma unroll
            for (int cc = 0; cc < kHalfCols / 32; ++cc)
                sx_pre[cc] = (m0 + cc * 32 + lane < M) ? __ldg(s_x + m0 + cc * 32 + lane) : 0.0f;
            ok = ptx::mbar_wait(bar_acc_full(buf), (uint32_t)((j >> 1) & 1), abort_flag, status_word);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const uint32_t tmem_acc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BNX + half * kHalfCols);
#pragma unroll 1
            for (int c0 = 0; c0 < kHalfCols; c0 += 16) {
                uint32_t v[16];
                ptx::tmem_ld_32x32b_x16(tmem_acc + (uint32_t)c0, v);
                ptx::tmem_ld_wait();
                if (m0 + c0 >= M) continue;  // warp-uniform
                float sx_lane = sx_pre[0];
#pragma unroll
                for (int cc = 1; cc < kHalfCols / 32; ++cc) sx_lane = (c0 >= cc * 32) ? sx_pre[cc] : sx_lane;
                float sx[16];
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) sx[jj] = __shfl_sync(0xFFFFFFFFu, sx_lane, (c0 & 16) + jj);
                if (out_dtype == W4A8_OUT_FP32) {
                    float* yp = reinterpret_cast<float*>(y) + (int64_t)(m0 + c0) * ldy + n;
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj)
                        if (m0 + c0 + jj < M) yp[(int64_t)jj * ldy] = __uint_as_float(v[jj]) * (sx[jj] * swn);
                } else {
                    __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(y) + (int64_t)(m0 + c0) * ldy + n;
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj)
                        if (m0 + c0 + jj < M)
                            yp[(int64_t)jj * ldy] = __float2bfloat16_rn(__uint_as_float(v[jj]) * (sx[jj] * swn));
                }
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive_cluster(ptx::map_to_cta(bar_acc_empty(buf), 0u));
        }
    } else {
        // ------------------------------------------------------------------ dequantization groups
        const int dw = warp - 10;
        const int g = dw >> 2;
        const int r = (dw & 3) * 32 + lane;
        for (int it = g; it < n_it; it += G) {
            const int s1 = it % S1, s2 = it % S2;
            if (!ptx::mbar_wait(bar_full(s1), (uint32_t)((it / S1) & 1), abort_flag, status_word)) break;
            if (it >= S2) {
                if (!ptx::mbar_wait(bar_free2(s2), (uint32_t)((it / S2 - 1) & 1), abort_flag, status_word)) break;
            }
            dequant_row_to_smem<Cfg::FMT>(stage_w(s1) + tiled_row_offset(r),
                                          stage_w(s1) + 8192u + (uint32_t)(r * Cfg::kMeta), r,
                                          stage_w8(s2) + (uint32_t)r * 128u);
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive_cluster(ptx::map_to_cta(bar_w8_full(s2), 0u));
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();  // nothing of the pair touches the other's barriers or tensor memory any more
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, Cfg::kTmemCols);
    }
}

}  // namespace w4a8
