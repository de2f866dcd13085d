// Decode-sized W4A8 linear (M <= 64 tokens) for sm_100a: the weight-bandwidth-bound regime.
//
// The output channels are cut into as many contiguous row ranges as there are SMs (multiples of
// 8 rows, at most 256, so every SM streams the same share of the packed weights within a few
// percent); each CTA walks the whole K range of its rows: no split along K, no partial sums, no
// workspace.
//
// Data path of one k-block of a CTA's rows:
//   HBM --bulk copy--> shared memory (INT4 codes + group scales [+ zero-points])
//       --one thread per row: look-up-table expansion to E4M3 (Eq. 10) in registers-->
//       tensor memory (tcgen05.st; the dequantized weights never touch shared memory)
//       --tcgen05.mma kind::f8f6f4 with the weights as the A operand read from tensor memory
//         (128 rows per instruction, rows beyond the range are ignored) and the FP8 activations
//         (TMA tile, 16 or 64 tokens) as the B operand from shared memory-->
//       accumulator in tensor memory (lane = output channel, column = token)
//       --epilogue: Eq. 4 / Eq. 11 scales, BF16 cast--> Y.
// Keeping the dequantized operand out of shared memory matters: the MMA would otherwise re-read
// it from there four times per k-block, next to the copies and the dequantizers' own traffic,
// and shared-memory bandwidth, not HBM, would set the pace.
//
// The single-thread roles (copy issue, MMA issue) handle several k-blocks per pipeline stage and
// keep running ring positions instead of dividing: one thread executes dependent integer code at
// only a few cycles per instruction.
//
// Launched with programmatic stream serialization: weight loads, which depend on no earlier
// kernel, start before griddepcontrol.wait; activations and outputs are touched after it.
#pragma once

#include <cuda_bf16.h>

#include "w4a8_ptx.cuh"
#include "w4a8_tiled_format.cuh"

namespace w4a8 {


template <int MT_, int G_, int FMT_>
struct SnCfg {
    static constexpr int MT = MT_;      // tokens per tile = MMA N (16 or 64)
    static constexpr int G = G_;        // dequantization groups of 4 warps
    static constexpr int FMT = FMT_;
    static constexpr int kS1Max = 16;   // ring of TMA stages (runtime depth <= this)
    static constexpr int kS2 = MT_ == 16 ? 3 : 4;  // ring of dequantized stages in tensor memory
    static constexpr int kItems = 2;    // (k-block, 128-row block) pairs per stage
    static constexpr int kMeta = meta_bytes(FMT);
    static constexpr int kTmemCols = MT_ == 16 ? 256 : 512;
    static constexpr int kAStageCols = kItems * 32;        // 128 bytes per row and item
    static constexpr int kDCol = kS2 * kAStageCols;        // accumulators start after the A ring
    static constexpr int kThreads = 32 * (6 + 4 * G);
    static constexpr int kBarBytes = 512;
    // Decode-sized launches (<= 16 tokens) take half an SM each, so that the CTAs of the next
    // kernel in the stream can start -- and prefetch their weights -- while this one finishes.
    static constexpr int kSmemBudget = MT_ == 16 ? 100 * 1024 : 200 * 1024;
    static_assert(MT == 16 || MT == 64, "token tile");
    static_assert(kDCol + 2 * MT <= kTmemCols, "tensor memory columns");
    static_assert((3 * kS1Max + kS2 + 3) * 8 + 16 <= kBarBytes, "barrier area");
};

// Launch-time plan shared by host and device.
struct SnPlan {
    int T;         // number of row ranges (tiles); range t covers 8-row units [t*NU/T, (t+1)*NU/T)
    int MBLK;      // 128-row blocks per range (1 or 2)
    int KS;        // k-blocks per pipeline stage (KS * MBLK == 2)
    int S1;        // depth of the TMA ring (>= kS2)
    int meta_off;  // offset of the meta pieces inside a packed stage
    int wstage;    // bytes per stage: packed codes + meta
    int xstage;    // bytes per stage: activation tiles
    int smem;      // dynamic shared memory to request
};

template <class Cfg>
__global__ void __launch_bounds__(Cfg::kThreads)
linear_splitn_kernel(const __grid_constant__ CUtensorMap tmap_x,  // X8 u8 [M][K], box 128 x MT, 128B swizzle
                     const uint8_t* __restrict__ wpp, const float* __restrict__ s_x,
                     const float* __restrict__ s_w, int sw_stride, void* __restrict__ y, int64_t ldy,
                     int out_dtype, int M, int N, int K, const SnPlan plan, unsigned int* status_word) {
    constexpr int MT = Cfg::MT, G = Cfg::G, S2 = Cfg::kS2, MB = Cfg::kMeta;
    constexpr int S1M = Cfg::kS1Max;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw_addr);

    const int S1 = plan.S1, KS = plan.KS, MBLK = plan.MBLK, T = plan.T;
    const uint32_t x_ring = base;
    const uint32_t w_ring = x_ring + (uint32_t)(S1 * plan.xstage);
    const uint32_t bars_off = (uint32_t)(S1 * (plan.xstage + plan.wstage));
    const uint32_t bars_addr = base + bars_off;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + bars_off);
    const uint32_t bar_full0 = bars_addr;                      // [S1M] packed codes + meta landed
    const uint32_t bar_xfull0 = bars_addr + 8u * S1M;          // [S1M] activation tiles landed
    const uint32_t bar_free10 = bars_addr + 8u * (2 * S1M);    // [S1M] stage consumed by the MMAs
    const uint32_t bar_a_full0 = bars_addr + 8u * (3 * S1M);   // [S2]  dequantized stage written to tensor memory
    const uint32_t bar_acc_full = bars_addr + 8u * (uint32_t)(3 * S1M + S2);
    const uint32_t bar_acc_empty = bar_acc_full + 8u;
    const uint32_t bar_drain = bar_acc_full + 16u;
    constexpr int kNumBars = 3 * S1M + S2 + 3;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + kNumBars);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = K >> 7;
    const int64_t NU = N >> 3;           // the row partition works in units of 8 rows
    const int nst = (KB + KS - 1) / KS;  // stages per tile
    const int P = gridDim.x, p = blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S1; ++s) {
            ptx::mbar_init(bar_full0 + 8u * s, 1);
            ptx::mbar_init(bar_xfull0 + 8u * s, 1);
            ptx::mbar_init(bar_free10 + 8u * s, 1);
        }
        for (int s = 0; s < S2; ++s) ptx::mbar_init(bar_a_full0 + 8u * s, 128);
        ptx::mbar_init(bar_acc_full, 1);
        ptx::mbar_init(bar_acc_empty, 128);
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
    ptx::griddep_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (whole warp, one lane issues)
        {
            bool ok = true;
            bool waited = false;
            ptx::Ring r1;
            int issued = 0;
            const int64_t code_step = (int64_t)N * kRowCodeBytes;  // one k-block further
            const int64_t meta_step = (int64_t)N * MB;
            const uint8_t* meta_base = wpp + (int64_t)KB * code_step;
            for (int t = p; t < T && ok; t += P) {
                const int u0 = (int)((int64_t)t * NU / T), u1 = (int)((int64_t)(t + 1) * NU / T);
                const int R = (u1 - u0) * 8;
                const uint32_t cbytes = (uint32_t)(R * kRowCodeBytes), mbytes = (uint32_t)(R * MB);
                const uint8_t* cptr = wpp + (int64_t)u0 * 8 * kRowCodeBytes;
                const uint8_t* mptr = meta_base + (int64_t)u0 * 8 * MB;
                // Weights depend on no earlier kernel: issue a few stages of them before waiting
                // for the kernel that produces the activations.
                int ahead = S1 < 4 ? S1 : 4;  // must fit in the ring: nothing is consumed before the activations land
                if (nst < ahead) ahead = nst;
                if (waited) ahead = 0;
                int kb = 0, xkb = 0;
                ptx::Ring rx = r1;  // ring position of the next activation load
                for (int st = 0; st < nst; ++st) {
                    const uint32_t full = bar_full0 + 8u * (uint32_t)r1.idx;
                    ok = ptx::mbar_wait(bar_free10 + 8u * (uint32_t)r1.idx, r1.phase ^ 1u, abort_flag, status_word);
                    if (!ok) break;
                    const int ks = (KB - kb) < KS ? (KB - kb) : KS;
                    const uint32_t wdst = w_ring + (uint32_t)(r1.idx * plan.wstage);
                    const uint32_t mdst = wdst + (uint32_t)plan.meta_off;
                    const uint8_t* cptr1 = cptr + code_step;
                    const uint8_t* mptr1 = mptr + meta_step;
                    if (ptx::elect_one()) {
                        ptx::mbar_arrive_expect_tx(full, (uint32_t)ks * (cbytes + mbytes));
                        ptx::bulk_load(wdst, cptr, cbytes, full);
                        ptx::bulk_load(mdst, mptr, mbytes, full);
                        if (ks == 2) {
                            ptx::bulk_load(wdst + cbytes, cptr1, cbytes, full);
                            ptx::bulk_load(mdst + mbytes, mptr1, mbytes, full);
                        }
                    }
                    cptr += code_step * ks;
                    mptr += meta_step * ks;
                    kb += ks;
                    r1.advance(S1);
                    ++issued;
                    if (st + 1 < ahead) continue;  // still inside the weight-only prologue
                    if (!waited) {
                        ptx::griddep_wait();
                        waited = true;
                    }
                    // activation tiles of every stage issued so far
                    while (xkb < kb) {
                        const int ksx = (KB - xkb) < KS ? (KB - xkb) : KS;
                        const uint32_t xdst = x_ring + (uint32_t)(rx.idx * plan.xstage);
                        const uint32_t xfull = bar_xfull0 + 8u * (uint32_t)rx.idx;
                        const int x0 = xkb * 128;
                        if (ptx::elect_one()) {
                            ptx::mbar_arrive_expect_tx(xfull, (uint32_t)(ksx * MT * 128));
                            ptx::tma_load_2d(xdst, &tmap_x, x0, 0, xfull);
                            if (ksx == 2) ptx::tma_load_2d(xdst + (uint32_t)(MT * 128), &tmap_x, x0 + 128, 0, xfull);
                        }
                        xkb += ksx;
                        rx.advance(S1);
                    }
                }
            }
            if (!ok && lane == 0) {
                // Gave up: let the copies already in flight land before the CTA goes away.
                ptx::Ring rb = r1;
                const int n = issued < S1 ? issued : S1;
                for (int i = 0; i < n; ++i) {
                    if (--rb.idx < 0) {
                        rb.idx = S1 - 1;
                        rb.phase ^= 1u;
                    }
                    uint64_t t0 = ptx::globaltimer_ns();
                    while (!ptx::mbar_try_wait(bar_full0 + 8u * (uint32_t)rb.idx, rb.phase) &&
                           ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (whole warp, one lane issues)
        {
            bool ok = true;
            ptx::Ring r1, r2;
            uint32_t acc_phase = 0;
            const uint32_t b_lo0 = ptx::umma_desc_lo(x_ring);
            const uint32_t b_step = (uint32_t)plan.xstage >> 4;
            constexpr uint32_t idesc = ptx::umma_idesc_e4m3_f32(128, MT);
            const uint32_t d0 = tmem_base + (uint32_t)Cfg::kDCol;
            bool first_tile = true;
            for (int t = p; t < T && ok; t += P) {
                if (!first_tile) {
                    ok = ptx::mbar_wait(bar_acc_empty, acc_phase, abort_flag, status_word);
                    acc_phase ^= 1u;
                    if (!ok) break;
                }
                first_tile = false;
                uint32_t accumulate = 0;
                int kb = 0;
                for (int st = 0; st < nst; ++st) {
                    ok = ptx::mbar_wait(bar_xfull0 + 8u * (uint32_t)r1.idx, r1.phase, abort_flag, status_word);
                    ok = ok && ptx::mbar_wait(bar_a_full0 + 8u * (uint32_t)r2.idx, r2.phase, abort_flag, status_word);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    // A stage holds two (k-block, 128-row block) items: either two k-blocks of one
                    // row block or one k-block of two row blocks.
                    const int ks = (KB - kb) < KS ? (KB - kb) : KS;
                    const uint32_t b_lo = b_lo0 + (uint32_t)r1.idx * b_step;
                    const uint32_t a_col = tmem_base + (uint32_t)(r2.idx * Cfg::kAStageCols);
                    const uint32_t free_bar = bar_free10 + 8u * (uint32_t)r1.idx;
                    const bool second = (MBLK == 2) || (ks == 2);
                    const uint32_t b_lo1 = (MBLK == 2) ? b_lo : b_lo + ((uint32_t)(MT * 128) >> 4);
                    const uint32_t d1 = (MBLK == 2) ? d0 + (uint32_t)MT : d0;
                    const uint32_t acc1 = (MBLK == 2) ? accumulate : 1u;
                    if (ptx::elect_one()) {
                        ptx::umma_f8_kblock_ts(d0, a_col, b_lo, idesc, accumulate);
                        if (second) ptx::umma_f8_kblock_ts(d1, a_col + 32u, b_lo1, idesc, acc1);
                        ptx::umma_commit(free_bar);  // frees the stage and its tensor-memory slot
                    }
                    accumulate = 1u;
                    kb += ks;
                    r1.advance(S1);
                    r2.advance(S2);
                }
                if (!ok) break;
                if (ptx::elect_one()) ptx::umma_commit(bar_acc_full);
            }
            if (!ok && lane == 0) {
                // Gave up: wait (bounded) for the MMAs already issued before tensor memory is freed.
                ptx::umma_commit(bar_drain);
                uint64_t t0 = ptx::globaltimer_ns();
                while (!ptx::mbar_try_wait(bar_drain, 0u) && ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                }
            }
        }
        __syncwarp();
    } else if (warp < 6) {
        // ------------------------------------------------------------------ epilogue
        // Accumulator: lane = row of the 128-row block, column = token.
        const int q = warp & 3;
        const int r = q * 32 + lane;
        bool ok = true;
        uint32_t acc_phase = 0;
        bool first_tile = true;
        for (int t = p; t < T && ok; t += P) {
            const int u0 = (int)((int64_t)t * NU / T), u1 = (int)((int64_t)(t + 1) * NU / T);
            const int R = (u1 - u0) * 8;
            const int n0 = u0 * 8;
            ok = ptx::mbar_wait(bar_acc_full, acc_phase, abort_flag, status_word);
            acc_phase ^= 1u;
            if (!ok) break;
            ptx::tc_fence_after_sync();
            if (first_tile) {
                ptx::griddep_wait();  // s_x comes from, and Y may still be read by, earlier kernels
                first_tile = false;
            }
            for (int b = 0; b < MBLK; ++b) {
                const int row = b * 128 + r;
                const bool row_ok = row < R;
                const int n = n0 + row;
                const float swn = row_ok ? __ldg(s_w + (int64_t)n * sw_stride) : 0.0f;
#pragma unroll 1
                for (int c0 = 0; c0 < MT; c0 += 16) {
                    if (c0 >= M) break;  // uniform
                    uint32_t v[16];
                    ptx::tmem_ld_32x32b_x16(
                        tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(Cfg::kDCol + b * MT + c0), v);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int m = c0 + j;
                        if (m < M && row_ok) {
                            const float res = __uint_as_float(v[j]) * (__ldg(s_x + m) * swn);  // Eq. 4, Eq. 11
                            if (out_dtype == W4A8_OUT_FP32)
                                reinterpret_cast<float*>(y)[(int64_t)m * ldy + n] = res;
                            else
                                reinterpret_cast<__nv_bfloat16*>(y)[(int64_t)m * ldy + n] = __float2bfloat16_rn(res);
                        }
                    }
                }
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(bar_acc_empty);
        }
    } else {
        // ------------------------------------------------------------------ dequantization groups
        const int dw = warp - 6;
        const int g = dw >> 2;
        const int q = warp & 3;          // tensor-memory lane quarter this warp may access
        const int r = q * 32 + lane;     // row within a 128-row block
        // Group g handles every G-th stage; its ring positions advance by G per step.  The
        // tensor-memory slot it writes was last read by the stage S2 steps earlier, whose MMAs
        // signal the "stage consumed" barrier of that earlier stage (ring position rl).
        ptx::Ring r1, r2, rl;
        for (int i = 0; i < g; ++i) {
            r1.advance(S1);
            r2.advance(S2);
        }
        for (int i = 0; i < (4 * S1 - S2) % (2 * S1) + g; ++i) rl.advance(S1);  // rl = r1 - S2 modulo two rounds
        int done = g;  // global index of this group's next stage
        int turn = g;  // stages until this group's next turn, counted across tiles
        bool ok = true;
        for (int t = p; t < T && ok; t += P) {
            const int u0 = (int)((int64_t)t * NU / T), u1 = (int)((int64_t)(t + 1) * NU / T);
            const int R = (u1 - u0) * 8;
            int st = turn;
            for (; st < nst; st += G) {
                ok = ptx::mbar_wait(bar_full0 + 8u * (uint32_t)r1.idx, r1.phase, abort_flag, status_word);
                if (ok && done >= S2)
                    ok = ptx::mbar_wait(bar_free10 + 8u * (uint32_t)rl.idx, rl.phase, abort_flag, status_word);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const int kb = st * KS;
                const int ks = (KB - kb) < KS ? (KB - kb) : KS;
                const uint32_t wsrc = w_ring + (uint32_t)(r1.idx * plan.wstage);
                uint32_t a_col = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(r2.idx * Cfg::kAStageCols);
                for (int kbl = 0; kbl < ks; ++kbl) {
                    for (int b = 0; b < MBLK; ++b) {
                        const int row = b * 128 + r;  // row within the range
                        const int item = kbl * R + row;
                        dequant_row_to_tmem<Cfg::FMT>(wsrc + (uint32_t)(item * kRowCodeBytes),
                                                      wsrc + (uint32_t)(plan.meta_off + item * MB), row, row < R, a_col);
                        a_col += 32u;
                    }
                }
                ptx::tmem_st_wait();
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive(bar_a_full0 + 8u * (uint32_t)r2.idx);
                for (int i = 0; i < G; ++i) {
                    r1.advance(S1);
                    r2.advance(S2);
                    rl.advance(S1);
                }
                done += G;
            }
            turn = st - nst;
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
