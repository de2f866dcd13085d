// Decode-sized W4A8 linear (M <= 64 tokens) for sm_100a: the weight-bandwidth-bound regime.
//
// The output channels are cut into as many contiguous row ranges as there are SMs (multiples of
// 8 rows, so every SM streams the same share of the packed weights within a few percent); each
// CTA walks the whole K range of its rows: no split along K, no partial sums, no workspace.
// The MMA runs with the tokens on its M side (M = 64, rows beyond the real tokens are ignored)
// and the CTA's weight rows on its N side, which is what lets the row count be any multiple
// of 8.
//
// Per pipeline stage two bulk copies per k-block bring the rows' INT4 codes and their group
// scales [+ zero-points], and one TMA tile load brings the FP8 activations; G groups of four
// warps expand the codes to E4M3 (Eq. 10) into swizzled shared-memory tiles; one thread issues
// the tcgen05 kind::f8f6f4 MMAs; the epilogue applies the Eq. 4 / Eq. 11 scales and the cast.
// The single-thread roles (copy issue, MMA issue) keep running ring positions instead of
// dividing, because one thread executes dependent integer code at only a few cycles per
// instruction and would otherwise set the pace of the whole pipeline.
//
// Launched with programmatic stream serialization: weight loads, which depend on no earlier
// kernel, start before griddepcontrol.wait; activations and outputs are touched after it.
#pragma once

#include <cuda_bf16.h>

#include "w4a8_ptx.cuh"
#include "w4a8_tiled_format.cuh"

namespace w4a8 {

#ifdef W4A8_TIMING
#define SN_T(var) long long var = clock64()
#define SN_ADD(slot, v) sn_acc[(slot) & 3] += (v)
#define SN_FLUSH(slot0) for (int i_ = 0; i_ < 4; ++i_) g_dbg[blockIdx.x * 16 + (slot0) + i_] = sn_acc[i_]
#define SN_DECL long long sn_acc[4] = {0, 0, 0, 0}
#define SN_SET(slot, v) g_dbg[blockIdx.x * 16 + (slot)] = (v)
#else
#define SN_T(var)
#define SN_ADD(slot, v)
#define SN_SET(slot, v)
#define SN_FLUSH(slot0)
#define SN_DECL
#endif

template <int MT_, int G_, int FMT_>
struct SnCfg {
    static constexpr int MT = MT_;     // token rows loaded per k-block (16 or 64)
    static constexpr int G = G_;       // dequantization groups of 4 warps
    static constexpr int FMT = FMT_;
    static constexpr int kS1Max = 16;  // ring of TMA stages (runtime depth <= this)
    static constexpr int kS2Max = 4;   // ring of dequantized weight tiles (runtime depth <= this, <= TMA ring depth)
    static constexpr int kMeta = meta_bytes(FMT);
    static constexpr int kTmemCols = 256;
    static constexpr int kThreads = 32 * (6 + 4 * G);
    static constexpr int kBarBytes = 512;
    static constexpr int kSmemBudget = 200 * 1024;
    static_assert(MT == 16 || MT == 64, "token tile");
    static_assert((3 * kS1Max + kS2Max + 3) * 8 + 16 <= kBarBytes, "barrier area");
};

// Launch-time plan shared by host and device.
struct SnPlan {
    int T;         // number of row ranges (tiles); range t covers 8-row units [t*NU/T, (t+1)*NU/T)
    int KS;        // k-blocks per pipeline stage
    int S1;        // depth of the TMA ring
    int S2;        // depth of the ring of dequantized tiles (<= S1)
    int meta_off;  // offset of the meta pieces inside a packed stage
    int wstage;    // bytes per stage: packed codes + meta
    int xstage;    // bytes per stage: activation tiles
    int w8stage;   // bytes per stage: dequantized tiles
    int smem;      // dynamic shared memory to request
};

template <class Cfg>
__global__ void __launch_bounds__(Cfg::kThreads)
linear_splitn_kernel(const __grid_constant__ CUtensorMap tmap_x,  // X8 u8 [M][K], box 128 x MT, 128B swizzle
                     const uint8_t* __restrict__ wpp, const float* __restrict__ s_x,
                     const float* __restrict__ s_w, int sw_stride, void* __restrict__ y, int64_t ldy,
                     int out_dtype, int vec_ok, int M, int N, int K, const SnPlan plan,
                     unsigned int* status_word) {
    constexpr int MT = Cfg::MT, G = Cfg::G, S2M = Cfg::kS2Max, MB = Cfg::kMeta;
    constexpr int S1M = Cfg::kS1Max;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw_addr);

    const int S1 = plan.S1, S2 = plan.S2, KS = plan.KS, T = plan.T;
    const uint32_t x_ring = base;
    const uint32_t w8_ring = x_ring + (uint32_t)(S1 * plan.xstage);
    const uint32_t w_ring = w8_ring + (uint32_t)(S2 * plan.w8stage);
    const uint32_t bars_off = (uint32_t)(S1 * plan.xstage + S2 * plan.w8stage + S1 * plan.wstage);
    const uint32_t bars_addr = base + bars_off;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + bars_off);
    const uint32_t bar_full0 = bars_addr;                          // [S1M] packed codes + meta landed
    const uint32_t bar_xfull0 = bars_addr + 8u * S1M;              // [S1M] activation tiles landed
    const uint32_t bar_free10 = bars_addr + 8u * (2 * S1M);        // [S1M] stage consumed by the MMAs
    const uint32_t bar_w8_full0 = bars_addr + 8u * (3 * S1M);      // [S2]  dequantized tile written
    const uint32_t bar_acc_full = bars_addr + 8u * (uint32_t)(3 * S1M + S2M);
    const uint32_t bar_acc_empty = bar_acc_full + 8u;
    const uint32_t bar_drain = bar_acc_full + 16u;
    constexpr int kNumBars = 3 * S1M + S2M + 3;
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
        for (int s = 0; s < S2; ++s) {
            ptx::mbar_init(bar_w8_full0 + 8u * s, 128);
        }
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
    if (threadIdx.x == 32) SN_SET(0, clock64());
    ptx::griddep_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
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
                // Weights depend on no earlier kernel: issue a ring's worth of them before
                // waiting for the kernel that produces the activations.
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
                    ptx::mbar_arrive_expect_tx(full, (uint32_t)ks * (cbytes + mbytes));
                    const uint32_t wdst = w_ring + (uint32_t)(r1.idx * plan.wstage);
                    for (int kbl = 0; kbl < ks; ++kbl, ++kb) {
                        ptx::bulk_load(wdst + (uint32_t)kbl * cbytes, cptr, cbytes, full);
                        ptx::bulk_load(wdst + (uint32_t)plan.meta_off + (uint32_t)kbl * mbytes, mptr, mbytes, full);
                        cptr += code_step;
                        mptr += meta_step;
                    }
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
                        ptx::mbar_arrive_expect_tx(xfull, (uint32_t)(ksx * MT * 128));
                        for (int kbl = 0; kbl < ksx; ++kbl, ++xkb)
                            ptx::tma_load_2d(xdst + (uint32_t)(kbl * MT * 128), &tmap_x, xkb * 128, 0, xfull);
                        rx.advance(S1);
                    }
                }
            }
            if (!ok) {
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
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool ok = true;
            SN_DECL;
            ptx::Ring r1, r2;
            uint32_t acc_phase = 0;
            const uint32_t a_lo0 = ptx::umma_desc_lo(x_ring), b_lo0 = ptx::umma_desc_lo(w8_ring);
            const uint32_t a_step = (uint32_t)plan.xstage >> 4, b_step = (uint32_t)plan.w8stage >> 4;
            bool first_tile = true;
            for (int t = p; t < T && ok; t += P) {
                const int u0 = (int)((int64_t)t * NU / T), u1 = (int)((int64_t)(t + 1) * NU / T);
                const int R = (u1 - u0) * 8;
                const uint32_t idesc = ptx::umma_idesc_e4m3_f32(64, R);
                const uint32_t b_kbl = (uint32_t)(R * 128) >> 4;  // next k-block inside a dequantized stage
                if (!first_tile) {
                    ok = ptx::mbar_wait(bar_acc_empty, acc_phase, abort_flag, status_word);
                    acc_phase ^= 1u;
                    if (!ok) break;
                }
                first_tile = false;
                uint32_t accumulate = 0;
                int kb = 0;
                for (int st = 0; st < nst; ++st) {
                    SN_T(tm0);
                    ok = ptx::mbar_wait(bar_xfull0 + 8u * (uint32_t)r1.idx, r1.phase, abort_flag, status_word);
                    SN_T(tm1);
                    ok = ok && ptx::mbar_wait(bar_w8_full0 + 8u * (uint32_t)r2.idx, r2.phase, abort_flag, status_word);
                    SN_T(tm2);
                    SN_ADD(0, tm1 - tm0);
                    SN_ADD(1, tm2 - tm1);
                    if (st == 0) SN_SET(4, tm2);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    uint32_t a_lo = a_lo0 + (uint32_t)r1.idx * a_step;
                    uint32_t b_lo = b_lo0 + (uint32_t)r2.idx * b_step;
                    const int ks = (KB - kb) < KS ? (KB - kb) : KS;
                    for (int kbl = 0; kbl < ks; ++kbl, ++kb) {
                        ptx::umma_f8_lo(tmem_base, a_lo, b_lo, idesc, accumulate);
                        ptx::umma_f8_lo(tmem_base, a_lo + 2u, b_lo + 2u, idesc, 1u);
                        ptx::umma_f8_lo(tmem_base, a_lo + 4u, b_lo + 4u, idesc, 1u);
                        ptx::umma_f8_lo(tmem_base, a_lo + 6u, b_lo + 6u, idesc, 1u);
                        accumulate = 1u;
                        a_lo += (uint32_t)(MT * 128) >> 4;
                        b_lo += b_kbl;
                    }
                    ptx::umma_commit(bar_free10 + 8u * (uint32_t)r1.idx);  // frees the stage and its dequantized tile
                    r1.advance(S1);
                    r2.advance(S2);
                    SN_T(tm3);
                    SN_ADD(2, tm3 - tm2);
                }
                if (!ok) break;
                ptx::umma_commit(bar_acc_full);
                SN_SET(5, clock64());
            }
            SN_FLUSH(8);
            if (!ok) {
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
        // MMA M = 64: token i sits in tensor-memory lane 32*(i/16) + i%16, output channel in the column.
        const int q = warp & 3;
        const int m = q * 16 + lane;
        const bool has_rows = q * 16 < M;  // warp-uniform
        const bool valid = lane < 16 && m < M;
        bool ok = true;
        uint32_t acc_phase = 0;
        float sxm = 0.0f;
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
                if (valid) sxm = __ldg(s_x + m);
                first_tile = false;
            }
            if (has_rows) {
                const float sw0 = __ldg(s_w);
#pragma unroll 1
                for (int c0 = 0; c0 < R; c0 += 8) {
                    uint32_t v[8];
                    ptx::tmem_ld_32x32b_x8(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
                    ptx::tmem_ld_wait();
                    if (valid) {
                        float res[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float swn = sw_stride ? __ldg(s_w + n0 + c0 + j) : sw0;
                            res[j] = __uint_as_float(v[j]) * (sxm * swn);  // Eq. 4, Eq. 11
                        }
                        const int64_t o = (int64_t)m * ldy + n0 + c0;
                        if (out_dtype == W4A8_OUT_FP32) {
                            float* yp = reinterpret_cast<float*>(y) + o;
                            if (vec_ok) {
                                reinterpret_cast<float4*>(yp)[0] = make_float4(res[0], res[1], res[2], res[3]);
                                reinterpret_cast<float4*>(yp)[1] = make_float4(res[4], res[5], res[6], res[7]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 8; ++j) yp[j] = res[j];
                            }
                        } else {
                            __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(y) + o;
                            if (vec_ok) {
                                uint4 pk;
                                __nv_bfloat162 b0 = __floats2bfloat162_rn(res[0], res[1]);
                                __nv_bfloat162 b1 = __floats2bfloat162_rn(res[2], res[3]);
                                __nv_bfloat162 b2 = __floats2bfloat162_rn(res[4], res[5]);
                                __nv_bfloat162 b3 = __floats2bfloat162_rn(res[6], res[7]);
                                pk.x = *reinterpret_cast<uint32_t*>(&b0);
                                pk.y = *reinterpret_cast<uint32_t*>(&b1);
                                pk.z = *reinterpret_cast<uint32_t*>(&b2);
                                pk.w = *reinterpret_cast<uint32_t*>(&b3);
                                *reinterpret_cast<uint4*>(yp) = pk;
                            } else {
#pragma unroll
                                for (int j = 0; j < 8; ++j) yp[j] = __float2bfloat16_rn(res[j]);
                            }
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
        const int tid = (dw & 3) * 32 + lane;
        // Group g handles every G-th stage; its ring positions advance by G per step.  The
        // dequantized tile it writes was last used by the stage S2 steps earlier, whose MMAs
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
        SN_DECL;
        for (int t = p; t < T && ok; t += P) {
            const int u0 = (int)((int64_t)t * NU / T), u1 = (int)((int64_t)(t + 1) * NU / T);
            const int R = (u1 - u0) * 8;
            int st = turn;
            for (; st < nst; st += G) {
                SN_T(td0);
                ok = ptx::mbar_wait(bar_full0 + 8u * (uint32_t)r1.idx, r1.phase, abort_flag, status_word);
                SN_T(td1);
                if (ok && done >= S2)
                    ok = ptx::mbar_wait(bar_free10 + 8u * (uint32_t)rl.idx, rl.phase, abort_flag, status_word);
                SN_T(td2);
                if (!ok) break;
                const int kb = st * KS;
                const int ks = (KB - kb) < KS ? (KB - kb) : KS;
                const int items = ks * R;
                const uint32_t wsrc = w_ring + (uint32_t)(r1.idx * plan.wstage);
                const uint32_t wdst = w8_ring + (uint32_t)(r2.idx * plan.w8stage);
                for (int item = tid; item < items; item += 128) {
                    int row = item;
                    if (KS > 1) row = item % R;
                    dequant_row_to_smem<Cfg::FMT>(wsrc + (uint32_t)(item * kRowCodeBytes),
                                                  wsrc + (uint32_t)(plan.meta_off + item * MB), row,
                                                  wdst + (uint32_t)item * 128u);
                }
                ptx::fence_proxy_async_smem();
                ptx::mbar_arrive(bar_w8_full0 + 8u * (uint32_t)r2.idx);
#ifdef W4A8_TIMING
                SN_ADD(0, td1 - td0);
                SN_ADD(1, td2 - td1);
                SN_ADD(2, clock64() - td2);
#endif
                for (int i = 0; i < G; ++i) {
                    r1.advance(S1);
                    r2.advance(S2);
                    rl.advance(S1);
                }
                done += G;
            }
            turn = st - nst;
        }
#ifdef W4A8_TIMING
        if (dw == 0 && lane == 0) { SN_FLUSH(12); }
#endif
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 32) SN_SET(6, clock64());
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

}  // namespace w4a8
