// Persistent, load-balanced W4A8 linear for sm_100a on the tiled ("prepacked") weight layout.
//
// Work is the flattened space (weight tile of 128 rows, token tile of BNX rows, k-block of 128):
// every CTA takes an equal, contiguous share of it, so the SMs stay evenly loaded whatever the
// layer shape (decode-sized problems have fewer tiles than SMs).  A CTA whose share covers only
// part of a tile's K range stores an fp32 partial tile and bumps the tile's arrival counter.  When
// a CTA has finished its whole share it turns to the (at most two) tiles it shares with others:
// it waits (bounded) until all of that tile's partials have arrived and then reduces ITS columns
// of the tile -- contributor i of C takes the i-th slice of the token columns, adds the C partials
// in ascending CTA order, applies the Eq. 4 / Eq. 11 scales and stores the outputs.  The
// reduction is thus spread over all contributors with many independent loads in flight (one CTA
// adding whole partial tiles one after another spent tens of microseconds on L2 round trips), it
// needs no second kernel, and results are bit-identical from run to run.  The waits cannot
// deadlock: publishing a partial never waits for anything, and the grid is no larger than what
// is resident at once.
//
// Per k-block one bulk copy brings the tile's packed INT4 codes, BF16 group scales (and
// zero-points) and one TMA tile load brings the FP8 activations.  G groups of four warps expand
// the codes to E4M3 (Eq. 10) into a ring of swizzled shared-memory tiles; one thread issues the
// tcgen05 kind::f8f6f4 MMAs (weights on the M side, tokens on the N side); accumulators are
// double-buffered in tensor memory so the epilogue warps overlap the next tile's main loop.
//
// RB = 2 (whole tiles only): a tile is 256 weight rows x 256 tokens -- two 128-row blocks against one
// activation tile per k-block, two accumulators of 256 columns (all of tensor memory, so the
// epilogue of a tile no longer overlaps the next tile; the expansion warps, which have nothing to
// expand into meanwhile, help to drain it).  A k-block step then brings 18 KB of packed
// weights + 32 KB of activations for eight MMAs (about 1060 tensor-pipe cycles) instead of 9 + 32 KB
// for four: the activation bytes an SM pulls from L2 per flop are halved, and the SM's L2 port
// (about 64 bytes per clock) no longer sets the pace.  Measured on (2048, 4096, 4096), per CTA:
// 32 steps in 41.9 k cycles, of which the MMA warp waits 2.2 k for the first operands, 2.6 k for
// activation tiles and 3.3 k for expanded weights; the rest is the tensor pipe itself.
#pragma once

#include <cuda_bf16.h>

#include "w4a8_ptx.cuh"
#include "w4a8_tiled_format.cuh"

namespace w4a8 {


// W8 = true (the W8A8 comparison scheme of Sec. 4.3 on this kernel's skeleton): the weights are FP8
// E4M3 bytes [N][K] already; a TMA tile load puts them straight into the ring of swizzled weight
// tiles the MMAs read, the expansion groups have nothing to do.  Whole tiles only.
//
// CL = true (few tiles, at most 128 tokens): the CTAs that share a tile's K range form a thread-block
// cluster and exchange their partial sums through distributed shared memory instead of a workspace in
// global memory.  CTA i of the C takes the i-th slice of the tile's token columns: every CTA writes
// its accumulator into its own ring memory and sends each slice to the owner's ring memory with one
// bulk copy that completes on the owner's barrier -- once the MMAs of every CTA of the cluster have
// completed and all their rings are idle, which a cluster barrier establishes --; the owner adds the
// C partials in ascending rank order, applies the scales and stores the outputs.  No shared memory
// is set aside for the exchange, so the rings can be deep: with eight k-blocks per CTA all of a CTA's
// weights are requested at once.  Against the exchange through L2 -- partial tile out,
// fence, counter, wait, partial tiles back in, each a round trip of a microsecond or more: 7.4 us
// from the last MMA to the end of a (128, 4096, 4096) launch -- the tail of a (32, 4096, 4096)
// launch takes 2.8 us (accumulator complete 0.8, exchange and sum 1.2, closing cluster barrier 0.8).
// At 128 tokens a CTA exchanges 64 KB, which the SM-to-SM network moves in about 2.5 us (some
// 25 bytes per clock and SM): little is gained there.  Needs no workspace.
//
// W16 = true (the W4A16 comparison scheme of Sec. 4.3 on this kernel's skeleton): activations stay
// BF16 (two TMA loads of 64 values per k-block and token tile), the INT4 codes are expanded to BF16
// through a table of the group's eight magnitudes (two 128-byte panels per row and k-block), the
// MMAs are kind::f16 with K = 16, and there is no activation scale.  Sign-magnitude format, whole
// tiles only.
template <int BNX_, int G_, int S1_, int S2_, int FMT_, int RB_ = 1, bool W8_ = false, bool CL_ = false, bool W16_ = false>
struct SkCfg {
    static constexpr bool W8 = W8_;
    static constexpr bool CL = CL_;
    static constexpr bool W16 = W16_;
    static constexpr int BNX = BNX_;   // tokens per tile (MMA N)
    static constexpr int G = G_;       // dequantization groups of 4 warps
    static constexpr int S1 = S1_;     // ring of TMA stages (packed chunk + activation tile)
    static constexpr int S2 = S2_;     // ring of dequantized E4M3 weight tiles
    static constexpr int FMT = FMT_;
    static constexpr int kMeta = meta_bytes(FMT);
    static constexpr int RB = RB_;     // 128-row blocks per tile
    static constexpr int kCodeBytes = RB_ * 8192;   // packed codes of the tile's rows for one k-block
    static constexpr int kWStage = RB_ * 9216;  // rows x (64 code bytes + meta), padded to keep the activation tile 1024-aligned
    static constexpr int kXBytes = BNX * 128 * (W16_ ? 2 : 1);
    static constexpr int kStage1 = kWStage + kXBytes;
    static constexpr int kW8Bytes = RB_ * 128 * 128 * (W16_ ? 2 : 1);   // expanded weights of one k-block: E4M3 (W16: BF16, two panels)
    static constexpr int kBarBytes = 512;
    static constexpr int kSmemBytes = S1 * kStage1 + S2 * kW8Bytes + kBarBytes + 1024;
    static constexpr int kTmemCols = 2 * BNX < 32 ? 32 : 2 * BNX;   // RB = 1: two accumulators (double buffer); RB = 2: one per row block
    static constexpr int kThreads = 32 * (10 + 4 * G);
    static constexpr int kSlotFloats = BNX * 128;
    static_assert(BNX == 16 || BNX == 32 || BNX == 64 || BNX == 128 || BNX == 256, "token tile");
    static_assert(RB_ == 1 || (RB_ == 2 && BNX_ == 256), "two row blocks per tile only with 256-token tiles");
    static_assert(!W8_ || RB_ == 1, "the FP8-weight variant uses one row block per tile");
    static_assert(!W16_ || (RB_ == 1 && !W8_ && !CL_ && FMT_ == kFmtTiledSignMag), "the BF16 variant: one row block, sign-magnitude codes, whole tiles");
    static_assert(!CL_ || (RB_ == 1 && !W8_ && BNX_ <= 128), "the cluster exchange serves one row block and at most 128 tokens");
    // the exchange happens in the ring memory, idle by then in every CTA of the cluster: the CTA's own partial
    // tile (BNX columns x 128 channels, fp32) and behind it the slices it receives (C x ceil(BNX / C) columns)
    static_assert(!CL_ || S1_ * (RB_ * 9216 + BNX_ * 128) + S2_ * RB_ * 16384 >= (2 * BNX_ + 8) * 512, "room for the exchange");
    // A dequantization group handles every G-th stage, so it skips phases of the barriers it
    // waits on, and an mbarrier wait tells phases apart by parity only: the wait for use k of a
    // slot is sound only if use k-1 has completed before it starts.  That holds because a stage's
    // packed weights are requested only after the MMAs S1 stages back have completed (one release
    // per ring slot, weights and activations together): then the MMAs 2*S2 stages back have
    // completed too, provided S1 <= 2*S2.  (Releasing the packed weights right after their
    // expansion, to request them earlier, broke this: with G != S2 a group got two phases ahead of
    // a "slot free" barrier and overwrote an expanded tile still in use; with G == S2 and
    // S1 % G == 0 it was sound but no faster.)
    static_assert(S1 <= 2 * S2, "ring depths: see the comment above");
    // The same parity argument for the "packed weights landed" barriers: a group that has finished
    // stage i next waits for stage i + G in ring slot (i + G) % S1, whose previous use is stage
    // i + G - S1.  That stage must have landed before the wait starts, or the wait passes one phase
    // early and the group expands what is still in the slot.  With S1 a multiple of G it is one of
    // the group's own earlier stages (or stage i itself), which it has seen land.  With S1 = 5 or 6
    // and G = 4 it was another group's stage, issued earlier than stage i but not bound to land
    // earlier: first launches of a process (cold translation caches, latencies all over the
    // place) now and then summed a stale tile into a few outputs -- found when a second launch on
    // the same inputs disagreed with the first.
    static_assert(S1_ % G_ == 0, "the ring depth must be a multiple of the number of expansion groups");
    static_assert(kStage1 % 1024 == 0, "alignment of the swizzled tiles");
    static_assert((3 * S1 + 2 * S2 + 6) * 8 + 32 <= kBarBytes, "barrier area");
    static_assert(kSmemBytes <= 232448, "shared memory per CTA");
};

template <class Cfg>
__global__ void __launch_bounds__(Cfg::kThreads)
linear_streamk_kernel(const __grid_constant__ CUtensorMap tmap_x,  // X8 u8 [M][K], box 128 x BNX, 128B swizzle
                      const __grid_constant__ CUtensorMap tmap_w,  // W8 only: FP8 weights u8 [N][K], box 128 x 128, 128B swizzle
                      const uint8_t* __restrict__ wpp,             // tiled weights (panels, k-block major)
                      const float* __restrict__ s_x, const float* __restrict__ s_w, int sw_stride,
                      void* __restrict__ y, int64_t ldy, int out_dtype, unsigned int* counters,
                      float* slots, int M, int N, int K, int TM, int TN, int aligned, int cl,
                      unsigned int* status_word) {
    constexpr int BNX = Cfg::BNX, G = Cfg::G, S1 = Cfg::S1, S2 = Cfg::S2, RB = Cfg::RB;
    constexpr int TR = 128 * RB;   // weight rows per tile
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
    auto bar_xfull = [&](int s) { return bars_addr + 8u * (uint32_t)(2 * S1 + 2 * S2 + 5 + s); };
    const uint32_t bar_red = bars_addr + 8u * (uint32_t)(3 * S1 + 2 * S2 + 5);   // CL: partial sums of all CTAs of the cluster have arrived
    constexpr int kNumBars = 3 * S1 + 2 * S2 + 6;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + kNumBars);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile uint32_t* share_slot = tmem_slot + 2;  // [3] number of shared tiles and their indices

    auto stage_w = [&](int s) { return base + (uint32_t)(s * Cfg::kStage1); };
    auto stage_x = [&](int s) { return base + (uint32_t)(s * Cfg::kStage1 + Cfg::kWStage); };
    auto stage_w8 = [&](int s) { return base + (uint32_t)(kRing1 + s * Cfg::kW8Bytes); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = K >> 7;
    const uint8_t* meta_base = wpp + (int64_t)KB * N * kRowCodeBytes;
    const int64_t U = (int64_t)TM * TN * KB;
    const int64_t P = gridDim.x, p = blockIdx.x;
    // Share of this CTA: an equal slice of the unit space, or -- when there are enough tiles
    // for whole tiles to balance -- a run of whole tiles (then no partial tile is ever produced).
    const int64_t Tt = (int64_t)TM * TN;
    int64_t u_begin, u_end;
    if constexpr (Cfg::CL) {
        // CTA p is member p % cl of the cluster of tile p / cl and takes that share of the tile's k-blocks
        // (32-bit arithmetic: the 64-bit divisions of the general case cost a good part of a microsecond
        // at the head of a launch that lasts ten)
        const int pi = (int)blockIdx.x, tl = pi / cl, me = pi - tl * cl;
        u_begin = (int64_t)tl * KB + me * KB / cl;
        u_end = (int64_t)tl * KB + (me + 1) * KB / cl;
    } else {
        u_begin = aligned ? (p * Tt / P) * KB : p * U / P;
        u_end = aligned ? ((p + 1) * Tt / P) * KB : (p + 1) * U / P;
    }
    const int n_it = (int)(u_end - u_begin);
    // first tile and k-block of the share
    const int64_t tile_begin = Cfg::CL ? (int64_t)((int)blockIdx.x / cl) : u_begin / KB;
    const int kb_begin = (int)(u_begin - tile_begin * KB);

    if (warp == 0) {
        // barrier i of the area, one lane each; arrival counts: 128 expanding threads on a "weights expanded"
        // barrier (W8: the TMA load), the draining threads on an "accumulator drained" barrier, one elsewhere
        for (int i = lane; i < kNumBars; i += 32) {
            uint32_t count = 1u;
            if (i >= 2 * S1 && i < 2 * S1 + S2) count = Cfg::W8 ? 1u : 128u;
            if (i >= 2 * S1 + 2 * S2 + 2 && i < 2 * S1 + 2 * S2 + 4) count = RB == 2 ? 256u + 128u * G : 256u;   // (RB = 2: the expansion warps drain too)
            ptx::mbar_init(bars_addr + 8u * (uint32_t)i, count);
        }
        if (lane == 0) {
            *abort_flag = 0u;
            ptx::prefetch_tensormap(&tmap_x);
        }
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), Cfg::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    // CL: first cluster barrier = "my MMAs have completed and my rings are idle" (a thread arrives when its role
    // is done: the epilogue threads once the accumulator is complete); it is waited for before the first copy
    // into a peer's rings.  Implies that the peer's barriers are initialized.  A cluster barrier is a hardware
    // wait without a limit: every thread arrives where its role ends, never behind a CTA-wide barrier that the
    // threads waiting for that arrival would have to reach first.
    bool cl_arrived = false, cl_waited = false;
    const uint32_t tmem_base = *tmem_slot;
    // Launched with programmatic stream serialization: the next kernel in the stream may start its
    // set-up and weight prefetch while this one runs; everything that depends on earlier kernels
    // (activations, scales, outputs, workspace) is touched only after griddepcontrol.wait.
    ptx::griddep_launch_dependents();

    // RB = 2: this warp's share of the 32 chunks (2 row blocks x 16 chunks of 16 token columns) of the
    // CTA's j-th tile -- Eq. 4 / Eq. 11 scales, cast, store.  The tile's two accumulators fill tensor
    // memory, so nothing overlaps its epilogue: besides the two epilogue warps of a lane quarter
    // (slots 0 and 1) the quarter's expansion warps (slot 2 + group), which have nothing to expand
    // into until the accumulators are free again, take chunks as well.
    auto drain_wide = [&](int j, int slot) -> bool {
        constexpr int kSlots = 2 + G;
        const int q = warp & 3, r = q * 32 + lane;
        const int64_t tile = tile_begin + j;
        const int nt = (int)(tile / TM), mt = (int)(tile - (int64_t)nt * TM);
        const int m0 = mt * BNX;
        const int n_lo = nt * TR + r, n_hi = n_lo + 128;
        const float swn_lo = n_lo < N ? __ldg(s_w + (int64_t)n_lo * sw_stride) : 0.0f;
        const float swn_hi = n_hi < N ? __ldg(s_w + (int64_t)n_hi * sw_stride) : 0.0f;
        // activation scales of the tile's 256 tokens, one per lane and 32 tokens, fetched before the
        // accumulator is ready and broadcast by shuffles later
        float sx_pre[BNX / 32];
#pragma unroll
        for (int c = 0; c < BNX / 32; ++c) sx_pre[c] = (m0 + c * 32 + lane < M) ? __ldg(s_x + m0 + c * 32 + lane) : 0.0f;
        const bool sx_vec = (reinterpret_cast<uintptr_t>(s_x) & 15u) == 0;
        if (!ptx::mbar_wait(bar_acc_full(0), (uint32_t)(j & 1), abort_flag, status_word)) return false;
        ptx::tc_fence_after_sync();
        const uint32_t tmem_acc0 = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
        for (int ch = slot; ch < 2 * (BNX / 16); ch += kSlots) {
            const int b = ch / (BNX / 16), c0 = (ch - b * (BNX / 16)) * 16;
            uint32_t v[16];
            ptx::tmem_ld_32x32b_x16(tmem_acc0 + (uint32_t)(b * BNX + c0), v);
            const int n = b == 0 ? n_lo : n_hi;
            const float swn = b == 0 ? swn_lo : swn_hi;
            float sx[16];
            if (sx_vec && m0 + c0 + 16 <= M) {
                // the chunk's sixteen activation scales: four 16-byte loads of one address per warp (L1 hits after
                // the first warp) instead of sixteen shuffles; issued while the tensor-memory load is in flight
#pragma unroll
                for (int v4 = 0; v4 < 4; ++v4) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(s_x + m0 + c0) + v4);
                    sx[4 * v4] = t.x;
                    sx[4 * v4 + 1] = t.y;
                    sx[4 * v4 + 2] = t.z;
                    sx[4 * v4 + 3] = t.w;
                }
            } else {
                float sx_lane = sx_pre[0];
#pragma unroll
                for (int c = 1; c < BNX / 32; ++c) sx_lane = (c0 >= c * 32) ? sx_pre[c] : sx_lane;
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) sx[jj] = __shfl_sync(0xFFFFFFFFu, sx_lane, (c0 & 16) + jj);
            }
            ptx::tmem_ld_wait();
            if (m0 + c0 >= M) continue;  // warp-uniform
            if (n < N) {
                if (out_dtype == W4A8_OUT_FP32) {
                    float* yp = reinterpret_cast<float*>(y) + (int64_t)(m0 + c0) * ldy + n;
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj)
                        if (m0 + c0 + jj < M) yp[(int64_t)jj * ldy] = __uint_as_float(v[jj]) * (sx[jj] * swn);
                } else if (m0 + c0 + 16 <= M) {
                    // (the whole chunk inside the problem: no test per token -- the drain is bound by issue slots)
                    __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(y) + (int64_t)(m0 + c0) * ldy + n;
#pragma unroll
                    for (int jj = 0; jj < 16; jj += 2) {
                        // two tokens per multiply (packed FP32 pairs: the same two roundings per value)
                        float sc0, sc1, r0, r1;
                        ptx::mul_f32x2(sx[jj], sx[jj + 1], swn, swn, sc0, sc1);
                        ptx::mul_f32x2(__uint_as_float(v[jj]), __uint_as_float(v[jj + 1]), sc0, sc1, r0, r1);
                        yp[(int64_t)jj * ldy] = __float2bfloat16_rn(r0);
                        yp[(int64_t)(jj + 1) * ldy] = __float2bfloat16_rn(r1);
                    }
                } else {
                    __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(y) + (int64_t)(m0 + c0) * ldy + n;
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj)
                        if (m0 + c0 + jj < M)
                            yp[(int64_t)jj * ldy] = __float2bfloat16_rn(__uint_as_float(v[jj]) * (sx[jj] * swn));
                }
            }
        }
        ptx::tc_fence_before_sync();
        ptx::mbar_arrive(bar_acc_empty(0));
        return true;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (whole warp, one lane issues)
        {
            bool ok = true;
            int issued = 0;
            ptx::Ring r1;
            const int64_t tile = tile_begin;
            int kb = kb_begin;
            int nt = (int)(tile / TM), mt = (int)(tile - (int64_t)nt * TM);
            // Weights depend on no earlier kernel: the first ring-full of packed tiles is requested
            // before waiting for the kernels that produce the activations.
            // (FP8 weights go straight into the operand ring, whose slots are freed by MMAs, and MMAs need
            // activations: the weight-only prologue may not be longer than that ring)
            constexpr int kAhead = Cfg::W8 ? (S2 < S1 ? S2 : S1) : S1;
            const int ahead = n_it < kAhead ? n_it : kAhead;
            // (the activation tiles of the first ring-full are requested by the MMA warp)
            const int nx = n_it < S1 ? n_it : S1;
            ptx::Ring rx;  // ring position of the next activation tile
            int xkb = kb, xmt = mt;
            int it_x = nx;  // activation tiles issued so far
            for (int i = 0; i < nx; ++i) {
                rx.advance(S1);
                if (++xkb == KB) {
                    xkb = 0;
                    if (++xmt == TM) xmt = 0;
                }
            }
            int it0 = 0;
            if constexpr (!Cfg::W8) {
                // The weights-only prologue as straight-line code: every slot is free, nothing to wait
                // for, and the requests of the ring-full go out back to back (as iterations of the
                // general loop below each took some 600 cycles, four times what the requests cost).
#pragma unroll
                for (int i = 0; i < S1; ++i) {
                    if (i < ahead) {
                        const int rows = (N - nt * TR) < TR ? (N - nt * TR) : TR;
                        const int64_t row0 = (int64_t)kb * N + (int64_t)nt * TR;
                        const uint8_t* csrc = wpp + row0 * kRowCodeBytes;
                        const uint8_t* msrc = meta_base + row0 * Cfg::kMeta;
                        const uint32_t cbytes = (uint32_t)(rows * kRowCodeBytes), mbytes = (uint32_t)(rows * Cfg::kMeta);
                        if (ptx::elect_one()) {
                            ptx::mbar_arrive_expect_tx(bar_full(i), cbytes + mbytes);
                            ptx::bulk_load(stage_w(i), csrc, cbytes, bar_full(i));
                            ptx::bulk_load(stage_w(i) + (uint32_t)Cfg::kCodeBytes, msrc, mbytes, bar_full(i));
                        }
                        r1.advance(S1);
                        ++issued;
                        if (++kb == KB) {
                            kb = 0;
                            if (++mt == TM) {
                                mt = 0;
                                ++nt;
                            }
                        }
                    }
                }
                it0 = ahead;
                ptx::griddep_wait();
            }
            for (int it = it0; it < n_it; ++it) {
                ok = ptx::mbar_wait(bar_free1(r1.idx), r1.phase ^ 1u, abort_flag, status_word);
                if (!ok) break;
                // (operands worked out by the whole warp: see elect_one)
                const int rows = (N - nt * TR) < TR ? (N - nt * TR) : TR;  // ragged last tile
                const int64_t row0 = (int64_t)kb * N + (int64_t)nt * TR;
                const uint32_t full = bar_full(r1.idx), wdst = stage_w(r1.idx);
                const uint8_t* csrc = wpp + row0 * kRowCodeBytes;
                const uint8_t* msrc = meta_base + row0 * Cfg::kMeta;
                const uint32_t cbytes = (uint32_t)(rows * kRowCodeBytes), mbytes = (uint32_t)(rows * Cfg::kMeta);
                if constexpr (Cfg::W8) {
                    // FP8 weights: straight into the ring of MMA operand tiles, once the MMAs that read
                    // the slot's previous tile have completed (every stage in turn: no phase is skipped)
                    const int s2 = it % S2;
                    if (it >= S2) {
                        ok = ptx::mbar_wait(bar_free2(s2), (uint32_t)((it / S2 - 1) & 1), abort_flag, status_word);
                        if (!ok) break;
                    }
                    if (ptx::elect_one()) {
                        ptx::mbar_arrive_expect_tx(bar_w8_full(s2), (uint32_t)Cfg::kW8Bytes);
                        ptx::tma_load_2d(stage_w8(s2), &tmap_w, kb * 128, nt * TR, bar_w8_full(s2));
                    }
                } else if (ptx::elect_one()) {
                    ptx::mbar_arrive_expect_tx(full, cbytes + mbytes);
                    ptx::bulk_load(wdst, csrc, cbytes, full);
                    ptx::bulk_load(wdst + (uint32_t)Cfg::kCodeBytes, msrc, mbytes, full);
                }
                r1.advance(S1);
                ++issued;
                if (++kb == KB) {
                    kb = 0;
                    if (++mt == TM) {
                        mt = 0;
                        ++nt;
                    }
                }
                if (it + 1 < ahead) continue;  // still inside the weight-only prologue
                if (it + 1 == ahead) ptx::griddep_wait();
                // activation tiles of every stage whose weights have been requested
                for (; it_x <= it; ++it_x) {
                    const uint32_t xfull = bar_xfull(rx.idx), xdst = stage_x(rx.idx);
                    const int x0 = xkb * (Cfg::W16 ? 256 : 128), y0 = xmt * BNX;   // (W16: X as bytes, 256 per k-block)
                    if (ptx::elect_one()) {
                        ptx::mbar_arrive_expect_tx(xfull, (uint32_t)Cfg::kXBytes);
                        ptx::tma_load_2d(xdst, &tmap_x, x0, y0, xfull);
                        if constexpr (Cfg::W16) ptx::tma_load_2d(xdst + (uint32_t)(BNX * 128), &tmap_x, x0 + 128, y0, xfull);
                    }
                    rx.advance(S1);
                    if (++xkb == KB) {
                        xkb = 0;
                        if (++xmt == TM) xmt = 0;
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
                    if constexpr (Cfg::W8) {
                        // (the FP8 tile of stage `st` went to slot st % S2 of the operand ring)
                        const int st = issued - 1 - i;
                        if (st >= issued - S2)
                            while (!ptx::mbar_try_wait(bar_w8_full(st % S2), (uint32_t)((st / S2) & 1)) &&
                                   ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                            }
                    } else {
                        while (!ptx::mbar_try_wait(bar_full(rb.idx), rb.phase) &&
                               ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                        }
                    }
                    const bool x_issued = issued - 1 - i < it_x;  // this stage's activation tile was requested too
                    while (x_issued && !ptx::mbar_try_wait(bar_xfull(rb.idx), rb.phase) &&
                           ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                    }
                }
            }
        }
        __syncwarp();
        if constexpr (Cfg::CL) {
            ptx::cluster_arrive();
            cl_arrived = true;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (whole warp, one lane issues)
        {
            constexpr uint32_t idesc = Cfg::W16 ? ptx::umma_idesc_bf16_f32(128, BNX) : ptx::umma_idesc_e4m3_f32(128, BNX);
            bool ok = true;
            ptx::Ring r1, r2;
            int j = 0;
            int64_t u = u_begin;
            {
                // The activation tiles of the first ring-full (every slot is free): requested here, while
                // the producer warp requests the weights -- one lane after the other, the first
                // activation tile went out only after the last of those, a microsecond late.
                ptx::griddep_wait();
                int xkb = kb_begin, xmt = (int)(tile_begin % TM);
                for (int i = 0; i < n_it && i < S1; ++i) {
                    if (ptx::elect_one()) {
                        ptx::mbar_arrive_expect_tx(bar_xfull(i), (uint32_t)Cfg::kXBytes);
                        ptx::tma_load_2d(stage_x(i), &tmap_x, xkb * (Cfg::W16 ? 256 : 128), xmt * BNX, bar_xfull(i));
                        if constexpr (Cfg::W16)
                            ptx::tma_load_2d(stage_x(i) + (uint32_t)(BNX * 128), &tmap_x, xkb * 256 + 128, xmt * BNX, bar_xfull(i));
                    }
                    if (++xkb == KB) {
                        xkb = 0;
                        if (++xmt == TM) xmt = 0;
                    }
                }
            }
            while (u < u_end && ok) {
                const int64_t tile = u / KB;
                const int kb0 = (int)(u - tile * KB);
                const int len = (int)((u_end - u) < (int64_t)(KB - kb0) ? (u_end - u) : (int64_t)(KB - kb0));
                // RB = 1: two accumulators used in turn; RB = 2: both belong to the one tile in flight
                const int buf = RB == 1 ? (j & 1) : 0;
                if (RB == 1 ? j >= 2 : j >= 1) {
                    const uint32_t par = RB == 1 ? (uint32_t)(((j >> 1) - 1) & 1) : (uint32_t)((j - 1) & 1);
                    ok = ptx::mbar_wait(bar_acc_empty(buf), par, abort_flag, status_word);
                    if (!ok) break;
                }
                const uint32_t tmem_acc = tmem_base + (uint32_t)(buf * BNX);
                uint32_t accumulate = 0;
                for (int i = 0; i < len; ++i) {
                    ok = ptx::mbar_wait(bar_xfull(r1.idx), r1.phase, abort_flag, status_word);
                    ok = ok && ptx::mbar_wait(bar_w8_full(r2.idx), r2.phase, abort_flag, status_word);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_lo = ptx::umma_desc_lo(stage_w8(r2.idx));
                    const uint32_t b_lo = ptx::umma_desc_lo(stage_x(r1.idx));
                    const uint32_t f1 = bar_free1(r1.idx), f2 = bar_free2(r2.idx);
                    if constexpr (Cfg::W16) {
                        if (ptx::elect_one()) {
                            // two panels of 64 BF16 values, four K = 16 slices (32 bytes) each
#pragma unroll
                            for (int k = 0; k < 8; ++k)
                                ptx::umma_bf16_lo(tmem_acc, a_lo + (uint32_t)((k >> 2) * (16384 >> 4) + (k & 3) * 2),
                                                  b_lo + (uint32_t)((k >> 2) * ((BNX * 128) >> 4) + (k & 3) * 2), idesc,
                                                  (accumulate | (uint32_t)k) != 0u ? 1u : 0u);
                            ptx::umma_commit(f1);
                            ptx::umma_commit(f2);
                        }
                    } else if (ptx::elect_one()) {
                        ptx::umma_f8_kblock(tmem_acc, a_lo, b_lo, idesc, accumulate);
                        if (RB == 2) ptx::umma_f8_kblock(tmem_acc + (uint32_t)BNX, a_lo + (16384u >> 4), b_lo, idesc, accumulate);
                        ptx::umma_commit(f1);
                        ptx::umma_commit(f2);
                    }
                    accumulate = 1u;
                    r1.advance(S1);
                    r2.advance(S2);
                }
                if (!ok) break;
                if (ptx::elect_one()) ptx::umma_commit(bar_acc_full(buf));
                u += len;
                ++j;
            }
            if (!ok && lane == 0) {
                // Gave up: let the MMAs already issued finish before tensor memory is freed.
                ptx::umma_commit(bar_drain);
                uint64_t t0 = ptx::globaltimer_ns();
                while (!ptx::mbar_try_wait(bar_drain, 0u) && ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {
                }
            }
        }
        __syncwarp();
        if constexpr (Cfg::CL) {
            ptx::cluster_arrive();
            cl_arrived = true;
        }
    } else if (warp < 10) {
        // ------------------------------------------------------------------ epilogue (8 warps)
        // Accumulator: lane = output channel of the tile, column = token.  Two warps share each
        // lane quarter and split the columns.
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        const int r = q * 32 + lane;
        const bool leader = (warp == 2 && lane == 0);
        constexpr int kHalfCols = BNX / 2;
        bool ok = true;
        int j = 0;
        int64_t u = u_begin;
        ptx::griddep_wait();  // scales come from, outputs and workspace may still be in use by, earlier kernels
        // Final value of one output: Eq. 4 / Eq. 11 scales and the cast.
        auto store_out = [&](int m, int n, float acc, float scale) {
            const float res = acc * scale;
            if (out_dtype == W4A8_OUT_FP32)
                reinterpret_cast<float*>(y)[(int64_t)m * ldy + n] = res;
            else
                reinterpret_cast<__nv_bfloat16*>(y)[(int64_t)m * ldy + n] = __float2bfloat16_rn(res);
        };
        int64_t shared_tile0 = 0, shared_tile1 = 0;  // tiles of which this CTA holds a partial (first and last segment)
        int n_shared = 0;
        if constexpr (RB == 2) {
            // whole tiles only: this warp's chunks of every tile of the CTA
            for (; u < u_end && ok; u += KB, ++j) ok = drain_wide(j, half);
        }
        // (RB = 2 is through; its instantiation does not carry the code below)
        if constexpr (RB == 1)
        while (u < u_end && ok) {
            const int64_t tile = u / KB;
            const int kb0 = (int)(u - tile * KB);
            const int len = (int)((u_end - u) < (int64_t)(KB - kb0) ? (u_end - u) : (int64_t)(KB - kb0));
            const int nt = (int)(tile / TM), mt = (int)(tile - (int64_t)nt * TM);
            const int m0 = mt * BNX + half * kHalfCols;
            const int buf = RB == 1 ? (j & 1) : 0;
            const bool whole = (len == KB);
            float swn_rb[RB];
#pragma unroll
            for (int b = 0; b < RB; ++b)
                swn_rb[b] = (nt * TR + b * 128 + r < N) ? __ldg(s_w + (int64_t)(nt * TR + b * 128 + r) * sw_stride) : 0.0f;
            // Activation scales of this warp's columns, one per lane and 32 columns, fetched before
            // the accumulator is ready and broadcast by shuffles later: global loads issued inside
            // the store loop queue behind the operand traffic of the main loop.
            float sx_pre[kHalfCols / 32];
#pragma unroll
            for (int c = 0; c < kHalfCols / 32; ++c)
                sx_pre[c] = Cfg::W16 ? 1.0f : ((m0 + c * 32 + lane < M) ? __ldg(s_x + m0 + c * 32 + lane) : 0.0f);   // (W16: no activation scale)
            ok = ptx::mbar_wait(bar_acc_full(buf), RB == 1 ? (uint32_t)((j >> 1) & 1) : (uint32_t)(j & 1), abort_flag, status_word);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const uint32_t tmem_acc0 =
                tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BNX + half * kHalfCols);
            // The CTA's first segment uses slot 0, a later (necessarily last) one slot 1.
            float* my_slot = slots + ((int64_t)p * 2 + (j == 0 ? 0 : 1)) * Cfg::kSlotFloats +
                             (int64_t)half * kHalfCols * 128;
            if constexpr (Cfg::CL) {
                if (!whole) {
                    // ---- exchange inside the cluster ----
                    ptx::cluster_arrive();
                    cl_arrived = true;
                    const uint32_t red_local = base + (uint32_t)(BNX * 512);   // [source rank][column of my slice][128 channels]
                    const int me = (int)ptx::cluster_ctarank();
                    const int ncol = (M - mt * BNX) < BNX ? (M - mt * BNX) : BNX;   // valid token columns of the tile
                    const int w = (ncol + cl - 1) / cl;                             // columns per slice
                    int wn = ncol - me * w;                                         // valid columns of my slice
                    wn = wn < 0 ? 0 : (wn > w ? w : wn);
                    if (leader) ptx::mbar_arrive_expect_tx(bar_red, (uint32_t)(cl * wn * 512));
                    // this thread's outputs as the owner of slice `me`: channels c4 .. c4 + 3 of the slice's
                    // columns te / 32, te / 32 + 8, ...; their scales are fetched before the wait
                    const int te = (warp - 2) * 32 + lane, c4 = (te & 31) * 4;
                    const int n4 = nt * 128 + c4;
                    float sw4[4], sxp[8];
#pragma unroll
                    for (int i = 0; i < 4; ++i) sw4[i] = (n4 + i < N) ? __ldg(s_w + (int64_t)(n4 + i) * sw_stride) : 0.0f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int tl = (te >> 5) + 8 * k;
                        sxp[k] = tl < wn ? __ldg(s_x + mt * BNX + me * w + tl) : 0.0f;
                    }
                    // accumulator -> this CTA's own ring memory (idle: the tile's MMAs have completed), as
                    // [column][128 channels]: the slice of owner d is one contiguous piece
                    const int t0 = half * kHalfCols;
#pragma unroll 1
                    for (int c0 = 0; c0 < kHalfCols; c0 += 16) {
                        uint32_t v[16];
                        ptx::tmem_ld_32x32b_x16(tmem_acc0 + (uint32_t)c0, v);
                        ptx::tmem_ld_wait();
                        if (t0 + c0 >= ncol) break;  // warp-uniform
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj)
                            asm volatile("st.shared.u32 [%0], %1;" ::"r"(base + (uint32_t)(((t0 + c0 + jj) * 128 + r) * 4)), "r"(v[jj])
                                         : "memory");
                    }
                    ptx::tc_fence_before_sync();
                    ptx::mbar_arrive(bar_acc_empty(buf));
                    ptx::fence_proxy_async_smem();
                    ptx::cluster_wait();   // the rings of every CTA of the cluster are idle
                    cl_waited = true;
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                    if (te < cl) {
                        // one bulk copy per owner: my partial sums of its slice into its staging area,
                        // completion counted on its barrier
                        int cols = ncol - te * w;
                        cols = cols < 0 ? 0 : (cols > w ? w : cols);
                        if (cols > 0)
                            ptx::bulk_copy_to_cta(ptx::map_to_cta(red_local + (uint32_t)(me * w * 512), (uint32_t)te),
                                                  base + (uint32_t)(te * w * 512), (uint32_t)(cols * 512),
                                                  ptx::map_to_cta(bar_red, (uint32_t)te));
                    }
                    ok = ptx::mbar_wait(bar_red, 0u, abort_flag, status_word);
                    if (!ok) break;
                    const bool vec_ok = (ldy & 3) == 0;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int tl = (te >> 5) + 8 * k;
                        if (tl >= wn) break;
                        float a0 = 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;
                        for (int sr = 0; sr < cl; ++sr) {   // ascending rank order: the same sum on every launch
                            float4 pv;
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                         : "=f"(pv.x), "=f"(pv.y), "=f"(pv.z), "=f"(pv.w)
                                         : "r"(red_local + (uint32_t)(((sr * w + tl) * 128 + c4) * 4)));
                            a0 += pv.x;
                            a1 += pv.y;
                            a2 += pv.z;
                            a3 += pv.w;
                        }
                        if (n4 >= N) continue;
                        const int m = mt * BNX + me * w + tl;
                        const float sxm = sxp[k];
                        const float r0 = a0 * (sxm * sw4[0]), r1 = a1 * (sxm * sw4[1]), r2 = a2 * (sxm * sw4[2]),
                                    r3 = a3 * (sxm * sw4[3]);
                        if (out_dtype == W4A8_OUT_FP32) {
                            float* yp = reinterpret_cast<float*>(y) + (int64_t)m * ldy + n4;
                            if (vec_ok) {
                                *reinterpret_cast<float4*>(yp) = make_float4(r0, r1, r2, r3);
                            } else {
                                yp[0] = r0;
                                yp[1] = r1;
                                yp[2] = r2;
                                yp[3] = r3;
                            }
                        } else {
                            __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(y) + (int64_t)m * ldy + n4;
                            if (vec_ok) {
                                const __nv_bfloat162 lo = __floats2bfloat162_rn(r0, r1), hi = __floats2bfloat162_rn(r2, r3);
                                uint2 pk;
                                pk.x = *reinterpret_cast<const uint32_t*>(&lo);
                                pk.y = *reinterpret_cast<const uint32_t*>(&hi);
                                *reinterpret_cast<uint2*>(yp) = pk;
                            } else {
                                yp[0] = __float2bfloat16_rn(r0);
                                yp[1] = __float2bfloat16_rn(r1);
                                yp[2] = __float2bfloat16_rn(r2);
                                yp[3] = __float2bfloat16_rn(r3);
                            }
                        }
                    }
                    u += len;
                    ++j;
                    continue;
                }
            }
#pragma unroll 1
            for (int cb = 0; cb < RB * kHalfCols; cb += 16) {
                // (RB = 2: the second row block's accumulator sits BNX columns further)
                const int b = cb / kHalfCols, c0 = cb - b * kHalfCols;
                const int n = nt * TR + b * 128 + r;
                const bool row_ok = n < N;
                const float swn = b == 0 ? swn_rb[0] : swn_rb[RB - 1];
                const uint32_t tmem_acc = tmem_acc0 + (uint32_t)(b * BNX);
                uint32_t v[16];
                ptx::tmem_ld_32x32b_x16(tmem_acc + (uint32_t)c0, v);
                ptx::tmem_ld_wait();
                if (m0 + c0 >= M) continue;  // warp-uniform
                if (whole) {
                    // this chunk's activation scales sit in lanes (c0 % 32) .. +15 of one prefetched register
                    float sx_lane = sx_pre[0];
#pragma unroll
                    for (int c = 1; c < kHalfCols / 32; ++c) sx_lane = (c0 >= c * 32) ? sx_pre[c] : sx_lane;
                    float sx[16];
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj) sx[jj] = __shfl_sync(0xFFFFFFFFu, sx_lane, (c0 & 16) + jj);
                    if (row_ok) {
                        const bool inside = m0 + c0 + 16 <= M;   // the whole chunk inside the problem: no test per token
                        if (out_dtype == W4A8_OUT_FP32) {
                            float* yp = reinterpret_cast<float*>(y) + (int64_t)(m0 + c0) * ldy + n;
                            if (inside) {
#pragma unroll
                                for (int jj = 0; jj < 16; ++jj) yp[(int64_t)jj * ldy] = __uint_as_float(v[jj]) * (sx[jj] * swn);
                            } else {
#pragma unroll
                                for (int jj = 0; jj < 16; ++jj)
                                    if (m0 + c0 + jj < M) yp[(int64_t)jj * ldy] = __uint_as_float(v[jj]) * (sx[jj] * swn);
                            }
                        } else {
                            __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(y) + (int64_t)(m0 + c0) * ldy + n;
                            if (inside) {
#pragma unroll
                                for (int jj = 0; jj < 16; ++jj)
                                    yp[(int64_t)jj * ldy] = __float2bfloat16_rn(__uint_as_float(v[jj]) * (sx[jj] * swn));
                            } else {
#pragma unroll
                                for (int jj = 0; jj < 16; ++jj)
                                    if (m0 + c0 + jj < M)
                                        yp[(int64_t)jj * ldy] = __float2bfloat16_rn(__uint_as_float(v[jj]) * (sx[jj] * swn));
                            }
                        }
                    }
                } else if (row_ok) {
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj)
                        if (m0 + c0 + jj < M) __stcg(my_slot + (c0 + jj) * 128 + r, __uint_as_float(v[jj]));
                }
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(bar_acc_empty(buf));
            if (!whole) {
                // Publish the partial tile and remember the tile for the reduction at the end.
                __threadfence();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (leader) atomicAdd(counters + tile, 1u);
                if (n_shared++ == 0) shared_tile0 = tile;
                else shared_tile1 = tile;
            }
            u += len;
            ++j;
        }
        if (leader) {
            share_slot[0] = (uint32_t)n_shared;
            share_slot[1] = (uint32_t)shared_tile0;
            share_slot[2] = (uint32_t)shared_tile1;
        }
    } else {
        // ------------------------------------------------------------------ dequantization groups
        const int dw = warp - 10;
        const int g = dw >> 2;
        const int r = (dw & 3) * 32 + lane;
        for (int it = Cfg::W8 ? n_it : g; it < n_it; it += G) {   // (W8: nothing to expand)
            const int s1 = it % S1, s2 = it % S2;
            if (!ptx::mbar_wait(bar_full(s1), (uint32_t)((it / S1) & 1), abort_flag, status_word)) break;
            if (it >= S2) {
                if (!ptx::mbar_wait(bar_free2(s2), (uint32_t)((it / S2 - 1) & 1), abort_flag, status_word)) break;
            }
            if constexpr (Cfg::W16)
                dequant_row_to_smem_bf16(stage_w(s1) + tiled_row_offset(r), stage_w(s1) + (uint32_t)Cfg::kCodeBytes + (uint32_t)(r * Cfg::kMeta), r,
                                         stage_w8(s2) + (uint32_t)r * 128u);
            else
#pragma unroll
            for (int b = 0; b < RB; ++b)
                dequant_row_to_smem<Cfg::FMT>(stage_w(s1) + tiled_row_offset(b * 128 + r),
                                              stage_w(s1) + (uint32_t)Cfg::kCodeBytes + (uint32_t)((b * 128 + r) * Cfg::kMeta), r,
                                              stage_w8(s2) + (uint32_t)(b * 16384) + (uint32_t)r * 128u);
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(bar_w8_full(s2));
            if constexpr (RB == 2) {
                // after this group's last stage of a tile: help to drain the tile's accumulators
                const int jt = it / KB;
                if (it + G >= n_it || (it + G) / KB != jt) {
                    ptx::griddep_wait();  // (scales and outputs may still be in use by earlier kernels; long satisfied by now)
                    if (!drain_wide(jt, 2 + g)) break;
                }
            }
        }
        if constexpr (Cfg::CL) {
            ptx::cluster_arrive();
            cl_arrived = true;
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
    // CL: no CTA leaves while a peer may still write into its shared memory or while its own copies,
    // which read its shared memory, are in flight (a peer arrives here only after they have landed);
    // also on the way out after a timeout
    if constexpr (Cfg::CL) {
        if (!cl_arrived) ptx::cluster_arrive();
        if (!cl_waited) ptx::cluster_wait();
        // (execution order only: a release here would first wait for this thread's output stores)
        ptx::cluster_arrive_relaxed();
        ptx::cluster_wait();
    }

    // ---- reduction of the shared tiles, by every thread of the CTA: this CTA's slice of the token
    // columns of each tile it holds a partial of ----
    if (aligned) return;
    ptx::griddep_wait();
    const int n_shared = (int)share_slot[0];
    unsigned int* done = counters + (int64_t)TM * TN;  // second counter per tile: finished reducers
    // Slot index of every contributor of the tile, worked out once (64-bit divisions: left inside
    // the adding loop they cost every thread more than the loads did).  The rings are idle by now.
    int* slot_of = reinterpret_cast<int*>(sm);
    for (int k = 0; k < n_shared; ++k) {
        const int64_t tile = (int64_t)share_slot[1 + k];
        const int64_t p_lo = ((tile * KB + 1) * P - 1) / U;  // first and last contributor
        const int64_t p_hi = (((tile + 1) * KB) * P - 1) / U;
        const int C = (int)(p_hi - p_lo) + 1, me = (int)(p - p_lo);
        __syncthreads();  // readers of the previous tile's table are done
        for (int i = (int)threadIdx.x; i < C; i += Cfg::kThreads) {
            // contributor q's slot for this tile: its first slot if the tile is where its share begins, else its second
            const int64_t q = p_lo + i;
            const int64_t first_tile = (q * U / P) / KB;
            slot_of[i] = (int)(q * 2 + (tile == first_tile ? 0 : 1));
        }
        if (threadIdx.x == 0 && *abort_flag == 0u) {
            // bounded wait for the C arrivals
            uint64_t t0 = 0;
            uint32_t spins = 0;
            while (ptx::ld_acquire_gpu(counters + tile) < (uint32_t)C) {
                if ((++spins & 63u) == 0u) {
                    const uint64_t now = ptx::globaltimer_ns();
                    if (t0 == 0) {
                        t0 = now;
                    } else if (now - t0 > ptx::kWaitLimitNs) {
                        *abort_flag = 1u;
                        atomicOr(status_word, kStatusTimeout);
                        break;
                    }
                }
            }
        }
        __syncthreads();
        if (*abort_flag != 0u) break;
        __threadfence();
        const int nt = (int)(tile / TM), mt = (int)(tile - (int64_t)nt * TM);
        const int nrow = (N - nt * 128) < 128 ? (N - nt * 128) : 128;
        const int ncol = (M - mt * BNX) < BNX ? (M - mt * BNX) : BNX;  // valid token columns of the tile
        const int c_lo = (int)((int64_t)me * ncol / C), c_hi = (int)((int64_t)(me + 1) * ncol / C);
        // element e of the slice: row e % 128 (consecutive threads, consecutive addresses), column c_lo + e / 128
        const int total = (c_hi - c_lo) * 128;
        for (int e0 = (int)threadIdx.x; e0 < total; e0 += 4 * Cfg::kThreads) {
            float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll 4
            for (int i = 0; i < C; ++i) {
                const float* sl = slots + (int64_t)slot_of[i] * Cfg::kSlotFloats + c_lo * 128;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int e = e0 + jj * Cfg::kThreads;
                    if (e < total && (e & 127) < nrow) acc[jj] += __ldcg(sl + e);
                }
            }
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int e = e0 + jj * Cfg::kThreads;
                if (e < total && (e & 127) < nrow) {
                    const int n = nt * 128 + (e & 127), m = mt * BNX + c_lo + (e >> 7);
                    const float res = acc[jj] * (__ldg(s_x + m) * __ldg(s_w + (int64_t)n * sw_stride));
                    if (out_dtype == W4A8_OUT_FP32)
                        reinterpret_cast<float*>(y)[(int64_t)m * ldy + n] = res;
                    else
                        reinterpret_cast<__nv_bfloat16*>(y)[(int64_t)m * ldy + n] = __float2bfloat16_rn(res);
                }
            }
        }
        // the last reducer to finish re-arms the tile's counters for the next launch
        __syncthreads();
        if (threadIdx.x == 0) {
            if (atomicAdd(done + tile, 1u) == (uint32_t)(C - 1)) {
                counters[tile] = 0u;
                done[tile] = 0u;
            }
        }
    }
}

}  // namespace w4a8
