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
#include "w4a8_simple_kernels.cuh"
#include "w4a8_tiled_format.cuh"

namespace w4a8 {



template <int MT_, int G_, int FMT_, bool SPLITK_ = false>
struct SnCfg {
    // SPLITK: the K range may be cut in chunks (layers with few output channels); otherwise the
    // chunk arithmetic is compiled out.
    static constexpr bool SPLITK = SPLITK_;
    static constexpr int MT = MT_;      // tokens per tile = MMA N (16 or 64)
    static constexpr int G = G_;        // dequantization groups of 4 warps
    static constexpr int FMT = FMT_;
    static constexpr int kS1Max = 16;   // ring of TMA stages (runtime depth <= this)
    static constexpr int kS2 = MT_ == 64 ? 4 : 3;  // ring of dequantized stages in tensor memory
    static constexpr int kItems = 2;    // (k-block, 128-row block) pairs per stage
    static constexpr int kMeta = meta_bytes(FMT);
    static constexpr int kTmemCols = MT_ == 16 ? 256 : 512;
    static constexpr int kAStageCols = kItems * 32;        // 128 bytes per row and item
    static constexpr int kDCol = kS2 * kAStageCols;        // accumulators start after the A ring
    static constexpr int kThreads = 32 * (6 + 4 * G);
    static constexpr int kBarBytes = 768;
    // Staging area of the epilogue: 16 tokens x 128 rows of outputs (FP32 at most), from which Y is
    // written in 16-byte pieces.  (Thirty-two 2-byte stores per warp instruction cost ~120 cycles
    // each, one after the other: 16 of them per thread made a 1 us tail.)
    static constexpr int kOutBytes = 16 * 128 * 4;
    // Decode-sized launches (<= 16 tokens) take half an SM each, so that the CTAs of the next
    // kernel in the stream can start -- and prefetch their weights -- while this one finishes.
    static constexpr int kSmemBudget = MT_ == 16 ? 100 * 1024 : (MT_ == 64 ? 200 * 1024 : 220 * 1024);
    static_assert(MT == 16 || MT == 64 || MT == 128, "token tile");
    static_assert(kDCol + 2 * MT <= kTmemCols, "tensor memory columns");
    static_assert((3 * kS1Max + kS2 + 3) * 8 + 16 + 3 * 64 + 16 <= kBarBytes, "barrier area");
};

// Launch-time plan shared by host and device.
struct SnPlan {
    int T;         // number of tiles = row ranges x K chunks; tile t = (row range t / KSPLIT, K chunk t % KSPLIT)
    int KSPLIT;    // K chunks per row range (1 = every CTA walks the whole K; > 1 needs the workspace)
    int MBLK;      // 128-row blocks per range (1 or 2)
    int KS;        // k-blocks per pipeline stage (KS * MBLK == 2)
    int S1;        // depth of the TMA ring (>= kS2)
    int meta_off;  // offset of the meta pieces inside a packed stage
    int wstage;    // bytes per stage: packed codes + meta
    int xstage;    // bytes per stage: activation tiles
    int smem;      // dynamic shared memory to request
    int P;         // CTAs that do the work; CTA p takes tiles p, p + P, ...
    int sched;     // -1: CTA p = blockIdx.x.  Otherwise twice P CTAs are launched and draw their worker indices at
                   // run time (see below): kSchedInWorkspace = the table sits in the caller's workspace,
                   // 0 .. kSchedSlots - 1 = slot of the library's own table
};

// ---- placement of the decode-sized launches -------------------------------------------------
// Two CTAs of this kernel fit on an SM so that the CTAs of the NEXT launch can move in beside
// the running ones, fetch their first weight stages and expand them while they wait for their
// activations.  That only pays if the two CTAs on an SM belong to different launches: two CTAs
// of one launch on one SM share its integer pipe and take twice as long, and the SM they left
// empty then receives two CTAs of the following launch, so the pattern persists.  The hardware
// places a CTA wherever there is room, so the kernel enforces the rule itself: a launch has
// twice as many CTAs ("candidates") as it needs workers.  A candidate that finds a worker of
// its own launch already on its SM retires at once (unless so few candidates are left that the
// work could otherwise go undone); the first candidate on an SM takes the next worker index.
// The state of a launch (one SchedSlot) is cleared by the last of its candidates to enter.  It
// lives in the caller's workspace when there is one (at byte kSchedWsOffset, after the split-K
// counters): launches that may run at the same time must have different workspaces anyway, and
// consecutive launches of one stream cannot meet in it, because the dependent launch starts only
// after every candidate of this one has entered (entering comes before the launch-dependents
// trigger in every candidate).  Without a workspace the state is a slot of a small table in the
// library image, handed out round-robin by the host over all launches of the process; that is
// safe only while fewer than kSchedSlots such launches are in flight, and a captured launch keeps
// the slot it drew at capture time.
constexpr int kSchedSlots = 64;
constexpr int kSchedInWorkspace = kSchedSlots;
constexpr int kSchedMaxSMs = 192;
constexpr int kSchedWsOffset = 1024;
struct __align__(16) SchedSlot {
    unsigned int started;   // candidates that have drawn a start number
    unsigned int issued;    // worker indices handed out
    unsigned int finished;  // candidates that have entered
    unsigned int gen;       // launches that have used and cleared this slot (never reset)
    unsigned int on_sm[kSchedMaxSMs];  // candidates of this launch seen per SM
};
static_assert(sizeof(SchedSlot) <= 1024, "the placement state has 1 KB of the workspace");
__device__ SchedSlot g_sched[kSchedSlots];

// Called by thread 0 of a candidate: returns its worker index, or -1 to retire.  Plain atomic adds
// only (a compare-and-swap loop on one word serialises hundreds of CTAs that start together at one
// L2 round trip each).
__device__ __forceinline__ int sched_enter(SchedSlot* sl, int workers, int candidates) {
    unsigned int smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    // The count of issued indices is read BEFORE this candidate takes its start number (an acquire
    // load: the adds below cannot move in front of it).  Then every index counted in i was drawn by
    // a candidate that is not among the `candidates - c` still to come, and the test below can only
    // err towards working.  (Read together with the adds it saved a round trip, but i could then
    // include draws of candidates with later start numbers, which the test counts again as still
    // to come: a decliner too many, an index never issued.)
    const unsigned int i = ptx::ld_acquire_gpu(&sl->issued);
    // (the two adds are independent: one L2 round trip for both)
    const unsigned int c = atomicAdd(&sl->started, 1u);
    const bool first_here = smid < (unsigned)kSchedMaxSMs ? atomicAdd(&sl->on_sm[smid], 1u) == 0u : true;
    bool want = first_here;
    if (!want) {
        // A second candidate on this SM works only if the candidates still to come could not
        // cover the indices still to be issued.  The count read above may lag behind the true
        // one, which errs towards working -- a candidate that then draws an index beyond the last
        // one retires after all; the candidate with the last start number therefore declines only
        // when every index has been issued.
        want = i < (unsigned)workers && (unsigned)workers - i >= (unsigned)candidates - c;
    }
    if (!want) return -1;
    const unsigned int idx = atomicAdd(&sl->issued, 1u);
    return idx < (unsigned)workers ? (int)idx : -1;
}
// Called once by every candidate after sched_enter: the slot is only needed while candidates
// enter, so the last one to have entered clears it (nothing of this runs at the end of the
// kernel, where it would delay the launch's completion).
// (`gen` = the slot's generation if the caller has read it during this launch, kSchedGenUnknown otherwise)
constexpr unsigned int kSchedGenUnknown = 0xFFFFFFFFu;
__device__ __forceinline__ void sched_entered(SchedSlot* sl, int candidates, unsigned int gen_in, int workers,
                                              unsigned int* status_word) {
    __threadfence();
    if (atomicAdd(&sl->finished, 1u) == (unsigned)candidates - 1u) {
        // Every candidate has entered, so every index that will ever be drawn has been: if one is
        // missing, a tile of this launch is never computed -- say so instead of leaving stale
        // outputs behind silently.
        if (*reinterpret_cast<volatile unsigned int*>(&sl->issued) < (unsigned)workers)
            atomicOr(status_word, kStatusPlacement);
        // The last one clears the slot.  This sits between the last candidate's arrival and the
        // release of the dependent launch, so it is kept short: 16-byte stores, the three counters
        // and the new generation (which releases the candidates that still hold their place) in
        // one of them, a single fence.
        static_assert(kSchedMaxSMs % 4 == 0 && sizeof(SchedSlot) == 16 + 4 * kSchedMaxSMs, "slot layout");
        const unsigned int gen =
            gen_in != kSchedGenUnknown ? gen_in : *reinterpret_cast<volatile unsigned int*>(&sl->gen);
        uint4* v = reinterpret_cast<uint4*>(sl);
#pragma unroll 8
        for (int i = 1; i <= kSchedMaxSMs / 4; ++i) v[i] = make_uint4(0u, 0u, 0u, 0u);
        v[0] = make_uint4(0u, 0u, 0u, gen + 1u == kSchedGenUnknown ? 0u : gen + 1u);
        __threadfence();
    }
}

// A candidate that declined keeps its place on the SM until every worker index has been handed
// out (bounded: a fraction of a millisecond).  If it left at once, the hardware would put the
// next waiting candidate into the same place, on an SM that already has its worker, and that
// one would decline too: on SMs with two free places (the previous launch had fewer workers than
// there are SMs) the whole surplus of candidates burnt away like this before the other SMs had
// room, and the last ones were then forced to work as second workers after all.
__device__ __forceinline__ void sched_hold(SchedSlot* sl, int workers, unsigned int gen0) {
    const uint64_t t0 = ptx::globaltimer_ns();
    // (gen0 = the slot's generation when this candidate entered: once it has moved on, the slot
    // belongs to a later launch and its counts say nothing about this one)
    while (*reinterpret_cast<volatile unsigned int*>(&sl->gen) == gen0 &&
           *reinterpret_cast<volatile unsigned int*>(&sl->issued) < (unsigned)workers &&
           ptx::globaltimer_ns() - t0 < 200000ull) {
        __nanosleep(500);
    }
}

// Epilogue of the split-N kernel: scales 16 tokens of accumulated sums (row r of 128-row block b,
// tokens c0..c0+15) with Eq. 4 / Eq. 11 and writes them to Y, through the staging area in 16-byte
// pieces when the rows of Y are 16-byte aligned.  Called by all 128 epilogue threads together.
template <class Cfg>
__device__ __forceinline__ void sn_emit(const uint32_t (&accv)[16], float swb, int b, int c0, int r, int et, int R,
                                        int n0, int M, int es, bool wide_out, uint32_t out_s, void* y, int64_t ldy,
                                        const float (&sx_lane)[Cfg::MT / 32 > 0 ? Cfg::MT / 32 : 1]) {
    constexpr int MT = Cfg::MT;

    const int row = b * 128 + r;
    const bool row_ok = row < R;
    const int n = n0 + row;
    float sxv = sx_lane[0];
#pragma unroll
    for (int c = 1; c < MT / 32; ++c)
        if (c0 >= 32 * c) sxv = sx_lane[c];
    float res[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float sxm = __shfl_sync(0xFFFFFFFFu, sxv, (c0 & 16) + j);
        res[j] = __uint_as_float(accv[j]) * (sxm * swb);  // Eq. 4, Eq. 11
    }
    if (wide_out) {
        // tokens x rows into the staging area, then 16-byte pieces of Y rows
        const uint32_t pitch = 128u * (uint32_t)es;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const uint32_t a = out_s + (uint32_t)j * pitch + (uint32_t)(r * es);
            if (es == 4)
                asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(res[j]) : "memory");
            else
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(a),
                             "h"(__bfloat16_as_ushort(__float2bfloat16_rn(res[j])))
                             : "memory");
        }
        asm volatile("bar.sync 3, 128;" ::: "memory");
        const int Rb = (R - b * 128) < 128 ? (R - b * 128) : 128;
        const int ppt = (Rb * es) >> 4;  // 16-byte pieces per token (rows come in eights)
        const int ntok = (M - c0) < 16 ? (M - c0) : 16;
        char* yb = static_cast<char*>(y) + ((int64_t)c0 * ldy + n0 + b * 128) * es;
        for (int id = et; id < ntok * ppt; id += 128) {
            const int tok = id / ppt, piece = id - tok * ppt;
            uint4 w;
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w)
                         : "r"(out_s + (uint32_t)tok * pitch + (uint32_t)(piece << 4)));
            *reinterpret_cast<uint4*>(yb + (int64_t)tok * ldy * es + (piece << 4)) = w;
        }
        asm volatile("bar.sync 3, 128;" ::: "memory");  // before the area is written again
    } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const int m = c0 + j;
            if (m < M && row_ok) {
                if (es == 4)
                    reinterpret_cast<float*>(y)[(int64_t)m * ldy + n] = res[j];
                else
                    reinterpret_cast<__nv_bfloat16*>(y)[(int64_t)m * ldy + n] = __float2bfloat16_rn(res[j]);
            }
        }
    }
}

// Register budget of the decode variant (<= 16 tokens): besides two of its CTAs an SM has to hold
// the small kernel that runs between two layers (activation quantization: 256 threads x 32..48
// registers), or the CTA that finds no room starts a whole layer late.  Bounds for 576 threads
// give 56 registers: 2 x 448 x 56 + 256 x 48 <= 65536.
template <class Cfg>
__global__ void __launch_bounds__(Cfg::MT == 16 ? 576 : Cfg::kThreads, Cfg::MT == 16 ? 2 : 1)
linear_splitn_kernel(const __grid_constant__ CUtensorMap tmap_x,  // X8 u8 [M][K], box 128 x MT, 128B swizzle
                     const uint8_t* __restrict__ wpp, const float* __restrict__ s_x,
                     const float* __restrict__ s_w, int sw_stride, void* __restrict__ y, int64_t ldy,
                     int out_dtype, int M, int N, int K, const SnPlan plan,
                     unsigned int* counters, float* partials, unsigned int* status_word) {
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
    const uint32_t out_s = bars_addr + (uint32_t)Cfg::kBarBytes;  // epilogue staging, kOutBytes
    volatile unsigned int* ticket_s = reinterpret_cast<volatile unsigned int*>(tmem_slot + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = K >> 7;
    const int64_t NU = N >> 3;           // the row partition works in units of 8 rows
    int P = gridDim.x, p = blockIdx.x;
    __shared__ int worker_s;
    // (thread 0 asks for a worker index while thread 32 sets up the barriers)
    SchedSlot* const sched_slot =
        plan.sched == kSchedInWorkspace
            ? reinterpret_cast<SchedSlot*>(reinterpret_cast<uint8_t*>(counters) + kSchedWsOffset)
            : &g_sched[plan.sched >= 0 ? plan.sched : 0];
    unsigned int sched_gen = 0u;  // (thread 0 only)
    if (plan.sched >= 0 && threadIdx.x == 0) {
        sched_gen = *reinterpret_cast<volatile unsigned int*>(&sched_slot->gen);
        worker_s = sched_enter(sched_slot, plan.P, (int)gridDim.x);
    }
    const int KSPLIT = Cfg::SPLITK ? plan.KSPLIT : 1, TR = T / KSPLIT;
    // Tile t: 8-row units [u0, u1) of row range t / KSPLIT, k-blocks [kb0, kb0 + nkb) of chunk t % KSPLIT.
    const int nst_all = (KB + KS - 1) / KS;  // stages per tile when K is not cut
    struct TileGeom {
        int u0, u1, kb0, nkb;
    };
    auto tile_geom = [&](int t) {
        TileGeom g;
        if constexpr (!Cfg::SPLITK) {
            g.u0 = (int)((int64_t)t * NU / T);
            g.u1 = (int)((int64_t)(t + 1) * NU / T);
            g.kb0 = 0;
            g.nkb = KB;
        } else {
            const int rt = t / KSPLIT, kc = t - rt * KSPLIT;
            g.u0 = (int)((int64_t)rt * NU / TR);
            g.u1 = (int)((int64_t)(rt + 1) * NU / TR);
            g.kb0 = (int)((int64_t)kc * KB / KSPLIT);
            g.nkb = (int)((int64_t)(kc + 1) * KB / KSPLIT) - g.kb0;
        }
        return g;
    };

    if (threadIdx.x == 32) {
        for (int s = 0; s < S1; ++s) {
            ptx::mbar_init(bar_full0 + 8u * s, 1);
            ptx::mbar_init(bar_xfull0 + 8u * s, 1u);
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
    if (plan.sched >= 0) {
        __syncthreads();
        p = worker_s;
        P = plan.P;
        if (p < 0) {  // a worker of this launch is already on this SM: retire
            if (threadIdx.x == 0) {
                sched_entered(sched_slot, (int)gridDim.x, sched_gen, plan.P, status_word);  // before the trigger: see the notes beside SchedSlot
                ptx::griddep_launch_dependents();
                sched_hold(sched_slot, plan.P, sched_gen);
            }
            return;
        }
        if (threadIdx.x == 64) sched_entered(sched_slot, (int)gridDim.x, kSchedGenUnknown, plan.P, status_word);  // an idle epilogue thread
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
                const TileGeom tg = tile_geom(t);
                const int u0 = tg.u0, u1 = tg.u1, kb0 = tg.kb0, nkb = tg.nkb;
                const int nst = Cfg::SPLITK ? (nkb + KS - 1) / KS : nst_all;
                const int R = (u1 - u0) * 8;
                const uint32_t cbytes = (uint32_t)(R * kRowCodeBytes), mbytes = (uint32_t)(R * MB);
                const uint8_t* cptr = wpp + (int64_t)kb0 * code_step + (int64_t)u0 * 8 * kRowCodeBytes;
                const uint8_t* mptr = meta_base + (int64_t)kb0 * meta_step + (int64_t)u0 * 8 * MB;
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
                    const int ks = (nkb - kb) < KS ? (nkb - kb) : KS;
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
                        const int ksx = (nkb - xkb) < KS ? (nkb - xkb) : KS;
                        const uint32_t xdst = x_ring + (uint32_t)(rx.idx * plan.xstage);
                        const uint32_t xfull = bar_xfull0 + 8u * (uint32_t)rx.idx;
                        const int x0 = (kb0 + xkb) * 128;
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
                const TileGeom tg = tile_geom(t);
                const int u0 = tg.u0, u1 = tg.u1, kb0 = tg.kb0, nkb = tg.nkb;
                const int nst = Cfg::SPLITK ? (nkb + KS - 1) / KS : nst_all;
                for (int st = 0; st < nst; ++st) {
                    ok = ptx::mbar_wait(bar_xfull0 + 8u * (uint32_t)r1.idx, r1.phase, abort_flag, status_word);
                    ok = ok && ptx::mbar_wait(bar_a_full0 + 8u * (uint32_t)r2.idx, r2.phase, abort_flag, status_word);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    // A stage holds two (k-block, 128-row block) items: either two k-blocks of one
                    // row block or one k-block of two row blocks.
                    const int ks = (nkb - kb) < KS ? (nkb - kb) : KS;
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
        // The scales are fetched before the accumulator is waited for (a global load issued after
        // it would add its full latency to the kernel's tail): s_x one or two per lane, broadcast
        // by shuffles later; s_w per row at the top of each range.
        const int et = (warp - 2) * 32 + lane;  // index among the 128 epilogue threads
        const int es = out_dtype == W4A8_OUT_FP32 ? 4 : 2;
        const bool wide_out = (((int64_t)ldy * es) & 15) == 0;  // Y rows 16-byte aligned (y itself is)
        float sx_lane[MT / 32 > 0 ? MT / 32 : 1];
        ptx::griddep_wait();  // s_x comes from, and Y may still be read by, earlier kernels
#pragma unroll
        for (int c = 0; c < (MT / 32 > 0 ? MT / 32 : 1); ++c)
            sx_lane[c] = (c * 32 + lane < M) ? __ldg(s_x + c * 32 + lane) : 0.0f;
        for (int t = p; t < T && ok; t += P) {
            const TileGeom tg = tile_geom(t);
            const int u0 = tg.u0, u1 = tg.u1, kb0 = tg.kb0, nkb = tg.nkb;
            const int nst = Cfg::SPLITK ? (nkb + KS - 1) / KS : nst_all;
            const int R = (u1 - u0) * 8;
            const int n0 = u0 * 8;
            float swn[2];
#pragma unroll
            for (int b = 0; b < 2; ++b)
                swn[b] = (b < MBLK && b * 128 + r < R) ? __ldg(s_w + (int64_t)(n0 + b * 128 + r) * sw_stride) : 0.0f;
            ok = ptx::mbar_wait(bar_acc_full, acc_phase, abort_flag, status_word);
            acc_phase ^= 1u;
            if (!ok) break;
            ptx::tc_fence_after_sync();
            // With the K range cut in KSPLIT chunks the accumulator is a partial sum: it goes to the
            // workspace (tile t, token-major: coalesced stores), and the CTA that arrives last at the row
            // range adds the chunks in ascending order (after the roles have joined).
            float* part = partials + (int64_t)t * (MT * 128);
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                if (b >= MBLK) break;
#pragma unroll 1
                for (int c0 = 0; c0 < MT; c0 += 16) {
                    if (c0 >= M) break;  // uniform
                    uint32_t v[16];
                    ptx::tmem_ld_32x32b_x16(
                        tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(Cfg::kDCol + b * MT + c0), v);
                    ptx::tmem_ld_wait();
                    if (KSPLIT == 1) {
                        sn_emit<Cfg>(v, swn[b], b, c0, r, et, R, n0, M, es, wide_out, out_s, y, ldy, sx_lane);
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (c0 + j < M) __stcg(part + (c0 + j) * 128 + r, __uint_as_float(v[j]));
                    }
                }
            }
            if (KSPLIT > 1) {
                const int rt = t / KSPLIT;
                __threadfence();
                asm volatile("bar.sync 3, 128;" ::: "memory");
                if (et == 0) *ticket_s = atomicAdd(counters + rt, 1u);
                asm volatile("bar.sync 3, 128;" ::: "memory");
                // (the CTA that drew the last ticket adds the chunks after the roles have joined, below)
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
            const TileGeom tg = tile_geom(t);
            const int u0 = tg.u0, u1 = tg.u1, kb0 = tg.kb0, nkb = tg.nkb;
            const int nst = Cfg::SPLITK ? (nkb + KS - 1) / KS : nst_all;
            const int R = (u1 - u0) * 8;
            // This thread's rows of the range (one per 128-row block).  A lane beyond the range
            // repeats the last row: its tensor-memory lane feeds accumulator rows nobody reads out.
            const int row0 = r < R ? r : R - 1;
            const int row1 = 128 + r < R ? 128 + r : R - 1;
            const uint32_t code_off = tiled_row_offset(row0);
            const uint32_t meta_off = (uint32_t)(plan.meta_off + row0 * MB);
            // address steps from one item of a stage to the next: (block 0 -> block 1), then on to
            // block 0 of the next k-block; with one block per k-block both are the k-block step
            const uint32_t code_kstep = (uint32_t)(R * kRowCodeBytes), meta_kstep = (uint32_t)(R * MB);
            const uint32_t code_s0 = MBLK == 2 ? tiled_row_offset(row1) - code_off : code_kstep;
            const uint32_t meta_s0 = MBLK == 2 ? (uint32_t)((row1 - row0) * MB) : meta_kstep;
            const uint32_t code_s1 = MBLK == 2 ? code_kstep - code_s0 : code_kstep;
            const uint32_t meta_s1 = MBLK == 2 ? meta_kstep - meta_s0 : meta_kstep;
            int st = turn;
            for (; st < nst; st += G) {
                const int kb = st * KS;
                const int ks = (nkb - kb) < KS ? (nkb - kb) : KS;
                // Both barriers are normally complete already.  The tensor-memory slot FIRST: once the
                // MMAs S2 stages back have completed, every earlier stage has landed -- among them the
                // previous use of this stage's ring slot (S1 >= S2) -- so the parity test of "weights
                // landed" cannot mistake the phase before last for this one.  (Tested the other way
                // round, a group ahead of a late copy could pass one phase early.)
                const uint32_t full_bar = bar_full0 + 8u * (uint32_t)r1.idx;
                const uint32_t free_bar = bar_free10 + 8u * (uint32_t)rl.idx;
                if (done >= S2 && !ptx::mbar_test_wait(free_bar, rl.phase))
                    ok = ptx::mbar_wait(free_bar, rl.phase, abort_flag, status_word);
                if (ok && !ptx::mbar_test_wait(full_bar, r1.phase))
                    ok = ptx::mbar_wait(full_bar, r1.phase, abort_flag, status_word);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t wsrc = w_ring + (uint32_t)(r1.idx * plan.wstage);
                uint32_t src = wsrc + code_off, msrc = wsrc + meta_off;
                uint32_t a_col = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(r2.idx * Cfg::kAStageCols);
                const int items = ks * MBLK;
                for (int i = 0; i < items; ++i) {
                    dequant_row_to_tmem<Cfg::FMT>(src, msrc, a_col);
                    a_col += 32u;
                    src += (i & 1) ? code_s1 : code_s0;
                    msrc += (i & 1) ? meta_s1 : meta_s0;
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
    if constexpr (Cfg::SPLITK) {
        // K was cut: a CTA holds exactly one tile.  The CTA that arrived last at its row range adds
        // the KSPLIT partial sums in ascending chunk order -- every thread of the CTA takes part, so
        // that many independent loads are in flight -- scales (Eq. 4, Eq. 11) and writes Y.
        if (KSPLIT > 1 && p < T && *ticket_s == (unsigned int)(KSPLIT - 1)) {
            ptx::griddep_wait();  // s_x comes from, and Y may still be read by, earlier kernels
            __threadfence();
            const int rt = p / KSPLIT;
            const TileGeom tg = tile_geom(p);
            const int R = (tg.u1 - tg.u0) * 8, n0 = tg.u0 * 8;
            const float* p0 = partials + (int64_t)rt * KSPLIT * (MT * 128);
            const int total = (M < MT ? M : MT) * 128;
#pragma unroll 2
            for (int e = (int)threadIdx.x; e < total; e += Cfg::kThreads) {
                const int row = e & 127, tok = e >> 7;
                if (row < R) {
                    float acc = 0.0f;
                    for (int kc = 0; kc < KSPLIT; ++kc) acc += __ldcg(p0 + (int64_t)kc * (MT * 128) + e);
                    const int n = n0 + row;
                    const float res = acc * (__ldg(s_x + tok) * __ldg(s_w + (int64_t)n * sw_stride));
                    if (out_dtype == W4A8_OUT_FP32)
                        reinterpret_cast<float*>(y)[(int64_t)tok * ldy + n] = res;
                    else
                        reinterpret_cast<__nv_bfloat16*>(y)[(int64_t)tok * ldy + n] = __float2bfloat16_rn(res);
                }
            }
            if (threadIdx.x == 0) counters[rt] = 0u;  // ready for the next launch
        }
    }
}

}  // namespace w4a8
