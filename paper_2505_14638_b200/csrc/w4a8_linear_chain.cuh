// One persistent launch for a chain of decode-sized W4A8 linear layers (M <= 16 tokens each) on
// sm_100a: the whole inference flow of Sec. 3 -- Eq. 13 activation quantization, Eq. 10 weight
// expansion, FP8 MMAs with FP32 accumulation, Eq. 4 / Eq. 11 epilogue -- for every problem of the
// chain, in order, inside one kernel.
//
// Why one launch: a decode-sized layer streams its packed weights in a few microseconds, and the
// hand-over between two dependent grids (completion of the first, release and start-up of the
// second) costs about as much again.  Here one CTA per SM owns the whole SM for the whole chain:
//   * the weight ring (bulk copies into ~190 KB of shared memory) never drains at a problem
//     boundary: the codes of problem i + 1 depend on nothing and are fetched while problem i is
//     still being multiplied;
//   * the CTA has all 512 tensor-memory columns: six stages of expanded weights in flight plus four
//     accumulator buffers, so the epilogues of up to four segments overlap the MMAs that follow;
//   * problems are handed over through counters in the caller's workspace: the activations of a
//     problem are quantized row by row by the epilogue warps of a few CTAs (one row per CTA),
//     published with a fence and one atomic add, and picked up by every CTA's activation loader
//     with a bounded acquire poll; a problem that reads the output of an earlier one waits (again
//     bounded) for that problem's "blocks written" counter first.
//
// Work partition.  The output channels of a problem are cut into blocks of 96 rows (three
// tensor-memory lane quarters; the fourth quarter's SM sub-partition is left to the warps that
// issue copies and MMAs, each of which costs its sub-partition tens of cycles).  As long as there
// are at least as many blocks left as CTAs, every CTA takes whole blocks (all of K, one or two
// blocks at a time, results written directly).  The remaining blocks are cut along K as well: their
// (block, k-block) items are dealt out evenly, a CTA gets one contiguous run (at most two blocks),
// writes its FP32 partial sums to the workspace, and the CTA that holds a block's lowest k range (the
// second part of its run: it reaches the block last) adds the partial sums in ascending k order -- a
// fixed order, so results repeat bit for bit -- and writes Y.  A CTA works on its run of the cut
// blocks first and on its whole blocks afterwards, so that the hand-over of the partial sums hides
// behind the whole blocks instead of standing at the end of the problem, where the next problem of
// a dependent chain waits for it.  Every CTA expands the same number of weights within one item,
// whatever N is.
//
// Data path of one (k-block, 96-row block) item: as in the split-N kernel --
//   HBM --bulk copy--> shared memory (INT4 codes + group scales [+ zero-points])
//       --one thread per row: look-up-table expansion to E4M3 (Eq. 10)--> tensor memory (A operand)
//       --tcgen05.mma kind::f8f6f4, B = FP8 activation tile from shared memory--> accumulator.
// The FP8 activations of a problem live in the workspace as ready-made operand tiles
// ([k-block][16 tokens][128 bytes], already in the 128-byte-swizzled order the MMA descriptor
// expects), so a plain bulk copy brings a tile in: no tensor map, nothing to encode on the host.
//
// Every wait is bounded; on expiry the waiter raises the CTA's abort flag, the chain's abort word
// (so that the other CTAs stop polling) and the time-out bit of the device status word.  The last
// CTA to leave clears the control block, after an orderly run and after an aborted one alike.
#pragma once

#include <cuda_bf16.h>

#include "w4a8_ptx.cuh"
#include "w4a8_simple_kernels.cuh"
#include "w4a8_tiled_format.cuh"

namespace w4a8 {

constexpr int kChainMaxProblems = W4A8_CHAIN_MAX_PROBLEMS;
constexpr int kChainMaxM = W4A8_CHAIN_MAX_M;   // tokens per problem = MMA N
constexpr int kChainKindPlain = W4A8_CHAIN_INPUT_PLAIN;
constexpr int kChainKindSiluMul = W4A8_CHAIN_INPUT_SILU_MUL;
constexpr int kChainBlockRows = 96;            // rows of a block: tensor-memory lane quarters 0..2
constexpr int kChainMaxSegs = 8;               // segments per CTA and problem: up to 12 whole blocks + two runs of the remainder

// One problem of the chain as the kernel sees it (filled by the host).
struct ChainProblem {
    const uint16_t* x;          // BF16 [M][ldx]: the layer's input, or gate|up (2 K columns) for the gated kind
    const uint8_t* wpp;         // tiled weights
    const float* s_w;
    void* y;
    uint8_t* x8_out;            // optional row-major copies of what the quantization produced
    float* s_x_out;
    const float* static_scale;  // nullptr = dynamic per-token scale
    int64_t ldx, ldy, ldx8_out;
    int M, N, K;
    int kind;                   // kChainKind*
    int dep;                    // index of the earlier problem whose output this one reads, or -1
    int sw_stride, out_dtype, scale_mode;
    int rounds;                 // whole blocks per CTA: CTA p owns blocks [p * rounds, (p + 1) * rounds)
    int rem_blocks;             // blocks behind them, cut along K into runs of (block, k-block) items
    int rem_rot;                // the runs go to CTAs rem_rot, rem_rot + 1, ... (mod P): a different set for every problem
    int job_base;               // quantization job t = m * nch + c (row m, chunk c) runs on CTA (job_base + t) % gridDim.x
    int nch;                    // chunks a row is cut into for its quantization (1: a CTA takes a whole row)
    uint32_t x8_off;            // byte offsets into the workspace: FP8 activation tiles,
    uint32_t part_off;          //   partial-sum slots (one per CTA, M x 96 floats),
    uint32_t cnt_off;           //   arrival counters of the blocks that are cut along K
};

struct ChainParams {
    ChainProblem prob[kChainMaxProblems];
    int count;
    int S1;       // depth of the weight ring
    int wslot;    // bytes per weight-ring slot
    int stash;    // bytes of the row stash (quantization) = output staging area (epilogue)
    unsigned long long wait_limit_ns;
};

// Control block at the start of the workspace (zero-filled once by the caller, left zero by every launch).
struct ChainCtl {
    unsigned int exit_count;                  // CTAs that have left
    unsigned int abort;                       // a wait ran out somewhere: stop polling
    unsigned int pad[2];
    unsigned int xready[kChainMaxProblems];   // rows of problem i quantized and published
    unsigned int done[kChainMaxProblems];     // blocks of problem i whose rows of Y have been written
};
constexpr size_t kChainCtlBytes = 1024;
constexpr size_t kChainScaleBytes = (size_t)kChainMaxProblems * kChainMaxM * sizeof(float);
// header: control block, then per (problem, token): activation scale, row maximum under construction
// (float bits, combined with atomicMax by the CTAs that share a row) and the count of chunks whose
// maximum is in
constexpr size_t kChainHeaderBytes = 6144;
static_assert(sizeof(ChainCtl) <= kChainCtlBytes && kChainCtlBytes + 3 * kChainScaleBytes <= kChainHeaderBytes,
              "workspace header");
constexpr int kChainXTileBytes = kChainMaxM * 128;            // one k-block of FP8 activations: 16 tokens x 128 bytes

template <int G_, int FMT_, bool FULL_ = true>
struct ChainCfg {
    static constexpr int G = G_;          // expansion groups (three warps each: lane quarters 0..2)
    static constexpr int FMT = FMT_;
    // FULL: the gated input kind, and rows cut into chunks that several CTAs quantize
    // (ChainProblem::nch > 1).  Launches that need neither run an instantiation without that code:
    // compiled into the one kernel, the extra code of the quantization jobs cost them 2 % (measured;
    // the roles of a CTA share the instruction caches).
    static constexpr bool kFull = FULL_;
    static constexpr bool kChunk = FULL_;
    static constexpr int kS1Max = 16;     // weight ring (runtime depth <= this)
    static constexpr int kNAcc = 4;       // accumulator buffers (two blocks of 16 columns each): segments the MMAs may run ahead of the epilogue
    static constexpr int kS2 = kNAcc == 4 ? 6 : 7;   // stages of expanded weights in tensor memory = activation-tile slots
    static constexpr int kMeta = meta_bytes(FMT_);
    static constexpr int kRowBytes = row_bytes(FMT_);   // bytes of one row of one k-block in the weight buffer
    static constexpr int kAStageCols = 64;                    // two items of 32 columns
    static constexpr int kDCol = kS2 * kAStageCols;           // 448: accumulators behind the A ring
    static constexpr int kTmemCols = 512;
    static constexpr int kWarpRows = G_ + 1 > 4 ? G_ + 1 : 4; // rows of four warps (role table in the kernel)
    static constexpr int kThreads = 128 * kWarpRows;
    static constexpr int kBarBytes = 1024;
    static constexpr int kSegBytes = kChainMaxProblems * (kChainMaxSegs + 1) * 16;   // segment table of this CTA
    static constexpr int kXRingBytes = kS2 * 2 * kChainXTileBytes;
    static constexpr int kSmemMax = 226 * 1024;
    static_assert(kDCol + kNAcc * 2 * kChainMaxM <= kTmemCols, "tensor memory columns");
    static_assert((2 * kS1Max + 2 * kS2 + 2 * kNAcc + 1) * 8 + 64 <= kBarBytes, "barrier area");
    static_assert(G_ >= 2 && G_ <= 4 && G_ <= kS2, "expansion groups");
};

// Bounded acquire poll on a counter in global memory.
__device__ __forceinline__ bool chain_poll_ge(const unsigned int* flag, unsigned int target, unsigned int* gabort,
                                              volatile uint32_t* abort_flag, unsigned int* status_word,
                                              unsigned long long limit_ns) {
    if (ptx::ld_acquire_gpu(flag) >= target) return true;
    uint64_t t0 = 0;
    uint32_t spins = 0;
    while (true) {
        if (ptx::ld_acquire_gpu(flag) >= target) return true;
        __nanosleep(40);   // one poller per role and CTA, with a pause: the counter's L2 line is shared by every CTA
        if ((++spins & 15u) == 0u) {
            if (*abort_flag) return false;
            if (*reinterpret_cast<const volatile unsigned int*>(gabort)) {
                *abort_flag = 1u;  // another CTA gave up: this one stops too
                return false;
            }
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > limit_ns) {
                *abort_flag = 1u;
                atomicExch(gabort, 1u);
                atomicOr(status_word, kStatusTimeout);
                return false;
            }
        }
    }
}

// All 32 lanes of a converged warp agree on whether to go on (a wait can run out for some lanes
// and complete for others; the single-lane roles and the warp-collective tensor-memory stores
// need the whole warp on one path).
__device__ __forceinline__ bool warp_all(bool ok) { return __all_sync(0xFFFFFFFFu, ok) != 0; }

// The same for the 128 threads of the epilogue role (named barrier 3 with an OR reduction).
__device__ __forceinline__ bool epi_any(bool flag) {
    uint32_t r;
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 3, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}\n"
        : "=r"(r)
        : "r"((uint32_t)flag)
        : "memory");
    return r != 0;
}

// mbarrier wait that also raises the chain's abort word when it runs out.
__device__ __forceinline__ bool chain_mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                unsigned int* gabort, unsigned int* status_word,
                                                unsigned long long limit_ns) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    uint32_t spins = 0;
    while (true) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0u) {
            if (*abort_flag) return false;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > limit_ns) {
                *abort_flag = 1u;
                atomicExch(gabort, 1u);
                atomicOr(status_word, kStatusTimeout);
                return false;
            }
        }
    }
}

// ---- the work partition (shared by host and device) -------------------------------------------
// One segment of a CTA's share of a problem: NB blocks of up to 96 rows starting at row n0 (rows
// b * 96 .. of the segment form block b), k-blocks [kb0, kb0 + nkb).
struct ChainSeg {
    int n0;        // first row
    int blk;       // block index (first block of the segment)
    short R;       // rows (NB == 2: the first block has 96)
    short kb0, nkb;  // K range in k-blocks
    signed char NB;    // 1 or 2 blocks (two blocks share every activation tile)
    signed char part;  // -1: all of K, results go straight to Y; 0 / 1: partial sums into this CTA's slot 0 / 1
};
static_assert(sizeof(ChainSeg) == 16, "one 16-byte entry of the segment table");
__host__ __device__ inline int chain_blocks(int N) { return (N + kChainBlockRows - 1) / kChainBlockRows; }
// The items of the blocks that are cut along K are dealt out to Pr CTAs: the CTA with logical index
// l = (p - rem_rot) mod P < Pr takes items [l * items / Pr, (l + 1) * items / Pr), never an empty
// run.  Pr = min(P, items / 4): runs of at least four k-blocks keep the number of partial sums per
// block (which one CTA has to add up) small; but never fewer CTAs than blocks, so that a run is at
// most K/128 items long and touches at most two blocks.  rem_rot moves on from problem to problem
// (the host sets it), so that the extra work and the adding-up do not always fall on the same CTAs.
constexpr int kChainMinRun = 4;
__host__ __device__ inline long long chain_rem_lo(int l, int Pr, long long items) { return (long long)l * items / Pr; }
__host__ __device__ inline int chain_rem_ctas(const ChainProblem& q, int P) {
    const long long items = (long long)q.rem_blocks * (q.K >> 7);
    long long pr = items / kChainMinRun;
    if (pr > P) pr = P;
    if (pr < q.rem_blocks) pr = q.rem_blocks;
    return (int)pr;
}
__host__ __device__ inline int chain_rem_logical(const ChainProblem& q, int p, int P) { return (p + P - q.rem_rot % P) % P; }
__host__ __device__ inline int chain_rem_physical(const ChainProblem& q, int l, int P) { return (l + q.rem_rot) % P; }
// Number of segments of CTA p for this problem.
__host__ __device__ inline int chain_num_segs(const ChainProblem& q, int p, int P) {
    int n = (q.rounds + 1) / 2;
    const int Pr = chain_rem_ctas(q, P);
    const int l = chain_rem_logical(q, p, P);
    if (l < Pr) {
        const int KB = q.K >> 7;
        const long long items = (long long)q.rem_blocks * KB;
        const long long lo = chain_rem_lo(l, Pr, items), hi = chain_rem_lo(l + 1, Pr, items);
        n += ((hi - 1) / KB > lo / KB) ? 2 : 1;
    }
    return n;
}
// Segment j of CTA p.  The CTA's run of the blocks that are cut along K comes FIRST, its whole blocks
// after it: the hand-over of partial sums and the adding-up then overlap the whole blocks' MMAs
// instead of standing at the end of the problem, where a dependent problem waits for them.
// (nsegs = chain_num_segs(q, p, P), passed in: it costs 64-bit divisions)
__host__ __device__ inline ChainSeg chain_seg(const ChainProblem& q, int p, int P, int j, int nsegs) {
    ChainSeg s;
    const int KB = q.K >> 7;
    const int full_segs = (q.rounds + 1) / 2;
    const int rem_segs = nsegs - full_segs;
    if (j >= rem_segs) {
        j -= rem_segs;
        const int b0 = p * q.rounds + 2 * j;
        s.NB = (signed char)((q.rounds - 2 * j) < 2 ? 1 : 2);
        s.blk = b0;
        s.n0 = b0 * kChainBlockRows;
        const int rows = s.NB * kChainBlockRows;
        s.R = (short)((q.N - s.n0) < rows ? (q.N - s.n0) : rows);
        s.kb0 = 0;
        s.nkb = (short)KB;
        s.part = -1;
        return s;
    }
    const int Pr = chain_rem_ctas(q, P);
    const int l = chain_rem_logical(q, p, P);
    const long long items = (long long)q.rem_blocks * KB;
    const long long lo = chain_rem_lo(l, Pr, items), hi = chain_rem_lo(l + 1, Pr, items);
    const int br0 = (int)(lo / KB);
    const long long cut = (long long)(br0 + 1) * KB;
    const int jj = j;
    const long long a = jj == 0 ? lo : cut, b = jj == 0 ? (hi < cut ? hi : cut) : hi;
    const int br = br0 + jj;
    s.NB = 1;
    s.blk = P * q.rounds + br;
    s.n0 = s.blk * kChainBlockRows;
    s.R = (short)((q.N - s.n0) < kChainBlockRows ? (q.N - s.n0) : kChainBlockRows);
    s.kb0 = (short)(a - (long long)br * KB);
    s.nkb = (short)(b - a);
    s.part = (signed char)((s.nkb == KB) ? -1 : jj);
    return s;
}
// The CTAs (logical indices) that contribute partial sums to remainder block br: first .. last, every
// one of them.  (lo(l) <= a  <=>  l < (a + 1) Pr / items, so the one that holds item a is
// ceil((a + 1) Pr / items) - 1.)
__host__ __device__ inline void chain_block_owners(const ChainProblem& q, int P, int br, int* first, int* last) {
    const int KB = q.K >> 7;
    const int Pr = chain_rem_ctas(q, P);
    const long long items = (long long)q.rem_blocks * KB;
    const long long a = (long long)br * KB, b = a + KB;    // the block's items: a .. b - 1
    *first = (int)(((a + 1) * Pr + items - 1) / items) - 1;
    *last = (int)((b * Pr + items - 1) / items) - 1;
}

// Adds the partial sums of contributors first + 1 .. last (logical indices; slot of the physical CTA,
// token-major, 96 floats per token, this thread's row at `row`) onto res, in ascending contributor
// order.  CB contributors x 32 / CB tokens are in flight at a time (32 independent loads per thread:
// the round trips to L2 are what the adding CTA waits for).
template <int CB>
__device__ __forceinline__ void chain_add_partials(float (&res)[16], const ChainProblem& q, const float* parts,
                                                   size_t slot_floats, int row, int first, int last, int P) {
    constexpr int TB = 32 / CB;   // tokens per batch
#pragma unroll
    for (int t0 = 0; t0 < 16; t0 += TB) {
        if (t0 >= q.M) break;   // uniform
#pragma unroll 1
        for (int c0 = first + 1; c0 <= last; c0 += CB) {
            float w[CB][TB];
#pragma unroll
            for (int cc = 0; cc < CB; ++cc) {
                const int c = c0 + cc;
                const float* src = parts + (size_t)chain_rem_physical(q, c <= last ? c : last, P) * slot_floats + row;
#pragma unroll
                for (int jj = 0; jj < TB; ++jj)
                    w[cc][jj] = (c <= last && t0 + jj < q.M) ? __ldcg(src + (t0 + jj) * kChainBlockRows) : 0.0f;
            }
#pragma unroll
            for (int cc = 0; cc < CB; ++cc)
#pragma unroll
                for (int jj = 0; jj < TB; ++jj) res[t0 + jj] += w[cc][jj];
        }
    }
}

template <class Cfg>
__global__ void __launch_bounds__(Cfg::kThreads, 1)
linear_chain_kernel(const __grid_constant__ ChainParams prm, uint8_t* __restrict__ ws, unsigned int* status_word) {
    constexpr int G = Cfg::G, S2 = Cfg::kS2, MB = Cfg::kMeta, S1M = Cfg::kS1Max;
    constexpr int BR = kChainBlockRows;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw_addr);

    const int S1 = prm.S1;
    const uint32_t x_ring = base;                                            // [S2][2][2 KB], 1 KB aligned
    const uint32_t w_ring = x_ring + (uint32_t)Cfg::kXRingBytes;             // [S1][wslot]
    const uint32_t stash_off = (uint32_t)Cfg::kXRingBytes + (uint32_t)(S1 * prm.wslot);
    const uint32_t stash_s = base + stash_off;                               // row stash / output staging
    const uint32_t bars_off = stash_off + (uint32_t)prm.stash;
    const uint32_t bars_addr = base + bars_off;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + bars_off);
    const uint32_t bar_wfull0 = bars_addr;                                   // [S1M] packed codes + meta landed
    const uint32_t bar_wfree0 = bars_addr + 8u * S1M;                        // [S1M] expanded: slot may be refilled
    const uint32_t bar_afull0 = bars_addr + 8u * (2 * S1M);                  // [S2]  stage ready: weights expanded into tensor memory, activation tiles landed
    const uint32_t bar_afree0 = bar_afull0 + 8u * S2;                        // [S2]  stage consumed by the MMAs
    constexpr int NA = Cfg::kNAcc;
    const uint32_t bar_accfull0 = bar_afree0 + 8u * S2;                      // [NA]
    const uint32_t bar_accempty0 = bar_accfull0 + 8u * NA;                   // [NA]
    const uint32_t bar_drain = bar_accempty0 + 8u * NA;
    constexpr int kNumBars = 2 * S1M + 2 * S2 + 2 * NA + 1;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + kNumBars);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float* red_s = reinterpret_cast<float*>(const_cast<uint32_t*>(tmem_slot) + 4);   // [4] warp maxima of a quantization job, [1] the row's maximum
    // This CTA's segments of every problem, worked out once (the partition needs 64-bit divisions,
    // which cost a single warp microseconds per problem if every role repeats them).
    const ChainSeg* seg_tab = reinterpret_cast<const ChainSeg*>(sm + bars_off + Cfg::kBarBytes);   // [problem][kChainMaxSegs]
    const int* nseg_tab = reinterpret_cast<const int*>(sm + bars_off + Cfg::kBarBytes + kChainMaxProblems * kChainMaxSegs * 16);

    ChainCtl* const ctl = reinterpret_cast<ChainCtl*>(ws);
    float* const sx_ws = reinterpret_cast<float*>(ws + kChainCtlBytes);      // [problem][16] activation scales
    unsigned int* const amax_ws = reinterpret_cast<unsigned int*>(ws + kChainCtlBytes + kChainScaleBytes);       // [problem][16]
    unsigned int* const qcnt_ws = reinterpret_cast<unsigned int*>(ws + kChainCtlBytes + 2 * kChainScaleBytes);   // [problem][16]
    unsigned int* const gabort = &ctl->abort;
    const unsigned long long limit = prm.wait_limit_ns;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Roles.  Warp w runs on SM sub-partition w % 4 and may access tensor-memory lane quarter w % 4.
    // Quarters 0..2 hold the 96 rows of a block; the warps with a single issuing lane -- whose bulk
    // copies and MMAs cost their sub-partition tens of cycles each -- all sit on sub-partition 3,
    // away from the expansion work.
    //   row 0: epilogue quarters 0..2 | MMA issuer          row 1: expansion group 0 | epilogue quarter 3 (no rows)
    //   row 2: expansion group 1 | weight loader            row 3: expansion group 2 | activation-tile loader
    //   row 4: expansion group 3 | -
    const int wq = warp & 3, wr = warp >> 2;
    const bool is_mma = wq == 3 && wr == 0;
    const bool is_wload = wq == 3 && wr == 2;
    const bool is_xload = wq == 3 && wr == 3;
    const bool is_epi = (wq < 3 && wr == 0) || (wq == 3 && wr == 1);
    const bool is_dq = wq < 3 && wr >= 1 && wr <= G;
    const int p = blockIdx.x, P = gridDim.x;
    const int count = prm.count;

    if (threadIdx.x == 32) {
        for (int s = 0; s < S1; ++s) {
            ptx::mbar_init(bar_wfull0 + 8u * s, 1);
            ptx::mbar_init(bar_wfree0 + 8u * s, 96);
        }
        for (int s = 0; s < S2; ++s) {
            ptx::mbar_init(bar_afull0 + 8u * s, 96 + 1);   // the expanding threads + the activation loader (with its byte count)
            ptx::mbar_init(bar_afree0 + 8u * s, 1);
        }
        for (int b = 0; b < NA; ++b) {
            ptx::mbar_init(bar_accfull0 + 8u * b, 1);
            ptx::mbar_init(bar_accempty0 + 8u * b, 128);
        }
        ptx::mbar_init(bar_drain, 1);
        *abort_flag = 0u;
        ptx::fence_mbar_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), Cfg::kTmemCols);
        ptx::tmem_relinquish();
    }
    if (threadIdx.x >= 64 && threadIdx.x < 64 + (unsigned)count) {
        const int i = (int)threadIdx.x - 64;
        const ChainProblem& q = prm.prob[i];
        const int n = chain_num_segs(q, p, P);
        const_cast<int*>(nseg_tab)[i] = n;
        for (int j = 0; j < n; ++j) const_cast<ChainSeg*>(seg_tab)[i * kChainMaxSegs + j] = chain_seg(q, p, P, j, n);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    ptx::griddep_launch_dependents();

    if (is_wload) {
        // ------------------------------------------------------------------ weight loader (one lane issues)
        bool ok = true;
        ptx::Ring r1;
        int issued = 0;
        for (int i = 0; i < count && ok; ++i) {
            const ChainProblem& q = prm.prob[i];
            const int nseg = nseg_tab[i];
            const int KB = q.K >> 7;
            constexpr int RBY = Cfg::kRowBytes;
            const int64_t code_step = (int64_t)q.N * RBY;   // one k-block further
            const int64_t meta_step = (int64_t)q.N * MB;
            for (int j = 0; j < nseg && ok; ++j) {
                const ChainSeg sg = seg_tab[i * kChainMaxSegs + j];
                const int KS = 2 / sg.NB;
                const uint32_t cbytes = (uint32_t)(sg.R * RBY), mbytes = (uint32_t)(sg.R * MB);
                const uint8_t* cptr = q.wpp + (int64_t)sg.kb0 * code_step + (int64_t)sg.n0 * RBY;
                const uint8_t* mptr = q.wpp + (int64_t)KB * code_step + (int64_t)sg.kb0 * meta_step + (int64_t)sg.n0 * MB;
                const uint32_t meta_off = (uint32_t)KS * cbytes;
                for (int kb = 0; kb < sg.nkb;) {
                    ok = warp_all(chain_mbar_wait(bar_wfree0 + 8u * (uint32_t)r1.idx, r1.phase ^ 1u, abort_flag, gabort,
                                                  status_word, limit));
                    if (!ok) break;
                    const int ks = (sg.nkb - kb) < KS ? (sg.nkb - kb) : KS;
                    const uint32_t full = bar_wfull0 + 8u * (uint32_t)r1.idx;
                    const uint32_t wdst = w_ring + (uint32_t)(r1.idx * prm.wslot);
                    const uint32_t mdst = wdst + meta_off;
                    const uint8_t* cptr1 = cptr + code_step;
                    const uint8_t* mptr1 = mptr + meta_step;
                    if (ptx::elect_one()) {
                        ptx::mbar_arrive_expect_tx(full, (uint32_t)ks * (cbytes + mbytes));
                        ptx::bulk_load(wdst, cptr, cbytes, full);
                        if (MB > 0) ptx::bulk_load(mdst, mptr, mbytes, full);
                        if (ks == 2) {
                            ptx::bulk_load(wdst + cbytes, cptr1, cbytes, full);
                            if (MB > 0) ptx::bulk_load(mdst + mbytes, mptr1, mbytes, full);
                        }
                    }
                    cptr += code_step * ks;
                    mptr += meta_step * ks;
                    kb += ks;
                    r1.advance(S1);
                    ++issued;
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
                const uint64_t t0 = ptx::globaltimer_ns();
                while (!ptx::mbar_try_wait(bar_wfull0 + 8u * (uint32_t)rb.idx, rb.phase) &&
                       ptx::globaltimer_ns() - t0 < limit) {
                }
            }
        }
        __syncwarp();
    } else if (is_mma) {
        // ------------------------------------------------------------------ MMA issuer (one lane issues)
        bool ok = true;
        ptx::Ring r2;
        int nacc = 0;
        const uint32_t b_lo0 = ptx::umma_desc_lo(x_ring);
        constexpr uint32_t b_step = (uint32_t)(2 * kChainXTileBytes) >> 4;
        constexpr uint32_t idesc = ptx::umma_idesc_e4m3_f32(128, kChainMaxM);
        for (int i = 0; i < count && ok; ++i) {
            const ChainProblem& q = prm.prob[i];
            const int nseg = nseg_tab[i];
            for (int j = 0; j < nseg && ok; ++j) {
                const ChainSeg sg = seg_tab[i * kChainMaxSegs + j];
                const int buf = nacc % NA;
                if (nacc >= NA) {
                    ok = warp_all(chain_mbar_wait(bar_accempty0 + 8u * (uint32_t)buf, (uint32_t)(nacc / NA - 1) & 1u,
                                                  abort_flag, gabort, status_word, limit));
                    if (!ok) break;
                }
                const uint32_t d0 = tmem_base + (uint32_t)(Cfg::kDCol + buf * 2 * kChainMaxM);
                const bool two_blocks = sg.NB == 2;
                // A stage holds two (k-block, block) items: two k-blocks of one block (the last stage
                // of an odd K range holds one), or one k-block of two blocks.
                const int nst = two_blocks ? sg.nkb : (sg.nkb + 1) >> 1;
                const bool odd_tail = !two_blocks && (sg.nkb & 1);
                const uint32_t d1 = two_blocks ? d0 + (uint32_t)kChainMaxM : d0;
                const uint32_t b_off1 = two_blocks ? 0u : ((uint32_t)kChainXTileBytes >> 4);
                uint32_t accumulate = 0;
                for (int st = 0; st < nst; ++st) {
                    ok = warp_all(chain_mbar_wait(bar_afull0 + 8u * (uint32_t)r2.idx, r2.phase, abort_flag, gabort,
                                                  status_word, limit));
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t b_lo = b_lo0 + (uint32_t)r2.idx * b_step;
                    const uint32_t a_col = tmem_base + (uint32_t)(r2.idx * Cfg::kAStageCols);
                    const bool second = !(odd_tail && st + 1 == nst);
                    const uint32_t acc1 = two_blocks ? accumulate : 1u;
                    if (ptx::elect_one()) {
                        ptx::umma_f8_kblock_ts(d0, a_col, b_lo, idesc, accumulate);
                        if (second) ptx::umma_f8_kblock_ts(d1, a_col + 32u, b_lo + b_off1, idesc, acc1);
                        ptx::umma_commit(bar_afree0 + 8u * (uint32_t)r2.idx);  // frees the expanded stage and its activation tiles
                    }
                    accumulate = 1u;
                    r2.advance(S2);
                }
                if (!ok) break;
                if (ptx::elect_one()) ptx::umma_commit(bar_accfull0 + 8u * (uint32_t)buf);
                ++nacc;
            }
        }
        if (!ok && lane == 0) {
            // Gave up: wait (bounded) for the MMAs already issued before tensor memory is freed.
            ptx::umma_commit(bar_drain);
            const uint64_t t0 = ptx::globaltimer_ns();
            while (!ptx::mbar_try_wait(bar_drain, 0u) && ptx::globaltimer_ns() - t0 < limit) {
            }
        }
        __syncwarp();
    } else if (is_xload) {
        // ------------------------------------------------------------------ activation-tile loader (one lane issues)
        bool ok = true;
        ptx::Ring r2;
        int issued = 0;
        ptx::griddep_wait();  // the workspace and the counters belong to the previous launch until it has completed
        for (int i = 0; i < count && ok; ++i) {
            const ChainProblem& q = prm.prob[i];
            const int nseg = nseg_tab[i];
            if (nseg == 0) continue;
            // the problem's activations must have been quantized (by the epilogue warps of M CTAs)
            if (lane == 0)
                ok = chain_poll_ge(&ctl->xready[i], (unsigned)(Cfg::kChunk ? q.M * q.nch : q.M), gabort, abort_flag,
                                   status_word, limit);
            ok = warp_all(ok);
            __syncwarp();
            if (!ok) break;
            // (lane 0 made the acquire; the warp barrier orders the other lanes behind it, and whichever lane is
            // elected to issue fences the quantizers' writes before its own bulk copies)
            asm volatile("fence.proxy.async.global;" ::: "memory");
            const uint8_t* xt = ws + q.x8_off;
            const uint32_t rows_bytes = (uint32_t)q.M * 128u;         // the token rows are the first M rows of a tile
            for (int j = 0; j < nseg && ok; ++j) {
                const ChainSeg sg = seg_tab[i * kChainMaxSegs + j];
                const int KS = 2 / sg.NB;
                for (int kb = 0; kb < sg.nkb;) {
                    ok = warp_all(chain_mbar_wait(bar_afree0 + 8u * (uint32_t)r2.idx, r2.phase ^ 1u, abort_flag, gabort,
                                                  status_word, limit));
                    if (!ok) break;
                    const int ks = (sg.nkb - kb) < KS ? (sg.nkb - kb) : KS;
                    const uint32_t full = bar_afull0 + 8u * (uint32_t)r2.idx;
                    const uint32_t xdst = x_ring + (uint32_t)(r2.idx * 2 * kChainXTileBytes);
                    const uint8_t* src = xt + (int64_t)(sg.kb0 + kb) * kChainXTileBytes;
                    if (ptx::elect_one()) {
                        ptx::mbar_arrive_expect_tx(full, (uint32_t)ks * rows_bytes);
                        ptx::bulk_load(xdst, src, rows_bytes, full);
                        if (ks == 2) ptx::bulk_load(xdst + (uint32_t)kChainXTileBytes, src + kChainXTileBytes, rows_bytes, full);
                    }
                    kb += ks;
                    r2.advance(S2);
                    ++issued;
                }
            }
        }
        if (!ok && lane == 0) {
            ptx::Ring rb = r2;
            const int n = issued < S2 ? issued : S2;
            for (int i = 0; i < n; ++i) {
                if (--rb.idx < 0) {
                    rb.idx = S2 - 1;
                    rb.phase ^= 1u;
                }
                const uint64_t t0 = ptx::globaltimer_ns();
                while (!ptx::mbar_try_wait(bar_afull0 + 8u * (uint32_t)rb.idx, rb.phase) &&
                       ptx::globaltimer_ns() - t0 < limit) {
                }
            }
        }
        __syncwarp();
    } else if (is_epi) {
        // ------------------------------------------------------------------ quantization jobs + epilogue
        const int qd = wq;                       // tensor-memory lane quarter
        const int r = qd * 32 + lane;            // lane of the accumulator = row within a block (rows 0..95)
        const int et = r;                        // index among the 128 threads of this role
        bool ok = true;
        ptx::griddep_wait();

        // Eq. 13 for chunk c of row m of problem j: absmax, scale, FP8 codes written as operand tiles
        // into the workspace, then published.  A row is one chunk, or -- long rows, above all the
        // gated kind, whose silu costs the 128 threads of a lone CTA tens of microseconds -- nch
        // chunks on nch CTAs, which combine their maxima through the workspace (atomicMax on the
        // float bits, a count of the chunks that are in, one bounded poll) before any of them
        // converts.  That wait cannot deadlock: a chunk's maximum is published before anything is
        // waited for, and every CTA reaches the jobs of a problem in the same order.  Called by all
        // 128 threads.
        auto quant_job = [&](int j, int m, int c) -> bool {
            const ChainProblem& q = prm.prob[j];
            bool good = true;
            if (q.dep >= 0) {
                if (et == 0)
                    good = chain_poll_ge(&ctl->done[q.dep], (unsigned)chain_blocks(prm.prob[q.dep].N), gabort,
                                         abort_flag, status_word, limit);
                if (epi_any(!good)) return false;   // (also the barrier behind which every thread may read the input)
            }
            const int K = q.K;
            const int nunits = K >> 4;  // 16 elements: 32 bytes of BF16 in, 16 bytes of FP8 out
            const uint16_t* xrow = q.x + (int64_t)m * q.ldx;
            int u_lo = 0, u_hi = nunits;
            if constexpr (Cfg::kChunk) {
                const int upc = (nunits + q.nch - 1) / q.nch;
                u_lo = c * upc;
                u_hi = (u_lo + upc) < nunits ? (u_lo + upc) : nunits;
            }
            float amax = 0.0f;
            for (int u = u_lo + et; u < u_hi; u += 128) {
                uint4 a, b;
                if (Cfg::kFull && q.kind == kChainKindSiluMul) {
                    const uint4* gp = reinterpret_cast<const uint4*>(xrow) + 2 * u;
                    const uint4* up = reinterpret_cast<const uint4*>(xrow + K) + 2 * u;
                    const uint4 g0 = __ldcg(gp), g1 = __ldcg(gp + 1), u0 = __ldcg(up), u1 = __ldcg(up + 1);
                    a.x = silu_mul_bf16x2(g0.x, u0.x);
                    a.y = silu_mul_bf16x2(g0.y, u0.y);
                    a.z = silu_mul_bf16x2(g0.z, u0.z);
                    a.w = silu_mul_bf16x2(g0.w, u0.w);
                    b.x = silu_mul_bf16x2(g1.x, u1.x);
                    b.y = silu_mul_bf16x2(g1.y, u1.y);
                    b.z = silu_mul_bf16x2(g1.z, u1.z);
                    b.w = silu_mul_bf16x2(g1.w, u1.w);
                } else {
                    const uint4* xp = reinterpret_cast<const uint4*>(xrow) + 2 * u;
                    a = __ldcg(xp);
                    b = __ldcg(xp + 1);
                }
                amax = absmax_bf16x8(a, amax);
                amax = absmax_bf16x8(b, amax);
                ptx::st_shared_v4(stash_s + (uint32_t)(u - u_lo) * 32u, a);
                ptx::st_shared_v4(stash_s + (uint32_t)(u - u_lo) * 32u + 16u, b);
            }
            float s, inv;
            if (q.static_scale != nullptr) {
                s = __ldg(q.static_scale);
                inv = __fdiv_rn(1.0f, s);
            } else {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
                if (lane == 0) red_s[qd] = amax;
                asm volatile("bar.sync 3, 128;" ::: "memory");
                amax = fmaxf(fmaxf(red_s[0], red_s[1]), fmaxf(red_s[2], red_s[3]));
                if constexpr (Cfg::kChunk) {
                    if (q.nch > 1) {
                        unsigned int* am = amax_ws + j * kChainMaxM + m;
                        unsigned int* qc = qcnt_ws + j * kChainMaxM + m;
                        if (et == 0) {
                            atomicMax(am, __float_as_uint(amax));   // non-negative floats order like their bit patterns
                            ptx::red_release_add(qc, 1u);
                            good = chain_poll_ge(qc, (unsigned)q.nch, gabort, abort_flag, status_word, limit);
                            red_s[4] = __uint_as_float(ptx::ld_acquire_gpu(am));
                        }
                        if (epi_any(!good)) return false;
                        amax = red_s[4];
                    }
                }
                if (amax == 0.0f) {
                    s = 1.0f;
                    inv = 1.0f;
                } else if (q.scale_mode == W4A8_SCALE_POW2) {
                    s = pow2_ceil(__fdiv_rn(amax, kE4M3Max));
                    inv = __fdiv_rn(1.0f, s);
                } else {
                    s = __fdiv_rn(amax, kE4M3Max);
                    inv = __fdiv_rn(kE4M3Max, amax);
                }
            }
            uint8_t* tiles = ws + q.x8_off;
            for (int u = u_lo + et; u < u_hi; u += 128) {
                uint4 a, b;
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w)
                             : "r"(stash_s + (uint32_t)(u - u_lo) * 32u));
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w)
                             : "r"(stash_s + (uint32_t)(u - u_lo) * 32u + 16u));
                const uint2 qa = quant_bf16x8(a, inv), qb = quant_bf16x8(b, inv);
                const uint4 o = make_uint4(qa.x, qa.y, qb.x, qb.y);
                // operand tile of k-block u / 8: token m is row m, its 16-byte chunk c sits at c ^ (m & 7)
                const int kb = u >> 3, ck = u & 7;
                *reinterpret_cast<uint4*>(tiles + (int64_t)kb * kChainXTileBytes + m * 128 + ((ck ^ (m & 7)) << 4)) = o;
                if (q.x8_out != nullptr)
                    *reinterpret_cast<uint4*>(q.x8_out + (int64_t)m * q.ldx8_out + (int64_t)u * 16) = o;
            }
            if (et == 0 && c == 0) {
                sx_ws[j * kChainMaxM + m] = s;
                if (q.s_x_out != nullptr) q.s_x_out[m] = s;
            }
            asm volatile("bar.sync 3, 128;" ::: "memory");   // every thread's tiles are out (and the stash may be reused)
            if (et == 0) ptx::red_release_add(&ctl->xready[j], 1u);
            return true;
        };
        auto my_job = [&](const ChainProblem& q) {
            // the quantization job (row * nch + chunk) of problem q that this CTA runs, or -1
            const int t = (int)(((unsigned)p + (unsigned)P - (unsigned)q.job_base % (unsigned)P) % (unsigned)P);
            return t < (Cfg::kChunk ? q.M * q.nch : q.M) ? t : -1;
        };
        // Cast and store of the M tokens of one block of up to 96 rows whose scaled sums this thread
        // holds in res (its row: lane r of the accumulator); through the staging area in 16-byte
        // pieces when the rows of Y are 16-byte aligned.  Called by all 128 threads.
        auto emit_block = [&](const ChainProblem& q, const float (&res)[16], int n0b, int Rb) {
            const int es = q.out_dtype == W4A8_OUT_FP32 ? 4 : 2;
            const bool wide_out = (((int64_t)q.ldy * es) & 15) == 0;  // rows of Y 16-byte aligned
            const uint32_t pitch = (uint32_t)(BR * es);
            if (r < BR) {
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) {
                    const uint32_t a = stash_s + (uint32_t)jj * pitch + (uint32_t)(r * es);
                    if (es == 4)
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(res[jj]) : "memory");
                    else
                        asm volatile("st.shared.u16 [%0], %1;" ::"r"(a),
                                     "h"(__bfloat16_as_ushort(__float2bfloat16_rn(res[jj])))
                                     : "memory");
                }
            }
            asm volatile("bar.sync 3, 128;" ::: "memory");
            char* yb = static_cast<char*>(q.y) + (int64_t)n0b * es;
            if (wide_out) {
                const int ppt = (Rb * es) >> 4;  // 16-byte pieces per token (rows come in eights)
                for (int id = et; id < q.M * ppt; id += 128) {
                    const int tok = id / ppt, piece = id - tok * ppt;
                    uint4 w;
                    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w)
                                 : "r"(stash_s + (uint32_t)tok * pitch + (uint32_t)(piece << 4)));
                    *reinterpret_cast<uint4*>(yb + (int64_t)tok * q.ldy * es + (piece << 4)) = w;
                }
            } else {
                // rows of Y that are not 16-byte aligned: the same staged values, two bytes at a time
                const int ppt = (Rb * es) >> 1;
                for (int id = et; id < q.M * ppt; id += 128) {
                    const int tok = id / ppt, piece = id - tok * ppt;
                    uint16_t w;
                    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(w) : "r"(stash_s + (uint32_t)tok * pitch + (uint32_t)(piece << 1)));
                    *reinterpret_cast<uint16_t*>(yb + (int64_t)tok * q.ldy * es + (piece << 1)) = w;
                }
            }
            asm volatile("bar.sync 3, 128;" ::: "memory");  // before the area is written again
        };

        // problems whose input exists before the launch: quantized right away, by M CTAs each
        for (int j = 0; j < count && ok; ++j) {
            const ChainProblem& q = prm.prob[j];
            if (q.dep >= 0) continue;
            const int t = my_job(q);
            if (t >= 0) ok = Cfg::kChunk ? quant_job(j, t / q.nch, t % q.nch) : quant_job(j, t, 0);
        }

        int nacc = 0;
        // "Activations ready" and the scales of the NEXT problem are looked up while this problem's
        // first accumulator is awaited: two L2 round trips per problem that would otherwise sit in
        // front of every problem's first segment (the epilogue warps are what paces short problems).
        bool pre_seen = false;    // this thread saw the next problem's activations complete ...
        float pre_sx = 0.0f;      // ... and read its lane's scale behind that acquire
        for (int i = 0; i < count && ok; ++i) {
            const ChainProblem& q = prm.prob[i];
            const int nseg = nseg_tab[i];
            float sx_mine = 0.0f;
            if (nseg > 0) {
                // every thread must have seen it (they take the same path: named barriers below)
                if (!epi_any(!pre_seen)) {
                    sx_mine = pre_sx;
                } else {
                    // the scales were published together with the tiles the MMAs consume
                    if (et == 0)
                        ok = chain_poll_ge(&ctl->xready[i], (unsigned)(Cfg::kChunk ? q.M * q.nch : q.M), gabort,
                                           abort_flag, status_word, limit);
                    ok = !epi_any(!ok);   // (the barrier orders the other threads behind thread 0's acquire)
                    if (!ok) break;
                    sx_mine = (lane < q.M) ? __ldcg(sx_ws + i * kChainMaxM + lane) : 0.0f;
                }
            }
            pre_seen = false;
            for (int j = 0; j < nseg && ok; ++j) {
                const ChainSeg sg = seg_tab[i * kChainMaxSegs + j];
                const int buf = nacc % NA;
                if (j == 0 && i + 1 < count && nseg_tab[i + 1] > 0) {
                    const ChainProblem& qn = prm.prob[i + 1];
                    pre_seen = ptx::ld_acquire_gpu(&ctl->xready[i + 1]) >= (unsigned)(Cfg::kChunk ? qn.M * qn.nch : qn.M);
                    pre_sx = (lane < qn.M) ? __ldcg(sx_ws + (i + 1) * kChainMaxM + lane) : 0.0f;
                }
                float swn[2];
#pragma unroll
                for (int b = 0; b < 2; ++b)
                    swn[b] = (sg.part < 0 && b < sg.NB && r < BR && b * BR + r < sg.R)
                                 ? __ldg(q.s_w + (int64_t)(sg.n0 + b * BR + r) * q.sw_stride)
                                 : 0.0f;
                ok = chain_mbar_wait(bar_accfull0 + 8u * (uint32_t)buf, (uint32_t)(nacc / NA) & 1u, abort_flag, gabort,
                                     status_word, limit);
                ok = !epi_any(!ok);   // all 128 threads take the same path (they meet at named barriers below)
                if (!ok) break;
                ptx::tc_fence_after_sync();
                if (sg.part < 0) {
#pragma unroll 1   // (one copy of the block's code: the roles of a CTA share the instruction caches)
                    for (int b = 0; b < 2; ++b) {
                        if (b >= sg.NB) break;
                        uint32_t v[16];
                        ptx::tmem_ld_32x32b_x16(tmem_base + ((uint32_t)(qd * 32) << 16) +
                                                    (uint32_t)(Cfg::kDCol + buf * 2 * kChainMaxM + b * kChainMaxM),
                                                v);
                        ptx::tmem_ld_wait();
                        float res[16];
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            const float sxm = __shfl_sync(0xFFFFFFFFu, sx_mine, jj);
                            res[jj] = __uint_as_float(v[jj]) * (sxm * (b == 0 ? swn[0] : swn[1]));  // Eq. 4, Eq. 11
                        }
                        const int Rb = (sg.R - b * BR) < BR ? (sg.R - b * BR) : BR;
                        emit_block(q, res, sg.n0 + b * BR, Rb);
                    }
                    ptx::tc_fence_before_sync();
                    ptx::mbar_arrive(bar_accempty0 + 8u * (uint32_t)buf);
                    ++nacc;
                    // this CTA's rows of Y are written: publish (the barrier orders every thread's stores
                    // before the release)
                    asm volatile("bar.sync 3, 128;" ::: "memory");
                    if (et == 0) ptx::red_release_add(&ctl->done[i], (unsigned)sg.NB);
                } else {
                    // A block that is cut along K.  The CTA that holds the lowest k range adds up: it is
                    // the one that reaches the block last (in the second part of its run, the others in
                    // the first part of theirs).  The others write their partial sums (token-major, 96
                    // floats per token) to their first slot and count themselves in; the adding CTA
                    // waits (bounded) for their count, then adds in ascending k order -- a fixed order.
                    uint32_t v[16];
                    ptx::tmem_ld_32x32b_x16(tmem_base + ((uint32_t)(qd * 32) << 16) +
                                                (uint32_t)(Cfg::kDCol + buf * 2 * kChainMaxM),
                                            v);
                    ptx::tmem_ld_wait();
                    ptx::tc_fence_before_sync();
                    ptx::mbar_arrive(bar_accempty0 + 8u * (uint32_t)buf);
                    ++nacc;
                    const size_t slot_floats = (size_t)q.M * BR;
                    float* parts = reinterpret_cast<float*>(ws + q.part_off);
                    const int br = sg.blk - P * q.rounds;
                    unsigned int* cnt = reinterpret_cast<unsigned int*>(ws + q.cnt_off) + br;
                    int first, last;
                    chain_block_owners(q, P, br, &first, &last);
                    const bool adder = chain_rem_logical(q, p, P) == first;
                    // (the adding CTA fetches its weight scale before it waits for the others)
                    const float sw = (adder && r < sg.R) ? __ldg(q.s_w + (int64_t)(sg.n0 + r) * q.sw_stride) : 0.0f;
                    if (!adder) {
                        float* mine = parts + (size_t)p * slot_floats;
                        if (r < BR) {
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj)
                                if (jj < q.M) __stcg(mine + jj * BR + r, __uint_as_float(v[jj]));
                        }
                        asm volatile("bar.sync 3, 128;" ::: "memory");
                        if (et == 0) ptx::red_release_add(cnt, 1u);   // every thread's stores are ordered before it
                    } else {
                        if (et == 0)
                            ok = chain_poll_ge(cnt, (unsigned)(last - first), gabort, abort_flag, status_word, limit);
                        ok = !epi_any(!ok);
                        if (!ok) break;
                        float res[16];
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) res[jj] = __uint_as_float(v[jj]);
                        if (r < sg.R) {
                            chain_add_partials<4>(res, q, parts, slot_floats, r, first, last, P);
                        }
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            const float sxm = __shfl_sync(0xFFFFFFFFu, sx_mine, jj);
                            res[jj] = res[jj] * (sxm * sw);  // Eq. 4, Eq. 11
                        }
                        emit_block(q, res, sg.n0, sg.R);
                        asm volatile("bar.sync 3, 128;" ::: "memory");
                        if (et == 0) {
                            *cnt = 0u;   // ready for the next launch
                            ptx::red_release_add(&ctl->done[i], 1u);
                        }
                    }
                }
            }
            // problems that read the output of problem i: quantize this CTA's row of them now
            for (int j = i + 1; j < count && ok; ++j) {
                const ChainProblem& qj = prm.prob[j];
                if (qj.dep != i) continue;
                const int t = my_job(qj);
                if (t >= 0) ok = Cfg::kChunk ? quant_job(j, t / qj.nch, t % qj.nch) : quant_job(j, t, 0);
            }
        }
    } else if (is_dq) {
        // ------------------------------------------------------------------ expansion (dequantization) warps
        const int qd = wq;                // tensor-memory lane quarter this warp may access
        const int r = qd * 32 + lane;     // row within a block (0..95)
        // Group g expands every G-th stage, counted across segments and problems.
        const int g = wr - 1;
        ptx::Ring r1, r2;
        r1.idx = g;   // (G <= S2 <= S1)
        r2.idx = g;
        int turn = g;  // stages until this group's next turn
        bool ok = true;
        for (int i = 0; i < count && ok; ++i) {
            const ChainProblem& q = prm.prob[i];
            const int nseg = nseg_tab[i];
            for (int j = 0; j < nseg && ok; ++j) {
                const ChainSeg sg = seg_tab[i * kChainMaxSegs + j];
                const int NB = sg.NB;
                const int KS = 2 / NB;
                const int nst = NB == 2 ? sg.nkb : (sg.nkb + 1) >> 1;
                // This thread's rows of the segment (one per block).  A lane beyond the rows repeats the
                // last row: its tensor-memory lane feeds accumulator rows nobody reads out; a warp whose
                // whole lane quarter is beyond the rows skips the work.
                const int Rb0 = sg.R < BR ? sg.R : BR;
                const int row0 = r < Rb0 ? r : Rb0 - 1;
                const int row1 = BR + r < sg.R ? BR + r : sg.R - 1;
                const bool have0 = qd * 32 < Rb0;
                const bool have1 = NB == 2 ? BR + qd * 32 < sg.R : have0;
                const uint32_t code_off = row_offset(Cfg::FMT, row0);
                const uint32_t meta_off = (uint32_t)(KS * sg.R * Cfg::kRowBytes + row0 * MB);
                const uint32_t code_kstep = (uint32_t)(sg.R * Cfg::kRowBytes), meta_kstep = (uint32_t)(sg.R * MB);
                const uint32_t code_s0 = NB == 2 ? row_offset(Cfg::FMT, row1) - code_off : code_kstep;
                const uint32_t meta_s0 = NB == 2 ? (uint32_t)((row1 - row0) * MB) : meta_kstep;
                int st = turn;
                for (; st < nst; st += G) {
                    const int ks = (sg.nkb - st * KS) < KS ? (sg.nkb - st * KS) : KS;
                    const uint32_t full_bar = bar_wfull0 + 8u * (uint32_t)r1.idx;
                    const uint32_t free_bar = bar_afree0 + 8u * (uint32_t)r2.idx;
                    // Both are normally complete already.  The tensor-memory stage FIRST: once the MMAs S2
                    // stages back have completed, every earlier stage has landed -- among them the previous
                    // use of this stage's ring slot (S1 >= S2) -- so the parity test of "weights landed"
                    // cannot mistake the phase before last for this one.
                    if (!ptx::mbar_test_wait(free_bar, r2.phase ^ 1u))
                        ok = chain_mbar_wait(free_bar, r2.phase ^ 1u, abort_flag, gabort, status_word, limit);
                    if (ok && !ptx::mbar_test_wait(full_bar, r1.phase))
                        ok = chain_mbar_wait(full_bar, r1.phase, abort_flag, gabort, status_word, limit);
                    ok = warp_all(ok);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t wsrc = w_ring + (uint32_t)(r1.idx * prm.wslot);
                    const uint32_t a_col = tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)(r2.idx * Cfg::kAStageCols);
                    if constexpr (Cfg::FMT == kFmtTiledFp8) {
                        // FP8 weights: nothing to expand, the rows go to tensor memory as they are
                        if (have0) copy_fp8_row_to_tmem(wsrc + code_off, a_col);
                        if (ks * NB == 2 && have1) copy_fp8_row_to_tmem(wsrc + code_off + code_s0, a_col + 32u);
                    } else if (ks * NB == 2 && have1) {
                        dequant_two_rows_to_tmem<Cfg::FMT>(wsrc + code_off, wsrc + meta_off, wsrc + code_off + code_s0,
                                                           wsrc + meta_off + meta_s0, a_col);
                    } else if (have0) {   // (one copy of the single-row expansion: the roles share the instruction caches)
                        dequant_row_to_tmem<Cfg::FMT>(wsrc + code_off, wsrc + meta_off, a_col);
                    }
                    ptx::mbar_arrive(bar_wfree0 + 8u * (uint32_t)r1.idx);   // this thread has read its codes
                    ptx::tmem_st_wait();
                    ptx::tc_fence_before_sync();
                    ptx::mbar_arrive(bar_afull0 + 8u * (uint32_t)r2.idx);
                    r1.idx += G;
                    if (r1.idx >= S1) {
                        r1.idx -= S1;
                        r1.phase ^= 1u;
                    }
                    r2.idx += G;
                    if (r2.idx >= S2) {
                        r2.idx -= S2;
                        r2.phase ^= 1u;
                    }
                }
                turn = st - nst;
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
    if (threadIdx.x == 32) {
        // The last CTA to leave clears the control block (nobody polls it any more), so that the
        // next launch -- which touches it only after this one has completed -- finds zeros.  After
        // an aborted run it also clears the arrival counters of the blocks cut along K.
        ptx::griddep_wait();
        __threadfence();
        if (atomicAdd(&ctl->exit_count, 1u) == (unsigned)P - 1u) {
            if (*reinterpret_cast<volatile unsigned int*>(gabort)) {
                for (int i = 0; i < count; ++i) {
                    unsigned int* cnt = reinterpret_cast<unsigned int*>(ws + prm.prob[i].cnt_off);
                    for (int b = 0; b < prm.prob[i].rem_blocks; ++b) cnt[b] = 0u;
                }
            }
            for (int i = 0; i < kChainMaxProblems; ++i) {
                ctl->xready[i] = 0u;
                ctl->done[i] = 0u;
            }
            if constexpr (Cfg::kChunk) {
                for (int i = 0; i < count; ++i) {
                    if (prm.prob[i].nch == 1) continue;
                    for (int m = 0; m < prm.prob[i].M; ++m) {
                        amax_ws[i * kChainMaxM + m] = 0u;
                        qcnt_ws[i * kChainMaxM + m] = 0u;
                    }
                }
            }
            ctl->abort = 0u;
            ctl->exit_count = 0u;
            __threadfence();
        }
    }
}

}  // namespace w4a8
