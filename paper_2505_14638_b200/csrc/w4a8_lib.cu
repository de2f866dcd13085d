// C-ABI entry points of the W4A8 library (see include/w4a8.h): argument validation, kernel
// selection, TMA descriptor set-up and launches.  Nothing here allocates device memory.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdlib>
#include <mutex>

#include "../../include/w4a8.h"
#include "w4a8_dpq_kernels.cuh"
#include "w4a8_linear_chain.cuh"
#include "w4a8_linear_splitn.cuh"
#include "w4a8_linear_pair.cuh"
#include "w4a8_linear_streamk.cuh"
#include "w4a8_linear_umma.cuh"
#include "w4a8_simple_kernels.cuh"

namespace w4a8 {

__device__ unsigned int g_status_word = 0;  // bit mask, see kStatus*

static std::atomic<uint64_t> g_launches{0};

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return W4A8_ERR_CUDA;
    static std::mutex mu;
    static int cached_dev = -1, cached_major = 0;
    std::lock_guard<std::mutex> lock(mu);
    if (cached_dev != dev) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
            return W4A8_ERR_CUDA;
        cached_dev = dev;
        cached_major = major;
    }
    return cached_major == 10 ? W4A8_OK : W4A8_ERR_UNSUPPORTED_DEVICE;
}

static unsigned int* status_word_ptr() {
    // Address of the device status word on the current device (looked up once per device).
    static std::mutex mu;
    static unsigned int* ptrs[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
        ptrs[dev] = static_cast<unsigned int*>(p);
    }
    return ptrs[dev];
}

// Device-side address of a page-locked (pinned or registered) host buffer, or nullptr when the
// buffer is ordinary pageable memory (which a kernel must not touch) or the query fails.
static const void* host_buffer_as_device_pointer(const void* p) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    if (a.type != cudaMemoryTypeHost || a.devicePointer == nullptr) return nullptr;
    return a.devicePointer;
}

// Split-K partial sums for callers that cannot provide a workspace (w4a8_linear_static_scratch).
// Device code could name the array directly; host code must not use the symbol as a pointer (it
// is only a host-side stand-in) and asks the runtime for the device address instead.
static __device__ __align__(256) unsigned char g_static_scratch[W4A8_STATIC_SCRATCH_BYTES];

static void* static_scratch_ptr() {
    // Device address of the built-in scratch array on the current device, looked up once per
    // device with that device current.
    static std::mutex mu;
    static void* ptrs[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) return nullptr;
        ptrs[dev] = p;
    }
    return ptrs[dev];
}

static inline int launch_status() {
    return cudaGetLastError() == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

// ------------------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// 2-D uint8 tensor [rows][cols] with row pitch `pitch` bytes; box = box_cols x box_rows.
static bool make_tmap_u8_2d(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint64_t pitch,
                            uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle swz) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// ------------------------------------------------------------------------------ linear plan
struct LinearPlan {
    int algo;      // W4A8_ALGO_SIMT or W4A8_ALGO_UMMA
    int bnx;       // token tile of the UMMA kernel
    int split_k;   // number of K slices
    size_t workspace_bytes;
};

static int pick_bnx(int64_t M) {
    if (M <= 16) return 16;
    if (M <= 32) return 32;
    if (M <= 64) return 64;
    if (M <= 128) return 128;
    return 256;
}

static int auto_split_k(int64_t M, int64_t N, int64_t K, int bnx) {
    const int64_t tiles = ((N + 127) / 128) * ((M + bnx - 1) / bnx);
    const int64_t kb = K / 128;
    if (M > 64 || tiles >= 148) return 1;
    // Fill about two CTAs per SM while keeping at least four K blocks per slice.
    int best = 1;
    for (int s = 1; s <= kb; ++s) {
        if (kb % s != 0) continue;
        if (kb / s < 4) break;
        if (tiles * s <= 2 * 148) best = s;
    }
    return best;
}

static int make_plan(int64_t M, int64_t N, int64_t K, int algo, int split_k, LinearPlan* plan) {
    if (algo == W4A8_ALGO_AUTO) algo = W4A8_ALGO_UMMA;
    if (algo != W4A8_ALGO_SIMT && algo != W4A8_ALGO_UMMA) return W4A8_ERR_INVALID_ARG;
    plan->algo = algo;
    plan->bnx = pick_bnx(M);
    plan->split_k = 1;
    plan->workspace_bytes = 0;
    if (algo == W4A8_ALGO_UMMA) {
        int s = split_k > 0 ? split_k : auto_split_k(M, N, K, plan->bnx);
        if ((K / 128) % s != 0) return W4A8_ERR_BAD_SHAPE;
        plan->split_k = s;
        if (s > 1) plan->workspace_bytes = (size_t)s * (size_t)M * (size_t)N * sizeof(float);
    } else if (split_k > 1) {
        return W4A8_ERR_INVALID_ARG;
    }
    return W4A8_OK;
}

template <class Cfg>
static int launch_umma(const CUtensorMap& tw, const CUtensorMap& tx, const uint16_t* gscale, const uint8_t* gzero,
                       const int32_t* g_idx, const float* s_x, const float* s_w, int sw_stride, void* y, int64_t ldy, int out_dtype,
                       float* partial, int M, int N, int K, int split_k, cudaStream_t st) {
    auto kern = linear_umma_kernel<Cfg>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
    });
    if (attr_err != cudaSuccess) return W4A8_ERR_CUDA;
    unsigned int* status = status_word_ptr();
    if (!status) return W4A8_ERR_CUDA;
    dim3 grid((unsigned)((N + 127) / 128), (unsigned)((M + Cfg::BNX - 1) / Cfg::BNX), (unsigned)split_k);
    kern<<<grid, Cfg::kThreads, Cfg::kSmemBytes, st>>>(tw, tx, gscale, gzero, g_idx, s_x, s_w, sw_stride, y, ldy,
                                                       out_dtype, partial, M, N, K, (K / 128) / split_k, status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_status();
}

// ------------------------------------------------------------------------------ persistent kernel plan
constexpr int kMaxSMs = 160;  // upper bound used to size workspaces without touching a device

static int sm_count() {
    static std::mutex mu;
    static int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    std::lock_guard<std::mutex> lock(mu);
    if (cached_dev != dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached_dev = dev;
        cached = n;
    }
    return cached;
}

constexpr int kNominalSMs = 148;  // for size queries made without a device

// Layout of every w4a8_linear workspace, whatever kernel and shape use it: a control area of fixed
// size at the start (tile counters of the persistent kernel; K-cut counters and placement state
// of the split-N kernel), which every launch leaves zero-filled, and behind it the data (partial
// sums), which may be left in any state.  With the control area at a shape-dependent size, one
// call's left-over partial sums could sit where the next call -- another layer, another kernel
// -- expects zeroed counters; callers do share one workspace between the layers of a model.
constexpr size_t kLinearCtlBytes = 65536;
// The split-N kernel's 2 KB (K-cut counters, placement state -- whose generation word stays non-zero
// by design) sit at the END of the control area, the persistent kernel's tile counters at its start.
constexpr size_t kLinearCtlSplitN = kLinearCtlBytes - 2048;

struct SkPlan {
    int bnx, TM, TN;
    int aligned;   // 1: whole tiles per CTA, nothing shared; 0: equal slices of the (tile, k-block) space
    int64_t P;     // CTAs
    int64_t U;
    size_t counter_bytes, workspace_bytes;
};

constexpr int kSplitNMaxM = 128;  // token counts served by the split-N (decode) kernel

// Token-tile width and schedule of the persistent kernel from a small cost model (microseconds):
// a (tile, k-block) unit costs the larger of the dequantization of its 128 x 128 weights and its
// four MMAs; whole tiles per CTA cost rounds x K/128 units; equal slices cost ceil(U / P) units
// plus the exchange of partial tiles.  Wider token tiles dequantize each weight fewer times.
static void make_sk_plan(int64_t M, int64_t N, int64_t K, int sms, SkPlan* pl) {
    const int64_t KB = K / 128;
    const int64_t TN = (N + 127) / 128;
    const int64_t cap = sms < kMaxSMs ? sms : kMaxSMs;
    double best = 1e30;
    for (int bnx = 256; bnx >= 64; bnx >>= 1) {
        if (bnx > 64 && bnx / 2 >= M) continue;  // more than half of the tile would be padding
        const int64_t TM = (M + bnx - 1) / bnx, Tt = TM * TN, U = Tt * KB;
        const double mma_cycles = 4.0 * (bnx / 2 > 47 ? bnx / 2 : 47);
        const double t_unit = mma_cycles / 1900.0 > 0.22 ? mma_cycles / 1900.0 : 0.22;
        const int64_t Pa = cap < Tt ? cap : Tt;
        const double t_aligned = (double)((Tt + Pa - 1) / Pa) * (double)KB * t_unit;
        int64_t Ps = cap < U ? cap : U;
        const double t_tail = 2.0 + bnx * 2048.0 / 1.0e5;   // exchange of partial tiles: two per CTA
        double t_split = (double)((U + Ps - 1) / Ps) * t_unit + t_tail;
        if (Tt < cap && KB % (cap / Tt) == 0) {
            // Fewer tiles than CTAs: a whole number of CTAs per tile instead of equal slices of the
            // unit space, where that number divides the k-blocks.  Every CTA then stays inside one
            // tile -- one partial tile to store, and a tile's contributors finish together -- at
            // the price of a few idle SMs (measured, us: (128, 4096, 4096) 13.4 against 17.9;
            // (512, 4096, 14336) 41.6 against 49.8; with a remainder -- (256, 6144, 4096), three CTAs
            // per tile, 32 k-blocks -- it was slower: 20.9 against 18.0).
            const int64_t Pk = Tt * (cap / Tt);
            const double t_k = (double)((U + Pk - 1) / Pk) * t_unit + 0.5 * t_tail;
            if (t_k < t_split) {
                t_split = t_k;
                Ps = Pk;
            }
        }
        // (tile counters must fit the control area: otherwise whole tiles per CTA, which need none)
        const bool al = t_aligned <= t_split || 2 * (size_t)Tt * sizeof(unsigned int) > kLinearCtlSplitN;
        const double t = al ? t_aligned : t_split;
        if (t < best) {
            best = t;
            pl->bnx = bnx;
            pl->TM = (int)TM;
            pl->TN = (int)TN;
            pl->U = U;
            pl->aligned = al ? 1 : 0;
            pl->P = al ? Pa : Ps;
        }
    }
    // arrivals and finished reducers per tile live in the control area; the size asked of the caller
    // covers every tile width and any SM count up to kMaxSMs, so that the query needs no device
    pl->counter_bytes = kLinearCtlBytes;
    pl->workspace_bytes = kLinearCtlBytes + (size_t)kMaxSMs * 2 * 256 * 128 * sizeof(float);
}

template <class Cfg>
static int launch_streamk(const CUtensorMap& tx, const uint8_t* wpp, const float* s_x, const float* s_w,
                          int sw_stride, void* y, int64_t ldy, int out_dtype, void* workspace, const SkPlan& pl,
                          int M, int N, int K, cudaStream_t st, const CUtensorMap* tw8 = nullptr, int cl = 0) {
    auto kern = linear_streamk_kernel<Cfg>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
    });
    if (attr_err != cudaSuccess) return W4A8_ERR_CUDA;
    unsigned int* status = status_word_ptr();
    if (!status) return W4A8_ERR_CUDA;
    const int64_t P = pl.P;
    const int aligned = pl.aligned;
    unsigned int* counters = static_cast<unsigned int*>(workspace);
    float* slots = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + pl.counter_bytes);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)P);
    cfg.blockDim = dim3(Cfg::kThreads);
    cfg.dynamicSmemBytes = (size_t)Cfg::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (Cfg::CL) {
        // the cl CTAs of a tile as one thread-block cluster (P = tiles x cl)
        if (cl < 2 || cl > 8 || P % cl != 0) return W4A8_ERR_INVALID_ARG;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)cl;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    // (the second tensor map is read only by the FP8-weight variant)
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tx, tw8 ? *tw8 : tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype,
                                       counters, slots, M, N, K, pl.TM, pl.TN, aligned, cl, status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (e != cudaSuccess) return W4A8_ERR_CUDA;
    return launch_status();
}

// Row partition and ring sizes of the split-N kernel for the current device.
// Workspace of the split-N kernel when it cuts K (bytes; fits any SM count up to kMaxSMs and 128 tokens).
// Layout: split-K counters (1 KB) and placement state of the launch (1 KB) at the end of the common
// control area, partial tiles behind that area.
constexpr size_t kSnCounterBytes = 1024;
constexpr size_t kSnSchedBytes = 1024;
static_assert(kSnCounterBytes == (size_t)kSchedWsOffset, "the kernel finds the placement state behind the counters");
static_assert(kLinearCtlSplitN + kSnCounterBytes + kSnSchedBytes == kLinearCtlBytes, "split-N control data at the end of the common control area");
constexpr size_t kSnWorkspaceBytes = kLinearCtlBytes + (size_t)kMaxSMs * 128 * 128 * sizeof(float);

template <class Cfg>
static bool make_sn_plan(int64_t N, int64_t K, int sms, bool may_split_k, SnPlan* pl) {
    const int64_t NU = N / 8;
    const int64_t KB = K / 128;
    int64_t P = sms < NU ? sms : NU;
    int64_t per = (NU + 32 * P - 1) / (32 * P);  // ranges per CTA so that none exceeds 256 rows
    pl->T = (int)(P * per);
    pl->KSPLIT = 1;
    // Few output channels (at most half as many 128-row blocks as SMs): ranges of whole 128-row
    // blocks, and the K range cut in chunks so that every SM gets a tile.  A CTA's MMA and
    // expansion work then covers 128 useful rows instead of a sliver, and its K walk is shorter;
    // the price is a small fix-up through the workspace.
    const int64_t blocks128 = (N + 127) / 128;
    // (With 64- and 128-token tiles the partial sums are four and eight times larger: only worth
    // it for a long K; with 64 tokens also from K = 4096 on when at most a quarter of the SMs would
    // otherwise get a 128-row block -- o projection at M = 32: 10.9 against 14.6 us.)
    const int64_t kb_min = Cfg::MT == 16 ? 8 : (Cfg::MT == 64 && blocks128 * 4 <= sms ? 32 : 64);
    if (may_split_k && blocks128 * 2 <= sms && KB >= kb_min) {
        int64_t ks = sms / blocks128;
        if (ks > KB / 4) ks = KB / 4;  // at least four k-blocks per chunk
        if (ks > 1 && blocks128 <= (int64_t)(kSnCounterBytes / sizeof(unsigned int)) &&
            blocks128 * ks <= kMaxSMs) {
            pl->KSPLIT = (int)ks;
            pl->T = (int)(blocks128 * ks);
        }
    }
    const int64_t TR = pl->T / pl->KSPLIT;
    const int rmax = (int)((NU + TR - 1) / TR) * 8;
    pl->MBLK = rmax > 128 ? 2 : 1;
    pl->KS = Cfg::kItems / pl->MBLK;
    if ((int64_t)pl->KS > K / 128) pl->KS = 1;
    pl->meta_off = pl->KS * rmax * kRowCodeBytes;
    pl->wstage = (pl->KS * rmax * (kRowCodeBytes + Cfg::kMeta) + 127) / 128 * 128;
    pl->xstage = pl->KS * Cfg::MT * 128;
    const int fixed = Cfg::kBarBytes + Cfg::kOutBytes + 1024;
    int s1 = (Cfg::kSmemBudget - fixed) / (pl->wstage + pl->xstage);
    if (s1 > Cfg::kS1Max) s1 = Cfg::kS1Max;
    if (s1 < Cfg::kS2 || s1 < Cfg::G) return false;  // the tensor-memory ring may not be deeper than the TMA ring, nor may there be more groups than slots
    pl->S1 = s1;
    pl->smem = s1 * (pl->wstage + pl->xstage) + fixed;
    return true;
}

// Launches without a workspace draw their placement slot round-robin over ALL decode launches of
// the process: one counter for every instantiation of the launcher (a counter per instantiation
// gave two kernels of a chain, e.g. a gate/up and a down projection, the same slot while both were
// in flight).  Launches with a workspace keep the state there and need no slot.
static std::atomic<unsigned int> g_sched_seq{0};

template <class Cfg>
static int launch_splitn_planned(const CUtensorMap& tx, const uint8_t* wpp, const float* s_x, const float* s_w,
                                 int sw_stride, void* y, int64_t ldy, int out_dtype, int M, int N, int K,
                                 cudaStream_t st, void* workspace, bool ws_usable, const SnPlan& pl, int sms);

template <int MT, int G, int FMT>
static int launch_splitn_cfg(const CUtensorMap& tx, const uint8_t* wpp, const float* s_x, const float* s_w,
                             int sw_stride, void* y, int64_t ldy, int out_dtype, int M, int N, int K, cudaStream_t st,
                             void* workspace = nullptr, size_t workspace_bytes = 0) {
    using Cfg = SnCfg<MT, G, FMT, false>;
    const int sms = sm_count();
    if (sms <= 0) return W4A8_ERR_CUDA;
    SnPlan pl;
    // K is cut only when the caller gave the (zero-initialised) workspace for the partial sums
    const bool ws_usable = workspace != nullptr && workspace_bytes >= kSnWorkspaceBytes && aligned16(workspace);
    if (!make_sn_plan<Cfg>(N, K, sms, ws_usable, &pl)) return W4A8_ERR_BAD_SHAPE;
    if (pl.KSPLIT > 1)
        return launch_splitn_planned<SnCfg<MT, G, FMT, true>>(tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, M, N, K,
                                                              st, workspace, ws_usable, pl, sms);
    return launch_splitn_planned<Cfg>(tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, M, N, K, st, workspace,
                                      ws_usable, pl, sms);
}

template <class Cfg>
static int launch_splitn_planned(const CUtensorMap& tx, const uint8_t* wpp, const float* s_x, const float* s_w,
                                 int sw_stride, void* y, int64_t ldy, int out_dtype, int M, int N, int K,
                                 cudaStream_t st, void* workspace, bool ws_usable, const SnPlan& pl, int sms) {
    auto kern = linear_splitn_kernel<Cfg>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBudget);
    });
    if (attr_err != cudaSuccess) return W4A8_ERR_CUDA;
    unsigned int* status = status_word_ptr();
    if (!status) return W4A8_ERR_CUDA;
    const int P = pl.T < sms ? pl.T : sms;
    SnPlan plan = pl;
    plan.P = P;
    plan.sched = -1;
    unsigned grid = (unsigned)P;
    if (Cfg::MT == 16 && sms <= kSchedMaxSMs && (K / 128) / pl.KSPLIT >= 16) {
        // two CTAs of this variant fit on an SM: launch twice the workers and let the kernel keep
        // one worker per SM (see the placement notes beside SchedSlot).  Not for short K walks
        // (under 16 k-blocks per tile): there the extra microsecond at the start of a launch costs
        // more than an occasional SM with two workers (o projection at M = 1: 8.4 against 6.6 us).
        plan.sched = ws_usable ? kSchedInWorkspace
                               : (int)(g_sched_seq.fetch_add(1, std::memory_order_relaxed) % (unsigned)kSchedSlots);
        grid = 2u * (unsigned)P;
    }
    unsigned int* counters = reinterpret_cast<unsigned int*>(static_cast<uint8_t*>(workspace) + kLinearCtlSplitN);
    float* partials = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + kLinearCtlBytes);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(Cfg::kThreads);
    cfg.dynamicSmemBytes = (size_t)pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, M, N, K, plan,
                                       counters, partials, status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (e != cudaSuccess) return W4A8_ERR_CUDA;
    return launch_status();
}

// The two-CTA kernel takes whole tiles of 256 output channels x 256 tokens, one CTA pair per tile
// and round.  Each CTA of a pair loads half of the activation tile (24.6 KB per step and SM
// instead of 41 KB, six ring stages instead of four), but the pair pays for it with remote
// barrier traffic and coarser tiles.  Measured against the one-CTA persistent kernel (us):
//   (M, N, K) = (8192, 28672, 8192): 1882 vs 2033;  (2048, 28672, 4096): 241 vs 254;
//   (1024, 28672, 4096): 133 vs 150;  (4096, 4096, 14336): 254 vs 255;
//   (4096, 28672, 4096): 459 vs 438;  (8192, 8192, 8192): 536 vs 523;
//   (4096, 6144, 4096): 113 vs 99;  (4096, 4096, 4096): 77 vs 66;  (2048, 4096, 4096): 42 vs 36.
// It is used where it won: many output channels, and either few token tiles or a long K.
static bool pair_kernel_applies(int64_t M, int64_t N, int64_t K, int sms) {
    if (N % 256 != 0 || N < 16384 || M < 1024 || K < 1024) return false;
    if (!(M <= 2048 || K >= 8192)) return false;
    const int64_t tiles = (N / 256) * ((M + 255) / 256);
    return tiles >= 4 * (int64_t)(sms / 2);
}

// Tiles of 256 weight rows x 256 tokens (two row blocks per activation tile, whole tiles per CTA)
// against tiles of 128 x 256: per k-block step about 1060 tensor-pipe cycles for 50 KB from L2 instead
// of 530 cycles for 41 KB, which the SM's L2 port (about 64 bytes per clock) turns into ~650.  The wide
// tile cannot be cut along K and its epilogue does not overlap the next tile, so it is used where
// whole tiles fill the SMs well (measured, us: (2048, 4096, 4096) 34.9 vs 37.7; (4096, 4096, 14336)
// 203 vs 265; (8192, 28672, 8192) 1785 vs 1906 for the two-CTA kernel) or where a model fitted to
// such measurements says so ((512, 28672, 4096): 68 vs 87).
static bool two_block_tiles_apply(int64_t M, int64_t N, int64_t K, int sms) {
    if (M < 512 || N < 256 || K < 512) return false;
    const int64_t TM = (M + 255) / 256;
    const int64_t t2 = TM * ((N + 255) / 256);
    const int64_t t1 = TM * ((N + 127) / 128);
    const int64_t KB = K / 128;
    const int64_t rounds2 = (t2 + sms - 1) / sms;
    if (5 * t2 >= 4 * rounds2 * sms) return true;   // at least 80 % of the tile slots of its rounds are used
    // microseconds: 0.857 per k-block step + 3.9 per tile for the wide tile; 0.61 per unit for the
    // 128-row tile (0.573 in the two-CTA kernel, 0.85 with at most two token tiles, where every
    // weight tile comes from HBM and four ring stages do not cover that latency)
    const double per_unit = pair_kernel_applies(M, N, K, sms) ? 0.573 : (TM <= 2 ? 0.85 : 0.61);
    const double c2 = (double)rounds2 * ((double)KB * 0.857 + 3.9);
    const double c1 = (double)((t1 * KB + sms - 1) / sms) * per_unit;
    return c2 < c1;
}

template <class Cfg>
static int launch_pair(const uint8_t* x8, int64_t ldx8, const uint8_t* wpp, const float* s_x, const float* s_w,
                       int sw_stride, void* y, int64_t ldy, int out_dtype, int M, int N, int K, int sms,
                       cudaStream_t st) {
    auto kern = linear_pair_kernel<Cfg>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
    });
    if (attr_err != cudaSuccess) return W4A8_ERR_CUDA;
    unsigned int* status = status_word_ptr();
    if (!status) return W4A8_ERR_CUDA;
    CUtensorMap tx;  // this CTA's half of an activation tile: 128 tokens x 128 bytes
    if (!make_tmap_u8_2d(&tx, x8, (uint64_t)M, (uint64_t)K, (uint64_t)ldx8, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B))
        return W4A8_ERR_CUDA;
    const int TM = (M + 255) / 256, TN2 = N / 256;
    int pairs = sms / 2;
    if (pairs > TM * TN2) pairs = TM * TN2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(Cfg::kThreads);
    cfg.dynamicSmemBytes = (size_t)Cfg::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, M, N, K, TM, TN2,
                                       status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (e != cudaSuccess) return W4A8_ERR_CUDA;
    return launch_status();
}

// Where the cluster plan cannot run (not all of its clusters resident at once on this device):
// 65..128 tokens on a layer with few output channels (at most a quarter as many 128-row tiles as
// SMs) take the persistent kernel with K cut between a whole number of CTAs per tile and the
// exchange through the workspace, instead of the split-N kernel, every CTA of which pulls the whole
// X8 through its L2 port (measured, us: o projection 13.4 against 15.3, down projection 21.5
// against 27.5; qkv and gate_up stay: 16.9 against 15.4, 33.6 against 27.1).
static bool streamk_for_128_tokens(int64_t M, int64_t N, int64_t K, int sms) {
    return M > 64 && M <= kSplitNMaxM && K >= 2048 && ((N + 127) / 128) * 4 <= sms;
}

// Tiles of 256 weight rows x Cfg::BNX tokens, whole tiles per CTA (no workspace).
template <class Cfg>
static int launch_two_block(const uint8_t* x8, int64_t ldx8, const uint8_t* wpp, const float* s_x, const float* s_w,
                            int sw_stride, void* y, int64_t ldy, int out_dtype, int64_t M, int64_t N, int64_t K, int sms,
                            cudaStream_t st) {
    SkPlan p2;
    p2.bnx = Cfg::BNX;
    p2.TM = (int)((M + Cfg::BNX - 1) / Cfg::BNX);
    p2.TN = (int)((N + 255) / 256);
    p2.aligned = 1;
    p2.U = (int64_t)p2.TM * p2.TN * (K / 128);
    p2.P = (int64_t)p2.TM * p2.TN < sms ? (int64_t)p2.TM * p2.TN : sms;
    p2.counter_bytes = 0;
    p2.workspace_bytes = 0;
    CUtensorMap tx2;
    if (!make_tmap_u8_2d(&tx2, x8, (uint64_t)M, (uint64_t)K, (uint64_t)ldx8, 128, (uint32_t)Cfg::BNX, CU_TENSOR_MAP_SWIZZLE_128B))
        return W4A8_ERR_CUDA;
    return launch_streamk<Cfg>(tx2, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, nullptr, p2, (int)M, (int)N, (int)K, st);
}

// Few tiles (at most half as many 128-row tiles as SMs) and at most 128 tokens: CTAs per tile of the plan
// that cuts K between the CTAs of a thread-block cluster (0: the plan does not apply).  Every CTA keeps
// at least two k-blocks.
static int cluster_kcut_ctas(int64_t M, int64_t N, int64_t K, int sms) {
    if (M > 128) return 0;
    const int64_t TN = (N + 127) / 128, KB = K / 128;
    int64_t c = sms / TN;
    if (c > 8) c = 8;
    while (c > 1 && KB < 2 * c) --c;
    return c >= 2 ? (int)c : 0;
}

// Launches the cluster plan; returns -1 (nothing launched) when the device cannot hold all of the
// launch's clusters at once -- a second wave would cost more than the exchange through L2 saves.
template <class Cfg>
static int launch_cluster_kcut(const uint8_t* x8, int64_t ldx8, const uint8_t* wpp, const float* s_x, const float* s_w,
                               int sw_stride, void* y, int64_t ldy, int out_dtype, int M, int N, int K, int cl,
                               cudaStream_t st) {
    const int TN = (N + 127) / 128;
    static std::atomic<int> fits[9];   // clusters of size cl resident at once (0: not asked yet)
    int have = fits[cl].load(std::memory_order_relaxed);
    if (have == 0) {
        auto kern = linear_streamk_kernel<Cfg>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess)
            return W4A8_ERR_CUDA;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(cl * 64));
        cfg.blockDim = dim3(Cfg::kThreads);
        cfg.dynamicSmemBytes = (size_t)Cfg::kSmemBytes;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cl;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) {
            cudaGetLastError();
            n = -1;
        }
        have = n > 0 ? n : -1;
        fits[cl].store(have, std::memory_order_relaxed);
    }
    if (have < TN) return -1;
    CUtensorMap tx;
    if (!make_tmap_u8_2d(&tx, x8, (uint64_t)M, (uint64_t)K, (uint64_t)ldx8, 128, (uint32_t)Cfg::BNX,
                         CU_TENSOR_MAP_SWIZZLE_128B))
        return W4A8_ERR_CUDA;
    SkPlan pl;
    pl.bnx = Cfg::BNX;
    pl.TM = 1;
    pl.TN = TN;
    pl.aligned = 1;
    pl.U = (int64_t)TN * (K / 128);
    pl.P = (int64_t)TN * cl;
    pl.counter_bytes = 0;
    pl.workspace_bytes = 0;
    return launch_streamk<Cfg>(tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, nullptr, pl, M, N, K, st, nullptr, cl);
}

static int linear_tiled_impl(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* wpp,
                             int fmt, const float* s_w, int sw_stride, int64_t N, int64_t K, void* y, int64_t ldy,
                             int out_dtype, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    if (M > 16) {
        // 17..128 tokens on a layer with few 128-row tiles: K cut between the CTAs of a cluster (measured, us,
        // against the split-N kernel or the persistent kernel with its exchange through L2:
        // (32, 4096, 4096) 8.0 / 9.8, (64, 2048, 4096) 7.4 / 12.6, (100, 512, 8192) 9.0 / 15.0,
        // (128, 4096, 4096) 11.9 / 12.9, (128, 4096, 14336) 19.0 / 21.2, (128, 6144, 4096) 13.5 / 14.5; at
        // 16 tokens and fewer the split-N kernel, which overlaps its set-up with the launch before, stays
        // ahead: (8, 4096, 4096) 8.5 / 7.3)
        const int sms_c = sm_count();
        const int cl0 = sms_c > 0 ? cluster_kcut_ctas(M, N, K, sms_c) : 0;
        for (int cl = cl0; cl >= 2; --cl) {   // the largest cluster size of which all clusters are resident at once
            int rc = check_device();
            if (rc != W4A8_OK) return rc;
            if (M <= 64)
                rc = fmt == kFmtTiledSignMag
                         ? launch_cluster_kcut<SkCfg<64, 4, 8, 4, kFmtTiledSignMag, 1, false, true>>(
                               x8, ldx8, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, (int)M, (int)N, (int)K, cl, st)
                         : launch_cluster_kcut<SkCfg<64, 4, 8, 4, kFmtTiled, 1, false, true>>(
                               x8, ldx8, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, (int)M, (int)N, (int)K, cl, st);
            else
                rc = fmt == kFmtTiledSignMag
                         ? launch_cluster_kcut<SkCfg<128, 3, 6, 3, kFmtTiledSignMag, 1, false, true>>(
                               x8, ldx8, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, (int)M, (int)N, (int)K, cl, st)
                         : launch_cluster_kcut<SkCfg<128, 3, 6, 3, kFmtTiled, 1, false, true>>(
                               x8, ldx8, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, (int)M, (int)N, (int)K, cl, st);
            if (rc != -1) return rc;
        }
    }
    bool split_n = M <= kSplitNMaxM;
    if (split_n && M > 64) {
        // (the persistent kernel needs its full workspace; without it the split-N kernel runs)
        SkPlan plq;
        make_sk_plan(M, N, K, kNominalSMs, &plq);
        const int sms_q = sm_count();
        if (sms_q > 0 && streamk_for_128_tokens(M, N, K, sms_q) && workspace != nullptr &&
            workspace_bytes >= plq.workspace_bytes && aligned16(workspace))
            split_n = false;
    }
    if (split_n) {
        int rc = check_device();
        if (rc != W4A8_OK) return rc;
        const int mt = M <= 16 ? 16 : (M <= 64 ? 64 : 128);
        CUtensorMap tx;
        if (!make_tmap_u8_2d(&tx, x8, (uint64_t)M, (uint64_t)K, (uint64_t)ldx8, 128, (uint32_t)mt,
                             CU_TENSOR_MAP_SWIZZLE_128B))
            return W4A8_ERR_CUDA;
        const int Mi = (int)M, Ni = (int)N, Ki = (int)K;
        if (mt == 128) {
            return fmt == kFmtTiledSignMag
                       ? launch_splitn_cfg<128, 4, kFmtTiledSignMag>(tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype,
                                                                     Mi, Ni, Ki, st, workspace,
                                                                     workspace_bytes)
                       : launch_splitn_cfg<128, 4, kFmtTiled>(tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, Mi, Ni,
                                                              Ki, st, workspace, workspace_bytes);
        }
        if (fmt == kFmtTiledSignMag) {
            return mt == 16 ? launch_splitn_cfg<16, 2, kFmtTiledSignMag>(tx, wpp, s_x, s_w, sw_stride, y, ldy,
                                                                            out_dtype, Mi, Ni, Ki, st,
                                                                            workspace, workspace_bytes)
                            : launch_splitn_cfg<64, 4, kFmtTiledSignMag>(tx, wpp, s_x, s_w, sw_stride, y, ldy,
                                                                            out_dtype, Mi, Ni, Ki, st,
                                                                            workspace, workspace_bytes);
        }
        return mt == 16 ? launch_splitn_cfg<16, 2, kFmtTiled>(tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, Mi,
                                                                 Ni, Ki, st, workspace, workspace_bytes)
                        : launch_splitn_cfg<64, 4, kFmtTiled>(tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, Mi,
                                                                 Ni, Ki, st, workspace, workspace_bytes);
    }
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return W4A8_ERR_BAD_ALIGNMENT;
    SkPlan pl;
    make_sk_plan(M, N, K, kNominalSMs, &pl);
    if (!workspace || workspace_bytes < pl.workspace_bytes) return W4A8_ERR_WORKSPACE_TOO_SMALL;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    const int sms = sm_count();
    if (sms <= 0) return W4A8_ERR_CUDA;
    if (two_block_tiles_apply(M, N, K, sms)) {
        // tiles of 256 weight rows x 256 tokens, whole tiles per CTA
        return fmt == kFmtTiledSignMag
                   ? launch_two_block<SkCfg<256, 3, 3, 2, kFmtTiledSignMag, 2>>(x8, ldx8, wpp, s_x, s_w, sw_stride, y, ldy,
                                                                               out_dtype, M, N, K, sms, st)
                   : launch_two_block<SkCfg<256, 3, 3, 2, kFmtTiled, 2>>(x8, ldx8, wpp, s_x, s_w, sw_stride, y, ldy,
                                                                        out_dtype, M, N, K, sms, st);
    }
    if (pair_kernel_applies(M, N, K, sms))
        return fmt == kFmtTiledSignMag
                   ? launch_pair<PairCfg<3, 6, 4, kFmtTiledSignMag>>(x8, ldx8, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype,
                                                                      (int)M, (int)N, (int)K, sms, st)
                   : launch_pair<PairCfg<3, 6, 4, kFmtTiled>>(x8, ldx8, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype,
                                                               (int)M, (int)N, (int)K, sms, st);
    make_sk_plan(M, N, K, sms, &pl);
    CUtensorMap tx;
    if (!make_tmap_u8_2d(&tx, x8, (uint64_t)M, (uint64_t)K, (uint64_t)ldx8, 128, (uint32_t)pl.bnx,
                         CU_TENSOR_MAP_SWIZZLE_128B))
        return W4A8_ERR_CUDA;
    const int Mi = (int)M, Ni = (int)N, Ki = (int)K;
#define W4A8_SK(BNX, G, S1, S2)                                                                                  \
    rc = (fmt == kFmtTiledSignMag)                                                                                \
             ? launch_streamk<SkCfg<BNX, G, S1, S2, kFmtTiledSignMag>>(tx, wpp, s_x, s_w, sw_stride, y, ldy,     \
                                                                       out_dtype, workspace, pl, Mi, Ni, Ki, st) \
             : launch_streamk<SkCfg<BNX, G, S1, S2, kFmtTiled>>(tx, wpp, s_x, s_w, sw_stride, y, ldy, out_dtype, \
                                                                workspace, pl, Mi, Ni, Ki, st)
    switch (pl.bnx) {
        case 64: W4A8_SK(64, 4, 8, 4); break;
        case 128: W4A8_SK(128, 4, 4, 4); break;
        default: W4A8_SK(256, 4, 4, 3); break;
    }
#undef W4A8_SK
    return rc;
}

static int linear_impl(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* codes,
                       const void* gscale, const uint8_t* gzero, int fmt, const float* s_w, int sw_stride,
                       int64_t N, int64_t K, int group, void* y, int64_t ldy, int out_dtype, void* workspace,
                       size_t workspace_bytes, int algo, int split_k, cudaStream_t st,
                       const int32_t* g_idx = nullptr) {
    if (fmt != kFmtCanonical && fmt != kFmtTiled && fmt != kFmtTiledSignMag) return W4A8_ERR_INVALID_ARG;
    if (g_idx && (fmt != kFmtCanonical || (reinterpret_cast<uintptr_t>(g_idx) & 3u))) return W4A8_ERR_INVALID_ARG;
    if (!x8 || !s_x || !codes || !s_w || !y) return W4A8_ERR_INVALID_ARG;
    if (fmt == kFmtCanonical && !gscale) return W4A8_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (sw_stride != 0 && sw_stride != 1) return W4A8_ERR_INVALID_ARG;
    if (out_dtype != W4A8_OUT_BF16 && out_dtype != W4A8_OUT_FP32) return W4A8_ERR_INVALID_ARG;
    if (group != kGroup || K % kGroup != 0 || N % 16 != 0) return W4A8_ERR_BAD_SHAPE;
    if (ldx8 < K || ldy < N) return W4A8_ERR_BAD_SHAPE;
    if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(x8) || !aligned16(codes) || !aligned16(y) || (ldx8 % 16) != 0) return W4A8_ERR_BAD_ALIGNMENT;
    if ((reinterpret_cast<uintptr_t>(gscale) & 1u) || (reinterpret_cast<uintptr_t>(s_x) & 3u) ||
        (reinterpret_cast<uintptr_t>(s_w) & 3u))
        return W4A8_ERR_BAD_ALIGNMENT;
    if (fmt != kFmtCanonical) {
        if (algo != W4A8_ALGO_AUTO || split_k > 0) return W4A8_ERR_INVALID_ARG;
        return linear_tiled_impl(x8, ldx8, s_x, M, codes, fmt, s_w, sw_stride, N, K, y, ldy, out_dtype, workspace,
                                 workspace_bytes, st);
    }
    LinearPlan plan;
    int rc = make_plan(M, N, K, algo, split_k, &plan);
    if (rc != W4A8_OK) return rc;
    if (plan.workspace_bytes > 0) {
        if (!workspace || workspace_bytes < plan.workspace_bytes) return W4A8_ERR_WORKSPACE_TOO_SMALL;
        if (reinterpret_cast<uintptr_t>(workspace) & 15u) return W4A8_ERR_BAD_ALIGNMENT;
    }
    rc = check_device();
    if (rc != W4A8_OK) return rc;

    const uint16_t* gs = static_cast<const uint16_t*>(gscale);
    if (plan.algo == W4A8_ALGO_SIMT) {
        dim3 grid((unsigned)((N + 31) / 32), (unsigned)((M + 7) / 8));
        linear_simt_kernel<<<grid, 256, 0, st>>>(x8, ldx8, s_x, M, codes, gs, gzero, s_w, sw_stride, N, K, y, ldy,
                                                 out_dtype);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        return launch_status();
    }

    CUtensorMap tw, tx;
    if (!make_tmap_u8_2d(&tw, codes, (uint64_t)N, (uint64_t)(K / 2), (uint64_t)(K / 2), 64, 128,
                         CU_TENSOR_MAP_SWIZZLE_64B))
        return W4A8_ERR_CUDA;
    if (!make_tmap_u8_2d(&tx, x8, (uint64_t)M, (uint64_t)K, (uint64_t)ldx8, 128, (uint32_t)plan.bnx,
                         CU_TENSOR_MAP_SWIZZLE_128B))
        return W4A8_ERR_CUDA;
    float* partial = plan.split_k > 1 ? static_cast<float*>(workspace) : nullptr;
    const int Mi = (int)M, Ni = (int)N, Ki = (int)K;
#define W4A8_LAUNCH(BNX, STG)                                                                                 \
    rc = g_idx ? launch_umma<UmmaCfg<BNX, STG, false, false, true>>(tw, tx, gs, gzero, g_idx, s_x, s_w, sw_stride, y, \
                                                                    ldy, out_dtype, partial, Mi, Ni, Ki,          \
                                                                    plan.split_k, st)                             \
               : launch_umma<UmmaCfg<BNX, STG>>(tw, tx, gs, gzero, nullptr, s_x, s_w, sw_stride, y, ldy, out_dtype,  \
                                                partial, Mi, Ni, Ki, plan.split_k, st)
    switch (plan.bnx) {
        case 16: W4A8_LAUNCH(16, 4); break;
        case 32: W4A8_LAUNCH(32, 4); break;
        case 64: W4A8_LAUNCH(64, 6); break;
        case 128: W4A8_LAUNCH(128, 5); break;
        default: W4A8_LAUNCH(256, 4); break;
    }
#undef W4A8_LAUNCH
    if (rc != W4A8_OK) return rc;
    if (plan.split_k > 1) {
        int64_t total = M * N;
        unsigned blocks = (unsigned)((total + 255) / 256);
        if (blocks > 148u * 8u) blocks = 148u * 8u;
        splitk_reduce_kernel<<<blocks, 256, 0, st>>>(partial, plan.split_k, M, N, s_x, s_w, sw_stride, y, ldy,
                                                     out_dtype);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        rc = launch_status();
    }
    return rc;
}

// W8A8 comparison path (Sec. 4.3): FP8 weights [N][K] through the same tcgen05 kernel, no expansion.
static int linear_w8a8_impl(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* w8,
                            const float* s_w, int sw_stride, int64_t N, int64_t K, void* y, int64_t ldy,
                            int out_dtype, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    if (!x8 || !s_x || !w8 || !s_w || !y) return W4A8_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (sw_stride != 0 && sw_stride != 1) return W4A8_ERR_INVALID_ARG;
    if (out_dtype != W4A8_OUT_BF16 && out_dtype != W4A8_OUT_FP32) return W4A8_ERR_INVALID_ARG;
    if (K % kGroup != 0 || N % 16 != 0 || ldx8 < K || ldy < N) return W4A8_ERR_BAD_SHAPE;
    if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(x8) || !aligned16(w8) || !aligned16(y) || (ldx8 % 16) != 0) return W4A8_ERR_BAD_ALIGNMENT;
    LinearPlan plan;
    int rc = make_plan(M, N, K, W4A8_ALGO_UMMA, 0, &plan);
    if (rc != W4A8_OK) return rc;
    if (plan.workspace_bytes > 0) {
        if (!workspace || workspace_bytes < plan.workspace_bytes) return W4A8_ERR_WORKSPACE_TOO_SMALL;
        if (reinterpret_cast<uintptr_t>(workspace) & 15u) return W4A8_ERR_BAD_ALIGNMENT;
    }
    rc = check_device();
    if (rc != W4A8_OK) return rc;
    CUtensorMap tw, tx;
    if (!make_tmap_u8_2d(&tw, w8, (uint64_t)N, (uint64_t)K, (uint64_t)K, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B))
        return W4A8_ERR_CUDA;
    {
        // Many tokens and at least as many 128 x 256 tiles as SMs: the persistent kernel of the W4A8
        // path with the expansion compiled out (whole tiles per CTA, no workspace) -- the like-for-like
        // partner of w4a8_linear at prefill sizes.
        const int sms = sm_count();
        const int64_t TM = (M + 255) / 256, TN = (N + 127) / 128;
        if (M > 128 && sms > 0 && TM * TN >= sms) {
            SkPlan p8;
            p8.bnx = 256;
            p8.TM = (int)TM;
            p8.TN = (int)TN;
            p8.aligned = 1;
            p8.U = TM * TN * (K / 128);
            p8.P = sms;
            p8.counter_bytes = 0;
            p8.workspace_bytes = 0;
            CUtensorMap tx8;
            if (!make_tmap_u8_2d(&tx8, x8, (uint64_t)M, (uint64_t)K, (uint64_t)ldx8, 128, 256, CU_TENSOR_MAP_SWIZZLE_128B))
                return W4A8_ERR_CUDA;
            return launch_streamk<SkCfg<256, 4, 4, 3, kFmtTiledSignMag, 1, true>>(tx8, w8, s_x, s_w, sw_stride, y, ldy,
                                                                                    out_dtype, nullptr, p8, (int)M,
                                                                                    (int)N, (int)K, st, &tw);
        }
    }
    if (!make_tmap_u8_2d(&tx, x8, (uint64_t)M, (uint64_t)K, (uint64_t)ldx8, 128, (uint32_t)plan.bnx,
                         CU_TENSOR_MAP_SWIZZLE_128B))
        return W4A8_ERR_CUDA;
    float* partial = plan.split_k > 1 ? static_cast<float*>(workspace) : nullptr;
    const int Mi = (int)M, Ni = (int)N, Ki = (int)K;
#define W4A8_LAUNCH8(BNX, STG)                                                                                   \
    rc = launch_umma<UmmaCfg<BNX, STG, true>>(tw, tx, nullptr, nullptr, nullptr, s_x, s_w, sw_stride, y, ldy, out_dtype,  \
                                              partial, Mi, Ni, Ki, plan.split_k, st)
    switch (plan.bnx) {
        case 16: W4A8_LAUNCH8(16, 4); break;
        case 32: W4A8_LAUNCH8(32, 4); break;
        case 64: W4A8_LAUNCH8(64, 6); break;
        case 128: W4A8_LAUNCH8(128, 5); break;
        default: W4A8_LAUNCH8(256, 4); break;
    }
#undef W4A8_LAUNCH8
    if (rc != W4A8_OK) return rc;
    if (plan.split_k > 1) {
        int64_t total = M * N;
        unsigned blocks = (unsigned)((total + 255) / 256);
        if (blocks > 148u * 8u) blocks = 148u * 8u;
        splitk_reduce_kernel<<<blocks, 256, 0, st>>>(partial, plan.split_k, M, N, s_x, s_w, sw_stride, y, ldy,
                                                     out_dtype);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        rc = launch_status();
    }
    return rc;
}

// W4A16 tile width over the tokens and split-K workspace (FP32 partial sums, one slab per K slice).
static int w4a16_bnx(int64_t M) { return M <= 16 ? 16 : (M <= 32 ? 32 : (M <= 64 ? 64 : 128)); }
static size_t w4a16_workspace(int64_t M, int64_t N, int64_t K) {
    const int s = auto_split_k(M, N, K, w4a16_bnx(M));
    return s > 1 ? (size_t)s * (size_t)M * (size_t)N * sizeof(float) : 0;
}

// W4A16 comparison path (Sec. 4.3): BF16 activations, INT4 codes expanded to BF16 in the kernel,
// kind::f16 MMAs; canonical weights, one tile per CTA.
static int linear_w4a16_impl(const void* x, int64_t ldx, int64_t M, const uint8_t* codes, const void* gscale,
                             const uint8_t* gzero, const float* s_w, int sw_stride, int64_t N, int64_t K, void* y,
                             int64_t ldy, int out_dtype, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    if (!x || !codes || !gscale || !s_w || !y) return W4A8_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (sw_stride != 0 && sw_stride != 1) return W4A8_ERR_INVALID_ARG;
    if (out_dtype != W4A8_OUT_BF16 && out_dtype != W4A8_OUT_FP32) return W4A8_ERR_INVALID_ARG;
    if (K % kGroup != 0 || N % 16 != 0 || ldx < K || ldy < N) return W4A8_ERR_BAD_SHAPE;
    if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX / 2) return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(x) || !aligned16(codes) || !aligned16(y) || (ldx % 8) != 0 || (K / 2) % 16 != 0)
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    const int bnx = w4a16_bnx(M);
    const int split_k = auto_split_k(M, N, K, bnx);
    const size_t need = w4a16_workspace(M, N, K);
    if (need > 0) {
        if (!workspace || workspace_bytes < need) return W4A8_ERR_WORKSPACE_TOO_SMALL;
        if (reinterpret_cast<uintptr_t>(workspace) & 15u) return W4A8_ERR_BAD_ALIGNMENT;
    }
    CUtensorMap tw, tx;
    if (!make_tmap_u8_2d(&tw, codes, (uint64_t)N, (uint64_t)(K / 2), (uint64_t)(K / 2), 64, 128,
                         CU_TENSOR_MAP_SWIZZLE_64B))
        return W4A8_ERR_CUDA;
    // X as bytes: rows of 2 K bytes, panels of 128 bytes (64 BF16 values)
    if (!make_tmap_u8_2d(&tx, x, (uint64_t)M, (uint64_t)(2 * K), (uint64_t)(2 * ldx), 128, (uint32_t)bnx,
                         CU_TENSOR_MAP_SWIZZLE_128B))
        return W4A8_ERR_CUDA;
    const uint16_t* gs = static_cast<const uint16_t*>(gscale);
    float* partial = split_k > 1 ? static_cast<float*>(workspace) : nullptr;
    const int Mi = (int)M, Ni = (int)N, Ki = (int)K;
#define W4A8_LAUNCH16(BNX, STG)                                                                                  \
    rc = launch_umma<UmmaCfg<BNX, STG, false, true>>(tw, tx, gs, gzero, nullptr, nullptr, s_w, sw_stride, y, ldy,         \
                                                     out_dtype, partial, Mi, Ni, Ki, split_k, st)
    switch (bnx) {
        case 16: W4A8_LAUNCH16(16, 4); break;
        case 32: W4A8_LAUNCH16(32, 4); break;
        case 64: W4A8_LAUNCH16(64, 3); break;
        default: W4A8_LAUNCH16(128, 3); break;
    }
#undef W4A8_LAUNCH16
    if (rc != W4A8_OK) return rc;
    if (split_k > 1) {
        int64_t total = M * N;
        unsigned blocks = (unsigned)((total + 255) / 256);
        if (blocks > 148u * 8u) blocks = 148u * 8u;
        splitk_reduce_kernel<<<blocks, 256, 0, st>>>(partial, split_k, M, N, nullptr, s_w, sw_stride, y, ldy,
                                                     out_dtype);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        rc = launch_status();
    }
    return rc;
}

// W4A16 on the persistent kernel (prepacked sign-magnitude weights, whole tiles per CTA).
static int linear_w4a16_tiled_impl(const void* x, int64_t ldx, int64_t M, const uint8_t* wpp, int fmt, const float* s_w,
                                   int sw_stride, int64_t N, int64_t K, void* y, int64_t ldy, int out_dtype,
                                   cudaStream_t st) {
    if (!x || !wpp || !s_w || !y) return W4A8_ERR_INVALID_ARG;
    if (fmt != kFmtTiledSignMag) return W4A8_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (sw_stride != 0 && sw_stride != 1) return W4A8_ERR_INVALID_ARG;
    if (out_dtype != W4A8_OUT_BF16 && out_dtype != W4A8_OUT_FP32) return W4A8_ERR_INVALID_ARG;
    if (K % kGroup != 0 || N % 16 != 0 || ldx < K || ldy < N) return W4A8_ERR_BAD_SHAPE;
    if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX / 2) return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(x) || !aligned16(wpp) || !aligned16(y) || (ldx % 8) != 0) return W4A8_ERR_BAD_ALIGNMENT;
    if (reinterpret_cast<uintptr_t>(s_w) & 3u) return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    const int sms = sm_count();
    if (sms <= 0) return W4A8_ERR_CUDA;
    // token tiles of 256 from 513 tokens on (measured, us, 256 / 128: (2048, 4096, 4096) 64 / 77,
    // (2048, 28672, 4096) 409 / 459, (512, 4096, 4096) 35 / 25)
    const int bnx = M > 512 ? 256 : (M > 64 ? 128 : 64);
    SkPlan pl;
    pl.bnx = bnx;
    pl.TM = (int)((M + bnx - 1) / bnx);
    pl.TN = (int)((N + 127) / 128);
    pl.aligned = 1;
    pl.U = (int64_t)pl.TM * pl.TN * (K / 128);
    pl.P = (int64_t)pl.TM * pl.TN < sms ? (int64_t)pl.TM * pl.TN : sms;
    pl.counter_bytes = 0;
    pl.workspace_bytes = 0;
    CUtensorMap tx;   // X as bytes: rows of 2 K bytes, boxes of 128 bytes (64 BF16 values) x bnx tokens
    if (!make_tmap_u8_2d(&tx, x, (uint64_t)M, (uint64_t)(2 * K), (uint64_t)(2 * ldx), 128, (uint32_t)bnx,
                         CU_TENSOR_MAP_SWIZZLE_128B))
        return W4A8_ERR_CUDA;
    // (the kernel reads no activation scale in this variant)
    if (bnx == 256)
        return launch_streamk<SkCfg<256, 2, 2, 2, kFmtTiledSignMag, 1, false, false, true>>(
            tx, wpp, s_w, s_w, sw_stride, y, ldy, out_dtype, nullptr, pl, (int)M, (int)N, (int)K, st);
    if (bnx == 128)
        return launch_streamk<SkCfg<128, 3, 3, 2, kFmtTiledSignMag, 1, false, false, true>>(
            tx, wpp, s_w, s_w, sw_stride, y, ldy, out_dtype, nullptr, pl, (int)M, (int)N, (int)K, st);
    return launch_streamk<SkCfg<64, 3, 3, 2, kFmtTiledSignMag, 1, false, false, true>>(
        tx, wpp, s_w, s_w, sw_stride, y, ldy, out_dtype, nullptr, pl, (int)M, (int)N, (int)K, st);
}

static int quantize_act_impl(const void* x, int64_t M, int64_t K, int64_t ldx, uint8_t* x8, int64_t ldx8,
                             float* s_x, int scale_mode, const float* static_scale, cudaStream_t st) {
    if (!x || !x8 || !s_x) return W4A8_ERR_INVALID_ARG;
    if (M <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (scale_mode != W4A8_SCALE_EXACT && scale_mode != W4A8_SCALE_POW2) return W4A8_ERR_INVALID_ARG;
    if (K % 16 != 0 || ldx < K || ldx8 < K || M > INT32_MAX) return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(x) || !aligned16(x8) || (ldx % 8) != 0 || (ldx8 % 16) != 0 ||
        (reinterpret_cast<uintptr_t>(s_x) & 3u))
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    const uint16_t* xs = static_cast<const uint16_t*>(x);
    const int64_t nchunks = K / 16;
    const unsigned rows = (unsigned)M;
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(rows);
    cfg.stream = st;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    cudaError_t lerr = cudaSuccess;
#define W4A8_AQ(T, C)                                                                                         \
    do {                                                                                                      \
        cfg.blockDim = dim3(T);                                                                               \
        lerr = cudaLaunchKernelEx(&cfg, act_quant_kernel<T, C>, xs, K, ldx, x8, ldx8, s_x, scale_mode,        \
                                  static_scale);                                                              \
    } while (0)
    if (nchunks <= 32) W4A8_AQ(32, 1);
    else if (nchunks <= 64) W4A8_AQ(64, 1);
    else if (nchunks <= 128) W4A8_AQ(128, 1);
    else if (nchunks <= 256) W4A8_AQ(256, 1);
    else if (nchunks <= 512) W4A8_AQ(256, 2);
    else if (nchunks <= 1024) W4A8_AQ(256, 4);
    else {
        cfg.blockDim = dim3(256);
        lerr = cudaLaunchKernelEx(&cfg, act_quant_kernel_2pass, xs, K, ldx, x8, ldx8, s_x, scale_mode, static_scale);
    }
#undef W4A8_AQ
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (lerr != cudaSuccess) return W4A8_ERR_CUDA;
    return launch_status();
}

static int silu_mul_quantize_impl(const void* gu, int64_t M, int64_t F, int64_t ldgu, uint8_t* x8, int64_t ldx8,
                                  float* s_x, int scale_mode, const float* static_scale, void* h_out, int64_t ldh,
                                  cudaStream_t st) {
    if (!gu || !x8 || !s_x) return W4A8_ERR_INVALID_ARG;
    if (M <= 0 || F <= 0) return W4A8_ERR_INVALID_ARG;
    if (scale_mode != W4A8_SCALE_EXACT && scale_mode != W4A8_SCALE_POW2) return W4A8_ERR_INVALID_ARG;
    if (F % 16 != 0 || F > 16384 || ldgu < 2 * F || ldx8 < F || (h_out && ldh < F) || M > INT32_MAX / 8)
        return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(gu) || !aligned16(x8) || (ldgu % 8) != 0 || (ldx8 % 16) != 0 ||
        (reinterpret_cast<uintptr_t>(s_x) & 3u) || (h_out && (!aligned16(h_out) || (ldh % 8) != 0)))
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    const int64_t nchunks = F / 16;
    // CTAs (one cluster) per token, 128 chunks each
    const int cl = nchunks <= 128 ? 1 : (nchunks <= 256 ? 2 : (nchunks <= 512 ? 4 : 8));
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = 1;
    attrs[1].id = cudaLaunchAttributeClusterDimension;
    attrs[1].val.clusterDim.x = (unsigned)cl;
    attrs[1].val.clusterDim.y = 1;
    attrs[1].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(M * cl));
    cfg.blockDim = dim3(128);
    cfg.stream = st;
    cfg.attrs = attrs;
    cfg.numAttrs = cl > 1 ? 2 : 1;
    const uint16_t* g = static_cast<const uint16_t*>(gu);
    uint16_t* h = static_cast<uint16_t*>(h_out);
    cudaError_t lerr;
    if (cl == 1)
        lerr = cudaLaunchKernelEx(&cfg, silu_mul_quant_kernel<1>, g, F, ldgu, x8, ldx8, s_x, scale_mode, static_scale,
                                  h, ldh);
    else if (cl == 2)
        lerr = cudaLaunchKernelEx(&cfg, silu_mul_quant_kernel<2>, g, F, ldgu, x8, ldx8, s_x, scale_mode, static_scale,
                                  h, ldh);
    else if (cl == 4)
        lerr = cudaLaunchKernelEx(&cfg, silu_mul_quant_kernel<4>, g, F, ldgu, x8, ldx8, s_x, scale_mode, static_scale,
                                  h, ldh);
    else
        lerr = cudaLaunchKernelEx(&cfg, silu_mul_quant_kernel<8>, g, F, ldgu, x8, ldx8, s_x, scale_mode, static_scale,
                                  h, ldh);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (lerr != cudaSuccess) return W4A8_ERR_CUDA;
    return launch_status();
}

// ------------------------------------------------------------------------------ chain of decode-sized layers
// Workspace layout: header (control block, activation scales), then per problem the FP8 activation
// tiles ([K/128][16][128] bytes), the partial-sum slots of the blocks that are cut along K (one per
// CTA, M x 96 floats) and their arrival counters.  Sized for any SM count up to kMaxSMs so that
// the query needs no device.
constexpr size_t kChainCntBytes = 1024;
static_assert(kMaxSMs * sizeof(unsigned int) <= kChainCntBytes, "one counter per block that is cut along K");
static size_t chain_part_bytes(int64_t M, int ctas) { return (size_t)ctas * (size_t)M * kChainBlockRows * sizeof(float); }
static size_t chain_workspace_need(const w4a8_chain_problem* pr, int count) {
    size_t need = kChainHeaderBytes;
    for (int i = 0; i < count; ++i)
        need += (size_t)pr[i].K * kChainMaxM + chain_part_bytes(pr[i].M, kMaxSMs) + kChainCntBytes;
    return need;
}

// Validation (device-independent part) of a chain description.
static int chain_validate(const w4a8_chain_problem* pr, int count) {
    if (!pr || count < 1 || count > kChainMaxProblems) return W4A8_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i) {
        const w4a8_chain_problem& q = pr[i];
        if (!q.x_bf16 || !q.weights || !q.s_w || !q.y) return W4A8_ERR_INVALID_ARG;
        if (q.M <= 0 || q.N <= 0 || q.K <= 0) return W4A8_ERR_INVALID_ARG;
        if (q.input_kind != kChainKindPlain && q.input_kind != kChainKindSiluMul) return W4A8_ERR_INVALID_ARG;
        if (q.depends_on < -1 || q.depends_on >= i) return W4A8_ERR_INVALID_ARG;
        // a problem that reads an earlier problem's output reads BF16: that output may not be FP32
        if (q.depends_on >= 0 && q.x_bf16 == pr[q.depends_on].y && pr[q.depends_on].out_dtype != W4A8_OUT_BF16)
            return W4A8_ERR_INVALID_ARG;
        if (q.scale_mode != W4A8_SCALE_EXACT && q.scale_mode != W4A8_SCALE_POW2) return W4A8_ERR_INVALID_ARG;
        if (q.weight_format != kFmtTiled && q.weight_format != kFmtTiledSignMag && q.weight_format != kFmtTiledFp8)
            return W4A8_ERR_INVALID_ARG;
        if (q.weight_format != pr[0].weight_format) return W4A8_ERR_INVALID_ARG;
        if (q.sw_stride != 0 && q.sw_stride != 1) return W4A8_ERR_INVALID_ARG;
        if (q.out_dtype != W4A8_OUT_BF16 && q.out_dtype != W4A8_OUT_FP32) return W4A8_ERR_INVALID_ARG;
        if (q.M > kChainMaxM || q.K % kGroup != 0 || q.N % 16 != 0) return W4A8_ERR_BAD_SHAPE;
        if (q.K > 16384 || q.N > (1 << 20)) return W4A8_ERR_BAD_SHAPE;
        const int64_t in_cols = q.input_kind == kChainKindSiluMul ? 2 * q.K : q.K;
        if (q.ldx < in_cols || q.ldy < q.N || (q.x8_out && q.ldx8_out < q.K)) return W4A8_ERR_BAD_SHAPE;
        if (!aligned16(q.x_bf16) || !aligned16(q.y) || (q.ldx % 8) != 0 ||
            (reinterpret_cast<uintptr_t>(q.weights) & 127u))
            return W4A8_ERR_BAD_ALIGNMENT;
        if (q.x8_out && (!aligned16(q.x8_out) || (q.ldx8_out % 16) != 0)) return W4A8_ERR_BAD_ALIGNMENT;
        if ((reinterpret_cast<uintptr_t>(q.s_w) & 3u) || (reinterpret_cast<uintptr_t>(q.s_x_out) & 3u) ||
            (reinterpret_cast<uintptr_t>(q.static_scale) & 3u))
            return W4A8_ERR_BAD_ALIGNMENT;
    }
    return W4A8_OK;
}

template <class Cfg>
static int launch_chain(const ChainParams& prm, int grid, int smem, uint8_t* ws, cudaStream_t st) {
    auto kern = linear_chain_kernel<Cfg>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemMax);
    });
    if (attr_err != cudaSuccess) return W4A8_ERR_CUDA;
    unsigned int* status = status_word_ptr();
    if (!status) return W4A8_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(Cfg::kThreads);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, prm, ws, status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (e != cudaSuccess) return W4A8_ERR_CUDA;
    return launch_status();
}

static int linear_chain_impl(const w4a8_chain_problem* pr, int count, void* workspace, size_t workspace_bytes,
                             int groups, cudaStream_t st) {
    int rc = chain_validate(pr, count);
    if (rc != W4A8_OK) return rc;
    if (groups != 0 && (groups < 2 || groups > 4)) return W4A8_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < chain_workspace_need(pr, count)) return W4A8_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(workspace) & 127u) return W4A8_ERR_BAD_ALIGNMENT;
    rc = check_device();
    if (rc != W4A8_OK) return rc;
    const int sms = sm_count();
    if (sms < kChainMaxM || sms > kMaxSMs) return W4A8_ERR_UNSUPPORTED_DEVICE;   // one quantization job per CTA and problem
    const int fmt = pr[0].weight_format;
    const int mb = meta_bytes(fmt);

    ChainParams prm;
    memset(&prm, 0, sizeof(prm));
    prm.count = count;
    prm.wait_limit_ns = ptx::kWaitLimitNs;
    int stash = 8192, jobs = 0, rot = 0;
    bool full = false;   // some problem is of the gated kind or has its rows quantized in chunks by several CTAs
    size_t off = kChainHeaderBytes;
    for (int i = 0; i < count; ++i) {
        const w4a8_chain_problem& q = pr[i];
        ChainProblem& d = prm.prob[i];
        d.x = static_cast<const uint16_t*>(q.x_bf16);
        d.wpp = q.weights;
        d.s_w = q.s_w;
        d.y = q.y;
        d.x8_out = q.x8_out;
        d.s_x_out = q.s_x_out;
        d.static_scale = q.static_scale;
        d.ldx = q.ldx;
        d.ldy = q.ldy;
        d.ldx8_out = q.ldx8_out;
        d.M = (int)q.M;
        d.N = (int)q.N;
        d.K = (int)q.K;
        d.kind = q.input_kind;
        d.dep = q.depends_on;
        d.sw_stride = q.sw_stride;
        d.out_dtype = q.out_dtype;
        d.scale_mode = q.scale_mode;
        // whole 96-row blocks per CTA while at least as many blocks as CTAs are left, the rest cut along K
        const int blocks = chain_blocks(d.N);
        d.rounds = blocks / sms;
        if ((d.rounds + 1) / 2 + 2 > kChainMaxSegs) return W4A8_ERR_BAD_SHAPE;   // more whole blocks per CTA than the segment table holds
        d.rem_blocks = blocks - d.rounds * sms;
        // rows of 4096 elements and more are cut into chunks of about 4096 (2048 for the gated kind:
        // silu costs far more per element than a load) quantized by different CTAs, if there is a
        // CTA for every chunk of every row
        // (the kernel with this in it is instantiated for the default number of expansion groups only)
        const int chunk = d.kind == kChainKindSiluMul ? 2048 : 4096;
        d.nch = (groups == 0 || groups == 4) ? (d.K + chunk - 1) / chunk : 1;
        while (d.nch > 1 && d.M * d.nch > sms) --d.nch;
        if (d.nch > 1 || d.kind == kChainKindSiluMul) full = true;
        d.job_base = jobs;
        jobs += d.M * d.nch;
        d.rem_rot = rot % sms;
        // the next problem's runs start behind this one's; when the runs cover every CTA, one CTA
        // further, so that the adding CTAs (every few CTAs one) are not the same ones problem after problem
        const int pr = chain_rem_ctas(d, sms);
        rot += pr < sms ? pr : 1;
        d.x8_off = (uint32_t)off;
        off += (size_t)q.K * kChainMaxM;
        d.part_off = (uint32_t)off;
        off += chain_part_bytes(q.M, kMaxSMs);
        d.cnt_off = (uint32_t)off;
        off += kChainCntBytes;
        if (off > 0xFFFFFFFFull) return W4A8_ERR_BAD_SHAPE;
        if (2 * (int)q.K > stash) stash = 2 * (int)q.K;
    }
    // a slot holds the two (k-block, block) items of a stage: 2 x 96 rows of codes and meta data
    prm.wslot = (2 * kChainBlockRows * (row_bytes(fmt) + mb) + 127) / 128 * 128;
    prm.stash = stash;
    using C0 = ChainCfg<4, kFmtTiledSignMag>;
    const int fixed = 1024 + C0::kXRingBytes + stash + C0::kBarBytes + C0::kSegBytes;
    int s1 = (C0::kSmemMax - fixed) / prm.wslot;
    if (s1 > C0::kS1Max) s1 = C0::kS1Max;
    if (s1 < C0::kS2) return W4A8_ERR_BAD_SHAPE;   // (the weight ring may not be shallower than the tensor-memory ring)
    prm.S1 = s1;
    const int smem = fixed + s1 * prm.wslot;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (groups == 0) groups = 4;
#define W4A8_CHAIN(GG)                                                                             \
    (fmt == kFmtTiledSignMag ? launch_chain<ChainCfg<GG, kFmtTiledSignMag>>(prm, sms, smem, ws, st) \
                             : launch_chain<ChainCfg<GG, kFmtTiled>>(prm, sms, smem, ws, st))
    if (fmt == kFmtTiledFp8)   // the W8A8 comparison scheme: one instantiation (four groups, everything compiled in)
        return launch_chain<ChainCfg<4, kFmtTiledFp8, true>>(prm, sms, smem, ws, st);
    if (groups == 4 && !full)
        return fmt == kFmtTiledSignMag ? launch_chain<ChainCfg<4, kFmtTiledSignMag, false>>(prm, sms, smem, ws, st)
                                       : launch_chain<ChainCfg<4, kFmtTiled, false>>(prm, sms, smem, ws, st);
    switch (groups) {
        case 2: return W4A8_CHAIN(2);
        case 3: return W4A8_CHAIN(3);
        default: return W4A8_CHAIN(4);
    }
#undef W4A8_CHAIN
}

// One CTA, one thread: a bounded wait on a barrier nobody arrives on (self-test of the time-out path).
__global__ void bounded_wait_selftest_kernel(unsigned long long limit_ns, unsigned long long* elapsed,
                                             unsigned int* status_word) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    __shared__ unsigned int chain_abort;
    const uint32_t b = ptx::smem_addr(&bar);
    ptx::mbar_init(b, 1);
    abort_flag = 0u;
    chain_abort = 0u;
    ptx::fence_mbar_init();
    const uint64_t t0 = ptx::globaltimer_ns();
    const bool ok = chain_mbar_wait(b, 0u, &abort_flag, &chain_abort, status_word, limit_ns);
    const uint64_t t1 = ptx::globaltimer_ns();
    if (elapsed) *elapsed = ok ? 0ull : (unsigned long long)(t1 - t0);
}

}  // namespace w4a8

using namespace w4a8;

extern "C" {

int w4a8_quantize_act(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* x8, int64_t ldx8,
                      float* s_x, int scale_mode, const float* static_scale, void* stream) {
    return quantize_act_impl(x_bf16, M, K, ldx, x8, ldx8, s_x, scale_mode, static_scale,
                             static_cast<cudaStream_t>(stream));
}

int w4a8_dequant_weight(const uint8_t* codes, const void* gscale_bf16, const uint8_t* gzero, int64_t N,
                        int64_t K, int group, uint8_t* w8, void* stream) {
    if (!codes || !gscale_bf16 || !w8) return W4A8_ERR_INVALID_ARG;
    if (N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (group != kGroup || K % kGroup != 0) return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(codes) || !aligned16(w8) || (reinterpret_cast<uintptr_t>(gscale_bf16) & 1u))
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    int64_t units = N * (K / 32);
    unsigned blocks = (unsigned)((units + 255) / 256 < 148 * 16 ? (units + 255) / 256 : 148 * 16);
    dequant_weight_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        codes, static_cast<const uint16_t*>(gscale_bf16), gzero, N, K, w8);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_status();
}

int w4a8_linear(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* weights,
                const void* gscale_bf16, const uint8_t* gzero, int weight_format, const float* s_w, int sw_stride,
                int64_t N, int64_t K, int group, void* y, int64_t ldy, int out_dtype, void* workspace,
                size_t workspace_bytes, void* stream) {
    return linear_impl(x8, ldx8, s_x, M, weights, gscale_bf16, gzero, weight_format, s_w, sw_stride, N, K, group, y,
                       ldy, out_dtype, workspace, workspace_bytes, W4A8_ALGO_AUTO, 0,
                       static_cast<cudaStream_t>(stream));
}

size_t w4a8_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int weight_format) {
    if (M <= 0 || N <= 0 || K <= 0 || K % kGroup != 0) return 0;
    if (weight_format == kFmtCanonical) return w4a8_linear_ex_workspace_bytes(M, N, K, W4A8_ALGO_AUTO, 0);
    if (weight_format != kFmtTiled && weight_format != kFmtTiledSignMag) return 0;
    if (M <= 64) return kSnWorkspaceBytes;  // used when the layer has few output channels and K is cut
    SkPlan pl;
    make_sk_plan(M, N, K, kNominalSMs, &pl);
    // (65..128 tokens: either kernel may run, the persistent one only with its full workspace)
    return M <= kSplitNMaxM && pl.workspace_bytes < kSnWorkspaceBytes ? kSnWorkspaceBytes : pl.workspace_bytes;
}

int w4a8_prepack_fp8(const uint8_t* w8, int64_t N, int64_t K, uint8_t* out, size_t out_bytes, void* stream) {
    if (!w8 || !out || N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (K % kGroup != 0 || N % 16 != 0) return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(w8) || (reinterpret_cast<uintptr_t>(out) & 127u)) return W4A8_ERR_BAD_ALIGNMENT;
    if (out_bytes < (size_t)N * (size_t)K) return W4A8_ERR_WORKSPACE_TOO_SMALL;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    const int64_t chunks = N * (K / 16);
    prepack_fp8_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(w8, N, K, out);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_status();
}

size_t w4a8_prepack_bytes(int64_t N, int64_t K, int weight_format) {
    if (N <= 0 || K <= 0 || K % kGroup != 0) return 0;
    if (weight_format == kFmtTiledFp8) return (size_t)N * (size_t)K;
    if (weight_format != kFmtTiled && weight_format != kFmtTiledSignMag) return 0;
    return (size_t)N * (size_t)(K / 128) * (size_t)(kRowCodeBytes + meta_bytes(weight_format));
}

int w4a8_prepack_weight(const uint8_t* codes, const void* gscale_bf16, const uint8_t* gzero, int64_t N, int64_t K,
                        int group, int weight_format, uint8_t* out, size_t out_bytes, void* stream) {
    if (!codes || !gscale_bf16 || !out) return W4A8_ERR_INVALID_ARG;
    if (N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (weight_format != kFmtTiled && weight_format != kFmtTiledSignMag) return W4A8_ERR_INVALID_ARG;
    if (weight_format == kFmtTiledSignMag && gzero != nullptr) return W4A8_ERR_INVALID_ARG;
    if (group != kGroup || K % kGroup != 0 || N % 8 != 0) return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(codes) || (reinterpret_cast<uintptr_t>(out) & 127u) ||
        (reinterpret_cast<uintptr_t>(gscale_bf16) & 1u))
        return W4A8_ERR_BAD_ALIGNMENT;
    if (out_bytes < w4a8_prepack_bytes(N, K, weight_format)) return W4A8_ERR_WORKSPACE_TOO_SMALL;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    unsigned int* status = status_word_ptr();
    if (!status) return W4A8_ERR_CUDA;
    const int64_t blocks = ((N + 127) / 128) * (K / 128);
    prepack_kernel<<<(unsigned)blocks, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        codes, static_cast<const uint16_t*>(gscale_bf16), gzero, N, K, weight_format, out, status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_status();
}

int w4a8_linear_ex(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* codes,
                   const void* gscale_bf16, const uint8_t* gzero, const float* s_w, int sw_stride, int64_t N,
                   int64_t K, int group, void* y, int64_t ldy, int out_dtype, void* workspace,
                   size_t workspace_bytes, int algo, int split_k, void* stream) {
    return linear_impl(x8, ldx8, s_x, M, codes, gscale_bf16, gzero, kFmtCanonical, s_w, sw_stride, N, K, group, y,
                       ldy, out_dtype, workspace, workspace_bytes, algo, split_k, static_cast<cudaStream_t>(stream));
}

int w4a8_linear_gidx(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* codes,
                     const void* gscale_bf16, const uint8_t* gzero, const int32_t* g_idx, const float* s_w,
                     int sw_stride, int64_t N, int64_t K, int group, void* y, int64_t ldy, int out_dtype,
                     void* workspace, size_t workspace_bytes, void* stream) {
    if (!g_idx) return W4A8_ERR_INVALID_ARG;
    return linear_impl(x8, ldx8, s_x, M, codes, gscale_bf16, gzero, kFmtCanonical, s_w, sw_stride, N, K, group, y,
                       ldy, out_dtype, workspace, workspace_bytes, W4A8_ALGO_UMMA, 0, static_cast<cudaStream_t>(stream),
                       g_idx);
}

int w4a8_linear_static_scratch(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* codes,
                               const void* gscale_bf16, const uint8_t* gzero, const float* s_w, int sw_stride,
                               int64_t N, int64_t K, int group, void* y, int64_t ldy, int out_dtype, int split_k,
                               void* stream) {
    if (M <= 0 || N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (group != kGroup || K % kGroup != 0 || N % 16 != 0) return W4A8_ERR_BAD_SHAPE;
    LinearPlan plan;
    int rc = make_plan(M, N, K, W4A8_ALGO_UMMA, split_k, &plan);
    if (rc != W4A8_OK) return rc;
    if (plan.workspace_bytes > (size_t)W4A8_STATIC_SCRATCH_BYTES) return W4A8_ERR_WORKSPACE_TOO_SMALL;
    void* scratch = nullptr;
    if (plan.workspace_bytes > 0) {
        rc = check_device();
        if (rc != W4A8_OK) return rc;
        scratch = static_scratch_ptr();
        if (!scratch) return W4A8_ERR_CUDA;
    }
    return linear_impl(x8, ldx8, s_x, M, codes, gscale_bf16, gzero, kFmtCanonical, s_w, sw_stride, N, K, group, y,
                       ldy, out_dtype, scratch, plan.workspace_bytes, W4A8_ALGO_UMMA, plan.split_k,
                       static_cast<cudaStream_t>(stream));
}

int w4a8_dequant_weight_gidx(const uint8_t* codes, const void* gscale_bf16, const uint8_t* gzero,
                             const int32_t* g_idx, int64_t N, int64_t K, int64_t G, uint8_t* w8, void* stream) {
    if (!codes || !gscale_bf16 || !g_idx || !w8) return W4A8_ERR_INVALID_ARG;
    if (N <= 0 || K <= 0 || G <= 0) return W4A8_ERR_INVALID_ARG;
    if (K % 2 != 0) return W4A8_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(gscale_bf16) & 1u) || (reinterpret_cast<uintptr_t>(g_idx) & 3u) ||
        (reinterpret_cast<uintptr_t>(w8) & 1u))
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    const int64_t total = N * (K / 2);
    dequant_weight_gidx_kernel<<<(unsigned)((total + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        codes, static_cast<const uint16_t*>(gscale_bf16), gzero, g_idx, N, K, G, w8);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_status();
}

int w4a8_linear_w8a8(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* w8,
                     const float* s_w, int sw_stride, int64_t N, int64_t K, void* y, int64_t ldy, int out_dtype,
                     void* workspace, size_t workspace_bytes, void* stream) {
    return linear_w8a8_impl(x8, ldx8, s_x, M, w8, s_w, sw_stride, N, K, y, ldy, out_dtype, workspace,
                            workspace_bytes, static_cast<cudaStream_t>(stream));
}

int w4a8_linear_w4a16(const void* x_bf16, int64_t ldx, int64_t M, const uint8_t* codes, const void* gscale_bf16,
                      const uint8_t* gzero, const float* s_w, int sw_stride, int64_t N, int64_t K, void* y,
                      int64_t ldy, int out_dtype, void* workspace, size_t workspace_bytes, void* stream) {
    return linear_w4a16_impl(x_bf16, ldx, M, codes, gscale_bf16, gzero, s_w, sw_stride, N, K, y, ldy, out_dtype,
                             workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

int w4a8_linear_w4a16_tiled(const void* x_bf16, int64_t ldx, int64_t M, const uint8_t* weights, int weight_format,
                            const float* s_w, int sw_stride, int64_t N, int64_t K, void* y, int64_t ldy, int out_dtype,
                            void* stream) {
    return linear_w4a16_tiled_impl(x_bf16, ldx, M, weights, weight_format, s_w, sw_stride, N, K, y, ldy, out_dtype,
                                   static_cast<cudaStream_t>(stream));
}

size_t w4a8_linear_w4a16_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K <= 0 || K % kGroup != 0) return 0;
    return w4a16_workspace(M, N, K);
}

int w4a8_silu_mul_quantize(const void* gate_up_bf16, int64_t M, int64_t F, int64_t ldgu, uint8_t* x8, int64_t ldx8,
                           float* s_x, int scale_mode, const float* static_scale, void* h_bf16_out, int64_t ldh,
                           void* stream) {
    return silu_mul_quantize_impl(gate_up_bf16, M, F, ldgu, x8, ldx8, s_x, scale_mode, static_scale, h_bf16_out, ldh,
                                  static_cast<cudaStream_t>(stream));
}

size_t w4a8_linear_ex_workspace_bytes(int64_t M, int64_t N, int64_t K, int algo, int split_k) {
    if (M <= 0 || N <= 0 || K <= 0 || K % kGroup != 0) return 0;
    LinearPlan plan;
    if (make_plan(M, N, K, algo, split_k, &plan) != W4A8_OK) return 0;
    return plan.workspace_bytes;
}

int w4a8_quantize_weight_rtn(const float* W, int64_t N, int64_t K, int group, int symmetric, int pow2,
                             int per_channel, uint8_t* codes, void* gscale_bf16, uint8_t* gzero, float* s_w,
                             void* stream) {
    if (!W || !codes || !gscale_bf16 || !s_w) return W4A8_ERR_INVALID_ARG;
    if (!symmetric && !gzero) return W4A8_ERR_INVALID_ARG;
    if (N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (group != kGroup || K % kGroup != 0) return W4A8_ERR_BAD_SHAPE;
    if (!aligned16(W) || !aligned16(codes) || (reinterpret_cast<uintptr_t>(gscale_bf16) & 1u) ||
        (reinterpret_cast<uintptr_t>(s_w) & 3u))
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned int* amax_bits = reinterpret_cast<unsigned int*>(s_w);
    if (per_channel) {
        absmax_f32_kernel<<<(unsigned)N, 256, 0, st>>>(W, N, K, 1, amax_bits);
    } else {
        if (cudaMemsetAsync(s_w, 0, sizeof(float), st) != cudaSuccess) return W4A8_ERR_CUDA;
        int64_t total = N * K;
        unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
        absmax_f32_kernel<<<blocks, 256, 0, st>>>(W, N, K, 0, amax_bits);
    }
    int64_t ns = per_channel ? N : 1;
    amax_to_scale_kernel<<<(unsigned)((ns + 255) / 256), 256, 0, st>>>(s_w, ns);
    int64_t warps = N * (K / 128);
    rtn_quant_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(W, N, K, symmetric, pow2, per_channel, s_w, codes,
                                                                  static_cast<uint16_t*>(gscale_bf16), gzero);
    g_launches.fetch_add(3, std::memory_order_relaxed);
    return launch_status();
}

size_t w4a8_gar_workspace_bytes(int64_t K) {
    if (K <= 0 || K % kGroup != 0) return 0;
    return (size_t)K * sizeof(int32_t) + (size_t)(K / kGroup) * sizeof(float);
}

int w4a8_gar_permutation(const float* hdiag, int64_t K, int group, int32_t* perm, void* workspace,
                         size_t workspace_bytes, void* stream) {
    if (!hdiag || !perm) return W4A8_ERR_INVALID_ARG;
    if (K <= 0) return W4A8_ERR_INVALID_ARG;
    if (group != kGroup || K % kGroup != 0 || K > INT32_MAX) return W4A8_ERR_BAD_SHAPE;
    if (!workspace || workspace_bytes < w4a8_gar_workspace_bytes(K)) return W4A8_ERR_WORKSPACE_TOO_SMALL;
    if ((reinterpret_cast<uintptr_t>(hdiag) & 3u) || (reinterpret_cast<uintptr_t>(perm) & 3u) ||
        (reinterpret_cast<uintptr_t>(workspace) & 3u))
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int G = (int)(K / kGroup);
    int32_t* within = static_cast<int32_t*>(workspace);
    float* gmax = reinterpret_cast<float*>(within + K);
    gar_within_kernel<<<(unsigned)G, 128, 0, st>>>(hdiag, within, gmax);
    gar_order_kernel<<<(unsigned)G, 128, 0, st>>>(within, gmax, G, perm);
    g_launches.fetch_add(2, std::memory_order_relaxed);
    return launch_status();
}

int w4a8_hessian_accumulate(const void* x_bf16, int64_t T, int64_t K, int64_t ldx, float* H, int accumulate,
                            void* stream) {
    if (!x_bf16 || !H || T <= 0 || K <= 0 || ldx < K) return W4A8_ERR_INVALID_ARG;
    if (K > 32768) return W4A8_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(x_bf16) & 1u) || (reinterpret_cast<uintptr_t>(H) & 3u)) return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    const int64_t nb = (K + kHessTile - 1) / kHessTile;
    hessian_xtx_kernel<<<(unsigned)(nb * (nb + 1) / 2), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint16_t*>(x_bf16), T, K, ldx, H, accumulate ? 1.0f : 0.0f);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_status();
}

int w4a8_hessian_prepare(const float* H, int64_t K, const int32_t* perm, float damp, float* H_out, float* scratch,
                         void* stream) {
    if (!H || !H_out || !scratch || K <= 0 || H == H_out) return W4A8_ERR_INVALID_ARG;
    if (!(damp >= 0.0f)) return W4A8_ERR_INVALID_ARG;
    if (K > 32768) return W4A8_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(H) & 3u) || (reinterpret_cast<uintptr_t>(H_out) & 3u) ||
        (reinterpret_cast<uintptr_t>(scratch) & 3u) || (reinterpret_cast<uintptr_t>(perm) & 3u))
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    hessian_diag_mean_kernel<<<1, 256, 0, st>>>(H, K, scratch);
    hessian_prepare_kernel<<<(unsigned)((K * K + 255) / 256), 256, 0, st>>>(H, K, perm, damp, scratch, H_out);
    g_launches.fetch_add(2, std::memory_order_relaxed);
    return launch_status();
}

size_t w4a8_dpq_workspace_bytes(int64_t N, int64_t K) {
    if (N <= 0 || K <= 0 || K % kGroup != 0) return 0;
    return ((size_t)N * (size_t)K + (size_t)N * 128) * sizeof(float);
}

int w4a8_dpq_quantize(const float* W, int64_t N, int64_t K, int group, const float* U, const int32_t* perm,
                      int symmetric, int mse_steps, int per_channel, uint8_t* codes, void* gscale_bf16,
                      uint8_t* gzero, float* s_w, void* workspace, size_t workspace_bytes, void* stream) {
    if (!W || !U || !codes || !gscale_bf16 || !s_w) return W4A8_ERR_INVALID_ARG;
    if (!symmetric && !gzero) return W4A8_ERR_INVALID_ARG;
    if (N <= 0 || K <= 0 || mse_steps < 0 || mse_steps > 11) return W4A8_ERR_INVALID_ARG;
    if (group != kGroup || K % kGroup != 0) return W4A8_ERR_BAD_SHAPE;
    if (!workspace || workspace_bytes < w4a8_dpq_workspace_bytes(N, K)) return W4A8_ERR_WORKSPACE_TOO_SMALL;
    if (!aligned16(W) || !aligned16(codes) || !aligned16(workspace) || (reinterpret_cast<uintptr_t>(U) & 3u) ||
        (reinterpret_cast<uintptr_t>(perm) & 3u) || (reinterpret_cast<uintptr_t>(gscale_bf16) & 1u) ||
        (reinterpret_cast<uintptr_t>(s_w) & 3u))
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    constexpr int kBlockSmem = 128 * 128 * 4 + kDpqRowsPerCta * 128;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(dpq_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBlockSmem);
    });
    if (attr_err != cudaSuccess) return W4A8_ERR_CUDA;
    // Eq. 6
    unsigned int* amax_bits = reinterpret_cast<unsigned int*>(s_w);
    if (per_channel) {
        absmax_f32_kernel<<<(unsigned)N, 256, 0, st>>>(W, N, K, 1, amax_bits);
    } else {
        if (cudaMemsetAsync(s_w, 0, sizeof(float), st) != cudaSuccess) return W4A8_ERR_CUDA;
        int64_t total = N * K;
        unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
        absmax_f32_kernel<<<blocks, 256, 0, st>>>(W, N, K, 0, amax_bits);
    }
    int64_t ns = per_channel ? N : 1;
    amax_to_scale_kernel<<<(unsigned)((ns + 255) / 256), 256, 0, st>>>(s_w, ns);
    float* work = static_cast<float*>(workspace);
    float* err = work + N * K;
    dpq_gather_kernel<<<(unsigned)((N * K + 255) / 256), 256, 0, st>>>(W, perm, N, K, work);
    uint64_t launches = 3;
    const int G = (int)(K / kGroup);
    for (int b = 0; b < G; ++b) {
        dpq_block_kernel<<<(unsigned)((N + kDpqRowsPerCta - 1) / kDpqRowsPerCta), 16 * kDpqRowsPerCta, kBlockSmem, st>>>(
            work, U, perm, N, K, b, symmetric, mse_steps, per_channel, s_w, codes,
            static_cast<uint16_t*>(gscale_bf16), gzero, err);
        ++launches;
        const int64_t rest = K - ((int64_t)b + 1) * 128;
        if (rest > 0) {
            dim3 grid((unsigned)(rest / 128), (unsigned)((N + 127) / 128));
            dpq_trailing_kernel<<<grid, 256, 0, st>>>(work, U, err, N, K, b);
            ++launches;
        }
    }
    g_launches.fetch_add(launches, std::memory_order_relaxed);
    return launch_status();
}

int w4a8_forward_host(const void* x_host_bf16, int64_t M, const uint8_t* weights, const void* gscale_bf16,
                      const uint8_t* gzero, int weight_format, const float* s_w, int sw_stride, int64_t N,
                      int64_t K, int group,
                      void* y_host_bf16, void* x_dev, uint8_t* x8_dev, float* s_x_dev, void* y_dev,
                      void* workspace, size_t workspace_bytes, void* stream) {
    if (!x_host_bf16 || !y_host_bf16 || !x_dev || !x8_dev || !s_x_dev || !y_dev) return W4A8_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return W4A8_ERR_INVALID_ARG;
    if (group != kGroup || K % kGroup != 0 || N % 16 != 0) return W4A8_ERR_BAD_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Validate the two stages before anything is enqueued.
    if (weight_format != kFmtCanonical && weight_format != kFmtTiled && weight_format != kFmtTiledSignMag)
        return W4A8_ERR_INVALID_ARG;
    if (!weights || !s_w || (weight_format == kFmtCanonical && !gscale_bf16)) return W4A8_ERR_INVALID_ARG;
    const size_t need = w4a8_linear_workspace_bytes(M, N, K, weight_format);
    if (need > 0 && (!workspace || workspace_bytes < need)) return W4A8_ERR_WORKSPACE_TOO_SMALL;
    if (!aligned16(x_dev) || !aligned16(x8_dev) || !aligned16(y_dev) || !aligned16(weights) ||
        (reinterpret_cast<uintptr_t>(workspace) & 15u))
        return W4A8_ERR_BAD_ALIGNMENT;
    int rc;
    // Decode-sized calls on pinned host buffers: the kernels read the activations from, and write the
    // result to, the host buffers themselves (they are mapped into the device's address space), which
    // moves the same bytes over the bus without two copy-engine operations and their hand-overs to
    // and from the compute engine (about 20 of the 37 us such a call took on the device).
    if (M <= kSplitNMaxM) {
        const void* xh = host_buffer_as_device_pointer(x_host_bf16);
        void* yh = const_cast<void*>(host_buffer_as_device_pointer(y_host_bf16));
        if (xh && yh && aligned16(xh) && aligned16(yh)) {
            rc = quantize_act_impl(xh, M, K, K, x8_dev, K, s_x_dev, W4A8_SCALE_EXACT, nullptr, st);
            if (rc != W4A8_OK) return rc;
            return linear_impl(x8_dev, K, s_x_dev, M, weights, gscale_bf16, gzero, weight_format, s_w, sw_stride, N,
                               K, group, yh, N, W4A8_OUT_BF16, workspace, workspace_bytes, W4A8_ALGO_AUTO, 0, st);
        }
    }
    if (cudaMemcpyAsync(x_dev, x_host_bf16, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return W4A8_ERR_CUDA;
    rc = quantize_act_impl(x_dev, M, K, K, x8_dev, K, s_x_dev, W4A8_SCALE_EXACT, nullptr, st);
    if (rc != W4A8_OK) return rc;
    rc = linear_impl(x8_dev, K, s_x_dev, M, weights, gscale_bf16, gzero, weight_format, s_w, sw_stride, N, K,
                     group, y_dev, N, W4A8_OUT_BF16, workspace, workspace_bytes, W4A8_ALGO_AUTO, 0, st);
    if (rc != W4A8_OK) return rc;
    if (cudaMemcpyAsync(y_host_bf16, y_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return W4A8_ERR_CUDA;
    return W4A8_OK;
}

size_t w4a8_linear_chain_workspace_bytes(const w4a8_chain_problem* problems_host, int count) {
    if (chain_validate(problems_host, count) != W4A8_OK) return 0;
    return chain_workspace_need(problems_host, count);
}

int w4a8_linear_chain(const w4a8_chain_problem* problems_host, int count, void* workspace, size_t workspace_bytes,
                      int groups, void* stream) {
    return linear_chain_impl(problems_host, count, workspace, workspace_bytes, groups,
                             static_cast<cudaStream_t>(stream));
}

int w4a8_host_buffer_device_pointer(const void* host, void** dev_out) {
    if (!host || !dev_out) return W4A8_ERR_INVALID_ARG;
    const void* d = host_buffer_as_device_pointer(host);
    if (!d) return W4A8_ERR_INVALID_ARG;
    *dev_out = const_cast<void*>(d);
    return W4A8_OK;
}

int w4a8_selftest_bounded_wait(uint64_t limit_ns, uint64_t* elapsed_ns_dev, void* stream) {
    if (limit_ns == 0 || limit_ns > 1000000000ull) return W4A8_ERR_INVALID_ARG;   // at most one second
    if (reinterpret_cast<uintptr_t>(elapsed_ns_dev) & 7u) return W4A8_ERR_BAD_ALIGNMENT;
    int rc = check_device();
    if (rc != W4A8_OK) return rc;
    unsigned int* status = status_word_ptr();
    if (!status) return W4A8_ERR_CUDA;
    bounded_wait_selftest_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(
        (unsigned long long)limit_ns, reinterpret_cast<unsigned long long*>(elapsed_ns_dev), status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_status();
}

int w4a8_query_device_status(unsigned int* flags_host) {
    if (!flags_host) return W4A8_ERR_INVALID_ARG;
    unsigned int v = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return W4A8_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&v, g_status_word, sizeof v) != cudaSuccess) return W4A8_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_status_word, &zero, sizeof zero) != cudaSuccess) return W4A8_ERR_CUDA;
    *flags_host = v;
    if (v & (kStatusTimeout | kStatusPlacement)) return W4A8_ERR_TIMEOUT;   // outputs of some launch are incomplete
    return (v != 0) ? W4A8_ERR_BAD_SHAPE : W4A8_OK;
}

uint64_t w4a8_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* w4a8_status_string(int status) {
    switch (status) {
        case W4A8_OK: return "ok";
        case W4A8_ERR_INVALID_ARG: return "invalid argument";
        case W4A8_ERR_BAD_SHAPE: return "unsupported shape";
        case W4A8_ERR_BAD_ALIGNMENT: return "pointer or leading dimension not 16-byte aligned";
        case W4A8_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case W4A8_ERR_UNSUPPORTED_DEVICE: return "device is not compute capability 10.x";
        case W4A8_ERR_CUDA: return "CUDA call failed";
        case W4A8_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        default: return "unknown status";
    }
}

}  // extern "C"
