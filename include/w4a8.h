/*
 * w4a8.h -- C ABI of the B200 (sm_100a) W4A8 linear-layer library.
 *
 * The library implements the inference flow of Sec. 3 of "Dual Precision Quantization":
 * weights stored as INT4 codes with group-wise scales are dequantized to FP8 E4M3 (Eq. 10),
 * activations are quantized from BF16 to FP8 (Eq. 13), the product runs as an FP8 matrix
 * multiplication with FP32 accumulation and the result is rescaled (Eq. 4, Eq. 11) to BF16.
 *
 * Conventions shared by every entry point
 *   - Pointers named *_dev / unqualified tensor pointers are DEVICE pointers owned by the
 *     caller (any allocator); pointers named *_host are HOST pointers.  The library never
 *     allocates or frees device memory and keeps no tensor state between calls.
 *   - `stream` is a cudaStream_t passed as void*.  Work is enqueued on it and the call returns
 *     without synchronising, unless stated otherwise.
 *   - Return value: W4A8_OK (0) or a negative W4A8_ERR_* code.  Arguments are validated before
 *     anything is launched; on error nothing has been enqueued.
 *   - Tensor formats
 *       X      BF16  [M][ldx]      activations, row = token                       (Sec. 3)
 *       X8     E4M3  [M][ldx8]     bytes, OCP "fn" variant, max finite 448        (Sec. 2.2, 4.1)
 *       s_x    FP32  [M]           per-token activation scale                      (Eq. 13)
 *       codes  u8    [N][K/2]      INT4 codes u in 0..15, element k in byte k/2,
 *                                  even k in the low nibble; row = output channel  (Eq. 9)
 *       gscale BF16  [N][K/128]    group scale s_g, groups of 128 consecutive k    (Eq. 8, Eq. 14)
 *       gzero  u8    [N][K/128]    zero-point z_g in 0..15; NULL = symmetric, z=8  (Eq. 8, Eq. 1)
 *       s_w    FP32  [N] or [1]    weight FP8 scale, per channel or per tensor     (Eq. 6)
 *       W8     E4M3  [N][K]        dequantized weights                             (Eq. 10)
 *       Y      BF16 or FP32 [M][ldy]                                               (Sec. 3)
 *   - Shape rules: group must be 128, K % 128 == 0, N % 16 == 0, M >= 1.  Base pointers must be
 *     16-byte aligned and leading dimensions must keep rows 16-byte aligned.
 */
#ifndef W4A8_H
#define W4A8_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define W4A8_OK 0
#define W4A8_ERR_INVALID_ARG (-1)         /* NULL pointer, non-positive size, unknown enum */
#define W4A8_ERR_BAD_SHAPE (-2)           /* K % 128, group != 128, N % 16, ... */
#define W4A8_ERR_BAD_ALIGNMENT (-3)       /* pointer or leading dimension not 16-byte aligned */
#define W4A8_ERR_WORKSPACE_TOO_SMALL (-4)
#define W4A8_ERR_UNSUPPORTED_DEVICE (-5)  /* current device is not compute capability 10.x */
#define W4A8_ERR_CUDA (-6)                /* a CUDA runtime / driver call failed */
#define W4A8_ERR_TIMEOUT (-7)             /* a bounded device-side wait gave up (see w4a8_query_device_status) */

#define W4A8_SCALE_EXACT 0 /* s_x = amax / 448 */
#define W4A8_SCALE_POW2 1  /* s_x rounded up to a power of two (Sec. 2.2) */

#define W4A8_OUT_BF16 0
#define W4A8_OUT_FP32 1

#define W4A8_ALGO_AUTO 0
#define W4A8_ALGO_SIMT 1 /* plain CUDA-core kernel: slow, for cross-checks (canonical weights only) */
#define W4A8_ALGO_UMMA 2 /* TMA + tcgen05 kernel, one tile per CTA (canonical weights only) */

/*
 * Weight storage formats.  CANONICAL is the boundary format described above (codes, gscale,
 * gzero as separate row-major arrays).  The TILED formats are produced offline by
 * w4a8_prepack_weight from the canonical arrays and hold the same information rearranged so
 * that one 128-row x 128-k block (codes, scales, zero-points) is one contiguous chunk:
 *   TILED          any codes and zero-points (the paper's asymmetric INT4 included);
 *   TILED_SIGNMAG  symmetric storage only (gzero == NULL, z = 8) with every code in 1..15, as the
 *                  symmetric quantizer of Eq. 1 produces; codes are kept as sign and magnitude
 *                  of (u - 8), which makes the Eq. 10 expansion cheaper.
 */
#define W4A8_FMT_CANONICAL 0
#define W4A8_FMT_TILED 1
#define W4A8_FMT_TILED_SIGNMAG 2
#define W4A8_FMT_TILED_FP8 3 /* FP8 E4M3 weights, tiled by w4a8_prepack_fp8: the W8A8 comparison scheme in w4a8_linear_chain */

/*
 * Activation FP8 quantization, Eq. 13 (with Eq. 3), one scale per token:
 *   amax = max_k |X[m][k]|;  s_x[m] = amax / 448 (fp32 division; 1 when the row is all zero);
 *   X8[m][k] = nearest_E4M3( X[m][k] * (448 / amax) )   -- one fp32 multiply, round-to-nearest-even,
 *   saturating at +-448.  scale_mode W4A8_SCALE_POW2 rounds s_x up to a power of two and scales
 *   exactly.  static_scale (device pointer to one float) != NULL selects the paper's static
 *   per-tensor mode: s_x[m] = *static_scale for every row, values beyond the range saturate.
 * K % 16 == 0; ldx % 8 == 0; ldx8 % 16 == 0.  Inputs must be finite.
 */
int w4a8_quantize_act(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* x8,
                      int64_t ldx8, float* s_x, int scale_mode, const float* static_scale,
                      void* stream);

/*
 * INT4 -> FP8 weight dequantization, Eq. 10 (Eq. 14 per group):
 *   W8[n][k] = nearest_E4M3( (u[n][k] - z_g) * s_g ),  g = k / 128,
 * a single rounding (to nearest even, saturating) of the exact product.
 */
int w4a8_dequant_weight(const uint8_t* codes, const void* gscale_bf16, const uint8_t* gzero,
                        int64_t N, int64_t K, int group, uint8_t* w8, void* stream);

/*
 * The W4A8 linear layer of Sec. 3 on already-quantized activations:
 *   Y[m][n] = s_x[m] * s_w[n*sw_stride] * sum_k X8[m][k] * W8[n][k]     (Eq. 4, Eq. 11)
 * with W8 produced on the fly from (codes, gscale, gzero) exactly as w4a8_dequant_weight
 * defines it, FP8 x FP8 products accumulated in FP32, output rounded to BF16 (out_dtype 0) or
 * kept in FP32 (out_dtype 1).  sw_stride is 1 (per channel) or 0 (per tensor).
 * weight_format selects how `weights` is read: W4A8_FMT_CANONICAL (weights = codes, with
 * gscale_bf16 / gzero) or a tiled format (weights = buffer written by w4a8_prepack_weight;
 * gscale_bf16 and gzero are ignored and may be NULL).
 * `workspace` holds fp32 partial tiles when the reduction over K is split between CTAs (they are
 * added in a fixed order: results repeat bit for bit).  Calls with M <= 128 on tiled
 * weights use it only for layers with few output channels and run without it, somewhat slower,
 * when it is NULL or too small; larger M requires it.  (With 17..128 tokens such layers normally
 * need none: the CTAs that share a tile form a thread-block cluster and exchange their partial
 * sums through shared memory, again added in a fixed order.)  It
 * needs w4a8_linear_workspace_bytes(M, N, K, weight_format) bytes and may be NULL when that is
 * 0.  For the tiled formats the workspace must have been zero-filled once (cudaMemset) before
 * its first use; every call leaves it ready for the next one, whatever that call's shape is (one
 * workspace of the largest size may serve all layers of a model) -- except a call during which a
 * bounded wait gave up (w4a8_query_device_status returns W4A8_ERR_TIMEOUT): zero-fill the
 * workspace again after that.  Calls that share a workspace must not overlap on the device.
 * Calls with M <= 16 on tiled weights place their worker CTAs at run time (at most one per SM and
 * launch, so that consecutive launches can share the SMs).  The bookkeeping (1 KB, cleared by the
 * kernel) lives in the workspace when one of the full size is given -- nothing more to observe
 * than the rule above: calls that may overlap on the device need different workspaces; calls
 * issued one after the other on one stream may share one.  Without a workspace it is an entry of a
 * 64-entry table in the library image, handed out round-robin over all such calls of the process
 * (a captured call keeps the entry it drew at capture): then no more than 64 such launches may be
 * in flight on a device at a time, replays of graphs captured far apart included.
 */
int w4a8_linear(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* weights,
                const void* gscale_bf16, const uint8_t* gzero, int weight_format, const float* s_w,
                int sw_stride, int64_t N, int64_t K, int group, void* y, int64_t ldy, int out_dtype,
                void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of workspace w4a8_linear needs for this problem (0 when none is used). */
size_t w4a8_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int weight_format);

/*
 * Offline re-layout of the stored weights (no arithmetic on values): canonical codes, scales and
 * zero-points -> a tiled buffer of w4a8_prepack_bytes(N, K, weight_format) bytes (128-byte
 * aligned) for weight_format W4A8_FMT_TILED or W4A8_FMT_TILED_SIGNMAG.  The dequantized weights
 * the linear layer sees are bit-identical to Eq. 10 on the canonical arrays.  If a code 0 is met
 * while writing W4A8_FMT_TILED_SIGNMAG, bit 1 of the device status word is raised
 * (w4a8_query_device_status) and the buffer must not be used.
 */
size_t w4a8_prepack_bytes(int64_t N, int64_t K, int weight_format);

/*
 * W8A8 comparison scheme (Sec. 4.3, Fig. 4) for the chain launch: re-layout (no arithmetic) of FP8
 * E4M3 weights w8 [N][K] -- e.g. the output of w4a8_dequant_weight -- into the tiled order
 * [K/128][N/8][8 chunks][8 rows][16 bytes] (N * K bytes, 128-byte aligned) that
 * w4a8_linear_chain reads with weight_format W4A8_FMT_TILED_FP8: the same kernel, partition and
 * MMAs as for the INT4 formats, the expansion replaced by a copy -- twice the weight bytes, no
 * integer work.  N % 16 == 0, K % 128 == 0.
 */
int w4a8_prepack_fp8(const uint8_t* w8, int64_t N, int64_t K, uint8_t* out, size_t out_bytes, void* stream);
int w4a8_prepack_weight(const uint8_t* codes, const void* gscale_bf16, const uint8_t* gzero, int64_t N,
                        int64_t K, int group, int weight_format, uint8_t* out, size_t out_bytes,
                        void* stream);

/*
 * Same computation as w4a8_linear with the kernel choice exposed, for cross-checks and tuning:
 * canonical weights only.  algo is W4A8_ALGO_*; split_k <= 0 lets the library choose, otherwise
 * it is the number of K slices (must divide K/128).  Workspace need:
 * w4a8_linear_ex_workspace_bytes (no zero-fill needed).
 */
int w4a8_linear_ex(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M,
                   const uint8_t* codes, const void* gscale_bf16, const uint8_t* gzero,
                   const float* s_w, int sw_stride, int64_t N, int64_t K, int group, void* y,
                   int64_t ldy, int out_dtype, void* workspace, size_t workspace_bytes, int algo,
                   int split_k, void* stream);
size_t w4a8_linear_ex_workspace_bytes(int64_t M, int64_t N, int64_t K, int algo, int split_k);

/*
 * Variant of w4a8_linear_ex (canonical weights, W4A8_ALGO_UMMA) for callers that cannot hand the
 * library a workspace.  (The paper has no counterpart; this is a deployment convenience.)
 * Typical cases: an inference-engine plugin whose enqueue hook receives only its input and
 * output tensors and is forbidden to allocate; a latency-critical serving loop in which a
 * cudaMalloc would stall the whole device; a process whose memory pool has been handed out in
 * full before the layer is first run.
 * The split-K partial sums live in an array that is part of the library image itself
 * (W4A8_STATIC_SCRATCH_BYTES bytes, resident on every GPU that loads the library until the
 * process exits).  The call allocates and frees nothing, on the host or on the device.
 *   - split_k <= 0 lets the library choose; the partial sums need split_k * M * N * 4 bytes, and
 *     a problem that needs more than W4A8_STATIC_SCRATCH_BYTES is rejected with
 *     W4A8_ERR_WORKSPACE_TOO_SMALL before anything is launched.
 *   - The first call on each device looks up the device address of the array (a synchronous
 *     runtime query).  Make that first call outside of any stream capture; later calls only
 *     enqueue kernels.
 *   - All calls on a device share the one array.  Each call overwrites every partial sum it
 *     later reads, so nothing has to be cleared between calls and stale contents are harmless,
 *     but two calls whose kernels overlap on the GPU (different streams, or graphs replayed
 *     concurrently) would race on it: serialise them.
 * Arguments and results are those of w4a8_linear_ex.
 */
#define W4A8_STATIC_SCRATCH_BYTES (4u << 20)
int w4a8_linear_static_scratch(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M,
                               const uint8_t* codes, const void* gscale_bf16, const uint8_t* gzero,
                               const float* s_w, int sw_stride, int64_t N, int64_t K, int group, void* y,
                               int64_t ldy, int out_dtype, int split_k, void* stream);

/*
 * A chain of decode-sized layers in ONE persistent launch (Sec. 3 inference flow for every
 * problem of the chain: Eq. 13 activation quantization, Eq. 10 weight dequantization, FP8 GEMM,
 * Eq. 4 / Eq. 11 epilogue; Sec. 1 on the memory-bound regime of small batches this is for).
 * Problem i computes  y_i = Linear_i( quantize_act( in_i ) )  with
 *   in_i = x_i                                   (input_kind W4A8_CHAIN_INPUT_PLAIN), or
 *   in_i = BF16( silu(G) * U ), G|U = x_i        (W4A8_CHAIN_INPUT_SILU_MUL: x_i has 2 K columns, gate
 *                                                 first, exactly as w4a8_silu_mul_quantize defines it),
 * and the results are those of w4a8_quantize_act (or w4a8_silu_mul_quantize) followed by
 * w4a8_linear on the same tiled weights with K not cut: same scales, same FP8 codes, same
 * accumulation order -- for the output channels whose K range one CTA walks alone; where the chain
 * cuts K (see below) the FP32 partial sums are added in a fixed order, so results still repeat bit
 * for bit from call to call, and agree with w4a8_linear within its output tolerance.  Problems run
 * in array order on one grid of one CTA per SM that stays resident for the whole chain; the packed
 * weights of the next problem are fetched while the current one is multiplied.
 * Partition: the output channels are cut into blocks of 96; while at least as many blocks as SMs
 * are left every CTA takes whole blocks, the remaining blocks are cut along K as well, into runs of
 * at least four 128-wide k-blocks, and the CTA that holds a block's lowest k range adds the
 * partial sums of the others (FP32, through the workspace) before it scales and writes the rows.
 *   x_bf16       device BF16 [M][ldx] (ldx % 8 == 0, 16-byte aligned), M <= W4A8_CHAIN_MAX_M.  x_bf16 and
 *                y may also be device-side addresses of page-locked host buffers
 *                (w4a8_host_buffer_device_pointer): decode-sized activations and outputs are small
 *                enough to be read and written over the bus by the kernel itself.
 *   depends_on   -1 when x_bf16 is complete before the call; otherwise the index (< i) of the
 *                problem of this chain that WRITES the memory x_bf16 points into (normally
 *                x_bf16 == that problem's y, out_dtype BF16): problem i is not quantized before
 *                every row of that output has been written.  Buffers of problems that are not
 *                linked this way must not overlap.
 *   scale_mode, static_scale    as in w4a8_quantize_act.
 *   weights      device, output of w4a8_prepack_weight (W4A8_FMT_TILED, W4A8_FMT_TILED_SIGNMAG) or, for
 *                the W8A8 comparison scheme, of w4a8_prepack_fp8 (W4A8_FMT_TILED_FP8: the weights are
 *                FP8 bytes, copied instead of expanded); one weight_format for the whole chain.
 *                K % 128 == 0, K <= 16384, N % 16 == 0, N <= 1152 rows per SM.
 *   x8_out / s_x_out  optional (NULL): row-major copies of the FP8 activations [M][ldx8_out] and
 *                of the M scales the layer multiplied with.
 * workspace: device, 128-byte aligned, w4a8_linear_chain_workspace_bytes(problems, count) bytes:
 * hand-over counters, activation scales, the FP8 activations as MMA operand tiles and the
 * partial sums of the blocks that are cut along K.  It must
 * have been zero-filled once before its first use; every launch leaves the counters zero again
 * (the last CTA to leave clears them, also after a time-out).  Launches that share a workspace
 * must not overlap on the device; launches enqueued one after the other on one stream may share it.
 * groups: 0 = the library's choice, 2..4 = number of 3-warp expansion groups (for tuning).
 * Every device-side wait (on a pipeline barrier or on a hand-over counter) is bounded: when one
 * runs out, all CTAs stop, outputs are incomplete and bit 0 of the device status word is set
 * (w4a8_query_device_status returns W4A8_ERR_TIMEOUT).
 * `problems` is a HOST array, read during the call only.  Errors: W4A8_ERR_INVALID_ARG (NULL,
 * count outside 1..W4A8_CHAIN_MAX_PROBLEMS, bad enum, depends_on >= i, mixed weight formats, an
 * input that is the FP32 output of the problem it depends on),
 * W4A8_ERR_BAD_SHAPE (M > 16, K % 128, N % 16, N too large, leading dimensions),
 * W4A8_ERR_BAD_ALIGNMENT, W4A8_ERR_WORKSPACE_TOO_SMALL; nothing is enqueued on error.
 */
#define W4A8_CHAIN_INPUT_PLAIN 0
#define W4A8_CHAIN_INPUT_SILU_MUL 1
#define W4A8_CHAIN_MAX_PROBLEMS 24
#define W4A8_CHAIN_MAX_M 16
typedef struct w4a8_chain_problem {
    const void* x_bf16;
    int64_t ldx;
    int32_t input_kind;
    int32_t depends_on;
    int32_t scale_mode;
    int32_t weight_format;
    const float* static_scale;
    const uint8_t* weights;
    const float* s_w;
    int32_t sw_stride;
    int32_t out_dtype;
    int64_t M, N, K;
    void* y;
    int64_t ldy;
    uint8_t* x8_out;
    int64_t ldx8_out;
    float* s_x_out;
} w4a8_chain_problem;
size_t w4a8_linear_chain_workspace_bytes(const w4a8_chain_problem* problems_host, int count);
int w4a8_linear_chain(const w4a8_chain_problem* problems_host, int count, void* workspace,
                      size_t workspace_bytes, int groups, void* stream);

/*
 * Device-side address of a page-locked HOST buffer (cudaHostAlloc / cudaHostRegister memory that
 * is mapped into the device's address space), for callers that want a kernel of this library to
 * read its activations from, or write its outputs to, host memory directly: w4a8_linear_chain
 * accepts such addresses for x_bf16 and y (the bytes then cross the bus inside the kernel, with
 * no copy-engine operation).  *dev_out receives the address; W4A8_ERR_INVALID_ARG when the
 * buffer is pageable memory (which a kernel must not touch) or not host memory at all.  (A
 * deployment helper; the paper has no counterpart.)
 */
int w4a8_host_buffer_device_pointer(const void* host, void** dev_out);

/*
 * Self-test of the bounded device-side waits (the mechanism every kernel of the library uses; the
 * paper has no counterpart): launches one CTA that waits, with a limit of `limit_ns` nanoseconds,
 * on a pipeline barrier nobody ever arrives on.  The kernel must come back by itself, with bit 0 of
 * the device status word set.  `elapsed_ns_dev` (device, one uint64, may be NULL) receives the time
 * the wait took.  Nothing faults, traps or spins without a limit.
 */
int w4a8_selftest_bounded_wait(uint64_t limit_ns, uint64_t* elapsed_ns_dev, void* stream);

/*
 * W4A16 comparison scheme (Sec. 4.3, Fig. 4): activations stay BF16, the INT4 codes are expanded
 * to BF16 on the fly and multiplied with BF16 tensor-core MMAs, FP32 accumulation:
 *   W16[n][k] = BF16( (u[n][k] - z[n][g]) * s_g[n][g] )      (one rounding to nearest even),
 *   Y[m][n]   = s_w[n*sw_stride] * sum_k X[m][k] * W16[n][k],  rounded to BF16 or kept in FP32.
 * The stored weights are those of the W4A8 path (canonical format: codes, BF16 group scales,
 * zero-points or NULL for z = 8, s_w per channel or per tensor), so the two schemes can be timed on
 * the same quantized layer; only the arithmetic of the multiplication differs.
 *   x_bf16 device BF16 [M][ldx] (ldx % 8 == 0, 16-byte aligned); K % 128 == 0, N % 16 == 0.
 * One 128-channel tile per CTA; with few tokens and few tiles K is cut into slices whose FP32
 * partial sums go through `workspace` (device, 16-byte aligned, at least
 * w4a8_linear_w4a16_workspace_bytes(M, N, K) bytes, owned by the caller, may be NULL when that is
 * 0) and are summed by a second kernel.  Errors as w4a8_linear, W4A8_ERR_WORKSPACE_TOO_SMALL
 * included.
 */
size_t w4a8_linear_w4a16_workspace_bytes(int64_t M, int64_t N, int64_t K);
int w4a8_linear_w4a16(const void* x_bf16, int64_t ldx, int64_t M, const uint8_t* codes,
                      const void* gscale_bf16, const uint8_t* gzero, const float* s_w, int sw_stride,
                      int64_t N, int64_t K, void* y, int64_t ldy, int out_dtype, void* workspace,
                      size_t workspace_bytes, void* stream);

/*
 * The same scheme on the persistent prefill kernel of the W4A8 path, for a like-for-like timing at
 * prefill sizes: prepacked weights (w4a8_prepack_weight, W4A8_FMT_TILED_SIGNMAG only: symmetric
 * storage; another format returns W4A8_ERR_INVALID_ARG), the same TMA / expansion-group / MMA /
 * epilogue roles, the codes expanded to the BF16 values defined above, kind::f16 MMAs, whole tiles
 * of 128 channels x 64, 128 or 256 tokens (by M) per CTA, no workspace.  Same result as
 * w4a8_linear_w4a16 up to the order of the FP32 additions.  Other arguments and errors as there.
 */
int w4a8_linear_w4a16_tiled(const void* x_bf16, int64_t ldx, int64_t M, const uint8_t* weights, int weight_format,
                            const float* s_w, int sw_stride, int64_t N, int64_t K, void* y, int64_t ldy,
                            int out_dtype, void* stream);

/*
 * Gated-MLP activation fused with the activation quantization of the next linear layer (the
 * paper quantizes the BF16 activations that enter a linear layer, Eq. 13; in a Llama MLP block
 * those of the down projection are silu(gate) * up, computed from the output of the stacked
 * gate/up projection):
 *   h[m][f]  = BF16( silu(G[m][f]) * U[m][f] ),  silu(g) = g / (1 + exp(-g)), evaluated in fp32,
 *   G = gate_up[m][0..F), U = gate_up[m][F..2F);
 *   (x8, s_x) = w4a8_quantize_act(h), same scale modes.
 * Saves writing h and reading it back (4 B per element) and one launch.
 *   gate_up_bf16  device BF16 [M][ldgu], ldgu >= 2 F, ldgu % 8 == 0, 16-byte aligned;
 *   F % 16 == 0, F <= 16384;  x8 device u8 [M][ldx8] (ldx8 % 16 == 0), s_x device float [M];
 *   h_bf16_out    optional (may be NULL): device BF16 [M][ldh], receives h (ldh % 8 == 0).
 * exp() comes from the CUDA math library (about 2 ulp), so h can differ from a correctly rounded
 * evaluation by one BF16 step on a small fraction of the elements; everything after h is exact
 * as in w4a8_quantize_act.  Errors as w4a8_quantize_act; W4A8_ERR_BAD_SHAPE for F > 16384.
 */
int w4a8_silu_mul_quantize(const void* gate_up_bf16, int64_t M, int64_t F, int64_t ldgu, uint8_t* x8,
                           int64_t ldx8, float* s_x, int scale_mode, const float* static_scale,
                           void* h_bf16_out, int64_t ldh, void* stream);


/*
 * Eq. 10 for weights quantized in an unconstrained activation order (the W4A8* rows of Table 3;
 * appendix "Activation Reordering"): column k takes the scale and zero-point of group g_idx[k]
 * instead of k / 128, so the groups are no longer runs of consecutive columns and the fused
 * kernels (one look-up table per row and group) do not apply -- which is the inference overhead
 * Group-Aware Reordering avoids.  This entry point materialises the FP8 weights (E4M3 bytes,
 * [N][K]) for w4a8_linear_w8a8; both launches together are the cost of that scheme.
 *   codes [N][K/2], gscale BF16 [N][G], gzero u8 [N][G] or NULL (z = 8), g_idx int32 [K] in [0, G).
 * g_idx values are not range-checked on the device.
 */
int w4a8_dequant_weight_gidx(const uint8_t* codes, const void* gscale_bf16, const uint8_t* gzero,
                             const int32_t* g_idx, int64_t N, int64_t K, int64_t G, uint8_t* w8, void* stream);

/*
 * The W4A8 linear layer on activation-ordered weights in ONE kernel (the W4A8* rows of Table 3;
 * appendix "Activation Reordering"): as w4a8_linear on canonical weights, except that column k of
 * the weights takes the scale and zero-point of group g_idx[k] (device int32 [K], values in
 * [0, K / 128), not range-checked on the device).  No look-up table can be shared by the columns of
 * a k-block, so Eq. 10 is evaluated weight by weight inside the kernel (a multiplication and a
 * conversion each, with two cached loads for the group's scale and zero-point): what this costs
 * against w4a8_linear on the same layer is the inference overhead of an unconstrained activation
 * order.  The FP8 weights it multiplies with are those of w4a8_dequant_weight_gidx, so the result
 * equals w4a8_linear_w8a8 on that output bit for bit.  Workspace:
 * w4a8_linear_ex_workspace_bytes(M, N, K, W4A8_ALGO_UMMA, 0) bytes.  Other arguments and errors
 * as in w4a8_linear_ex; W4A8_ERR_INVALID_ARG for a NULL or misaligned g_idx.
 */
int w4a8_linear_gidx(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* codes,
                     const void* gscale_bf16, const uint8_t* gzero, const int32_t* g_idx, const float* s_w,
                     int sw_stride, int64_t N, int64_t K, int group, void* y, int64_t ldy, int out_dtype,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * W8A8 comparison scheme (Sec. 4.3, Fig. 4): the same FP8 GEMM and epilogue on weights that are
 * stored as FP8 E4M3 bytes -- e.g. the output of w4a8_dequant_weight -- so that the cost of
 * streaming twice the bytes can be set against the cost of expanding INT4 on the fly, on the
 * same device and with the same MMA code.  w8: device u8 [N][K], 16-byte aligned.  Workspace:
 * w4a8_linear_ex_workspace_bytes(M, N, K, W4A8_ALGO_UMMA, 0) bytes (fp32 split-K partials).
 * Other arguments and errors as in w4a8_linear.
 */
int w4a8_linear_w8a8(const uint8_t* x8, int64_t ldx8, const float* s_x, int64_t M, const uint8_t* w8,
                     const float* s_w, int sw_stride, int64_t N, int64_t K, void* y, int64_t ldy, int out_dtype,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * Offline round-to-nearest weight quantizer (Eq. 6 -> 7 -> 8 -> 9, no error compensation),
 * so that a caller can produce the stored format on the device.  W is FP32 [N][K].
 *   symmetric != 0: s_g = max|w8| / 7, u = round(w8 / s_g) + 8 (codes 1..15), gzero may be NULL;
 *   symmetric == 0: Eq. 8 / Eq. 9 with the range widened to contain 0; gzero required.
 *   pow2 != 0: s_g rounded up to a power of two.  per_channel != 0: s_w has N entries, else 1.
 * Group scales are rounded to BF16 before the codes are computed; the integer rounding is
 * half-to-even.  Enqueues several kernels on `stream`.
 */
int w4a8_quantize_weight_rtn(const float* W, int64_t N, int64_t K, int group, int symmetric,
                             int pow2, int per_channel, uint8_t* codes, void* gscale_bf16,
                             uint8_t* gzero, float* s_w, void* stream);

/*
 * The layer Hessian the quantizer works with (Sec. 3.1; prepared as in Sec. 3.3): H = X^T X over the T
 * calibration tokens of the layer's input X (device BF16 [T][ldx]), FP32 sums, written as a full
 * symmetric matrix (device float [K][K]); accumulate != 0 adds to what H holds (batches of tokens).
 * Its diagonal is what w4a8_gar_permutation ranks by.  K <= 32768.
 */
int w4a8_hessian_accumulate(const void* x_bf16, int64_t T, int64_t K, int64_t ldx, float* H, int accumulate,
                            void* stream);

/*
 * Sec. 3.3 (dampening as in GPTQ): H_out = the Hessian in processing order -- rows and columns
 * permuted by perm (device int32 [K] from w4a8_gar_permutation, or NULL) --, with a unit diagonal
 * for input features whose diagonal entry is zero, and damp * mean(diag) added to the diagonal
 * (the mean taken after the unit-diagonal rule).  scratch: one device float.  H_out != H.
 * What remains between this matrix and the factor U that w4a8_dpq_quantize takes -- the inverse
 * and its upper Cholesky factor -- is a library factorization and the caller's.
 */
int w4a8_hessian_prepare(const float* H, int64_t K, const int32_t* perm, float damp, float* H_out, float* scratch,
                         void* stream);

/*
 * Group-Aware Reordering (Sec. 3.2 and its appendix): the order in which the DPQ quantizer
 * processes the input features, from the diagonal of the Hessian H = X^T X.  Inside each group
 * of 128 the columns go by descending diagonal, the groups by descending maximum diagonal (the
 * ranking the paper used); ties keep the original order.
 *   hdiag  device float [K];  perm  device int32 [K]: position p handles original column perm[p].
 *   workspace  device, w4a8_gar_workspace_bytes(K) bytes (scratch, no initialisation needed).
 */
size_t w4a8_gar_workspace_bytes(int64_t K);
int w4a8_gar_permutation(const float* hdiag, int64_t K, int group, int32_t* perm, void* workspace,
                         size_t workspace_bytes, void* stream);

/*
 * DPQ weight quantizer, Algorithm 1 (Sec. 3.1-3.3): Eq. 6, then per row and per group of 128
 * (in processing order) Eq. 8 -- optionally with the search of the scale of least squared error
 * of Sec. 3.3 -- and per weight Eq. 7, 9, 10, 11 followed by the error-compensating update of
 * Eq. 12 in its Cholesky form (Sec. 3.3, as in GPTQ): e = (w - w16^) / U_qq, w_v <- w_v - e U_qv.
 * Produces the same stored format as w4a8_quantize_weight_rtn, in the ORIGINAL column order.
 *   W     device fp32 [N][K], 16-byte aligned.
 *   U     device fp32 [K][K]: upper Cholesky factor of the inverse of the (dampened) Hessian with
 *         rows and columns in processing order; only the upper triangle is read.  H = X^T X and its
 *         preparation are w4a8_hessian_accumulate / w4a8_hessian_prepare; the two factorizations
 *         in between (inverse, Cholesky) are a library matter and the caller's.
 *   perm  device int32 [K] from w4a8_gar_permutation, or NULL for the original order.  Every run
 *         of 128 positions must hold the columns of one original group (not checked on the device).
 *   symmetric / per_channel   as in w4a8_quantize_weight_rtn (gzero may be NULL when symmetric).
 *   mse_steps  0 or 1: Eq. 8 as is; 2..11: that many shrink factors 1, 0.98, 0.96, ... are tried.
 *   workspace  device, 16-byte aligned, w4a8_dpq_workspace_bytes(N, K) bytes (scratch).
 * Every step that decides a code is a single correctly rounded fp32 operation, so the codes are
 * reproducible and independent of the launch geometry.  Enqueues about 2 K / 128 kernels.
 */
size_t w4a8_dpq_workspace_bytes(int64_t N, int64_t K);
int w4a8_dpq_quantize(const float* W, int64_t N, int64_t K, int group, const float* U, const int32_t* perm,
                      int symmetric, int mse_steps, int per_channel, uint8_t* codes, void* gscale_bf16,
                      uint8_t* gzero, float* s_w, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Whole layer from HOST activations to HOST output (Sec. 3 flow end to end): copies
 * x_host (BF16 [M][K], ideally pinned) to x_dev, runs w4a8_quantize_act and w4a8_linear, and
 * copies y_dev (BF16 [M][N]) to y_host, all enqueued on `stream`; the caller synchronises the
 * stream before reading y_host.  Weights stay resident on the device.  Scratch device buffers
 * are the caller's: x_dev (2*M*K bytes), x8_dev (M*K), s_x_dev (4*M), y_dev (2*M*N), workspace.
 * For M <= 128, when both host buffers are page-locked (pinned or registered, 16-byte aligned),
 * no copy is enqueued: the quantization kernel reads x_host and the linear kernel writes y_host
 * through their device mappings -- the same bytes cross the bus, without two copy-engine
 * operations; x_dev and y_dev are then left untouched.  Pageable buffers and larger M take the
 * copies.  x8_dev and s_x_dev hold the quantized activations afterwards in both cases.
 */
int w4a8_forward_host(const void* x_host_bf16, int64_t M, const uint8_t* weights,
                      const void* gscale_bf16, const uint8_t* gzero, int weight_format, const float* s_w,
                      int sw_stride, int64_t N, int64_t K, int group, void* y_host_bf16,
                      void* x_dev, uint8_t* x8_dev, float* s_x_dev, void* y_dev, void* workspace,
                      size_t workspace_bytes, void* stream);

/*
 * Reads and clears the device-side status word (synchronises the device).  *flags receives a
 * bit mask: bit 0 = a bounded wait inside a kernel gave up; bit 1 = w4a8_prepack_weight met a
 * code its target format cannot hold; bit 2 = the run-time placement of a decode launch
 * (w4a8_linear, M <= 16 on tiled weights) ended with a worker index unissued.  Bits 0 and 2 mean
 * that the outputs of some launch are incomplete: returns W4A8_ERR_TIMEOUT; W4A8_ERR_BAD_SHAPE when
 * only bit 1 was set, W4A8_OK otherwise.  After W4A8_ERR_TIMEOUT the workspaces of w4a8_linear
 * calls that were in flight must be zero-filled again before they are reused (their split-K
 * counters and placement state may have been left part-way); the workspace of w4a8_linear_chain
 * needs no such care (its last CTA clears it after an aborted launch too).
 */
int w4a8_query_device_status(unsigned int* flags_host);

/* Number of kernels the library has launched from this process (for accounting). */
uint64_t w4a8_launch_count(void);

/* Static string for a status code. */
const char* w4a8_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif
