"""GPU parity at the full sizes of the larger workloads, on sampled output channels.

The whole problem runs on the GPU in the launch configuration the benchmark times (prepacked
sign-magnitude weights, w4a8_quantize_act then w4a8_linear, BF16 output); the oracle follows
Sec. 3 (Eq. 13 -> Eq. 10 -> exact FP8 dot products -> Eq. 4 / Eq. 11) for every token but only a
sample of output channels: seeded random ones plus the channels next to tile boundaries.  The
weights are quantized on the GPU for all channels and by the oracle for the sampled ones, which
must agree bit for bit (the sample contains the channel that holds the tensor's absolute maximum,
so both see the same per-tensor scale, Eq. 6)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_bits, bf16_dev, weights_to_dev
from helpers import bf16_gate, fp32_gate
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _sample_channels(N, W, n_random, seed):
    rng = np.random.default_rng(seed)
    edge = [0, 1, 95, 96, 97, 127, 128, 129, 191, 192, 255, 256, N // 2 - 1, N // 2, N - 257, N - 129, N - 128, N - 33,
            N - 32, N - 1]
    edge += [r for r in (148 * 96 - 1, 148 * 96, 2 * 148 * 96 - 1, 2 * 148 * 96) if r < N]   # 96-row blocks: last whole one / first cut along K
    top = int(np.argmax(np.max(np.abs(W), axis=1)))  # the channel that fixes the per-tensor scale
    rows = np.unique(np.concatenate([rng.choice(N, n_random, replace=False), np.array(edge + [top])]))
    return rows.astype(np.int64)


def _quantized_layer(N, K, sigma, seed, n_random, symmetric=True):
    """Weights quantized on the GPU for all channels and by the oracle for a sample of them (which
    must agree bit for bit), prepacked.  Returns (tiled weight, sampled rows, oracle weights)."""
    W = inputs.make_weight(N, K, sigma, seed)
    rows = _sample_channels(N, W, n_random, seed)
    Wd = torch.from_numpy(W).cuda()
    codes, gscale, gzero, s_w = binding.quantize_weight_rtn(Wd, symmetric=symmetric)
    del Wd
    oc, og, oz, osw = oracle.quantize_weight_rtn(W[rows], symmetric=symmetric)
    del W
    ridx = torch.from_numpy(rows).cuda()
    assert np.array_equal(codes[ridx].cpu().numpy(), oc)
    assert np.array_equal(bf16_bits(gscale[ridx]), og)
    assert (oz is None) == (gzero is None)
    if oz is not None:
        assert np.array_equal(gzero[ridx].cpu().numpy(), oz)
    assert np.array_equal(s_w.cpu().numpy().view(np.uint32), osw.view(np.uint32))
    tw = binding.prepack_weight(codes, gscale, gzero, s_w)      # generic tiled format when asymmetric
    del codes, gscale
    assert binding.query_device_status() == 0
    return tw, rows, ridx, (oc, og, oz, osw)


def _run_case(M, N, K, sigma, frac, mult, seed, n_random, symmetric=True):
    tw, rows, ridx, (oc, og, oz, osw) = _quantized_layer(N, K, sigma, seed, n_random, symmetric)
    xb = inputs.make_activation(M, K, seed, frac, mult)
    x = bf16_dev(xb)
    x8, s_x = binding.quantize_act(x)
    ws = binding.new_workspace(M, N, K, tw.fmt)
    y = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_BF16, workspace=ws)
    y2 = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_BF16, workspace=ws)  # workspace reuse
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))

    x8_ref, s_x_ref = oracle.quantize_act(xb)
    assert np.array_equal(x8.cpu().numpy(), x8_ref)
    assert np.array_equal(s_x.cpu().numpy().view(np.uint32), s_x_ref.view(np.uint32))
    ref = oracle.linear(x8_ref, s_x_ref, oracle.dequant_weight(oc, og, oz), osw, want=("y64",))
    ok, dist = bf16_gate(bf16_bits(y[:, ridx]), ref["y64"])
    assert ok, dist


def test_config_c4_prefill_sampled_channels():
    # c4: M=8192, K=8192, N=28672, sigma 0.015, 0.5 % outlier channels x30
    _run_case(8192, 28672, 8192, 0.015, 0.005, 30.0, seed=4, n_random=24)


@pytest.mark.parametrize("name,K,N,M", [("qkv", 4096, 6144, 512), ("o", 4096, 4096, 128),
                                        ("gate_up", 4096, 28672, 4096), ("down", 14336, 4096, 4096),
                                        ("down", 14336, 4096, 32), ("gate_up", 4096, 28672, 8),
                                        ("qkv", 4096, 6144, 1), ("qkv", 4096, 6144, 32),
                                        ("o", 4096, 4096, 1), ("o", 4096, 4096, 32),
                                        ("gate_up", 4096, 28672, 128), ("down", 14336, 4096, 128)])
def test_config_c5_layers_sampled_channels(name, K, N, M):
    # c5: the four Llama-3-8B linears; token counts that reach the split-N kernel (<= 64: the
    # smallest layers there take the K-cut path), its 128-token tiles (128), the persistent kernel
    # with shared tiles (512) and with whole tiles (4096)
    _run_case(M, N, K, 0.02, 0.01, 20.0, seed=500 + M + N // 64, n_random=40)


@pytest.mark.parametrize("K,N,M", [(4096, 14336, 16), (4096, 6144, 2048)])
def test_asymmetric_storage_at_layer_size_sampled_channels(K, N, M):
    # the paper's stored format is asymmetric INT4 (Sec. 2.1, Sec. 4.1): zero-points per group, the
    # generic tiled layout, at Llama layer sizes on the decode and on the prefill kernel
    _run_case(M, N, K, 0.02, 0.01, 20.0, seed=900 + M, n_random=40, symmetric=False)


def test_chain_launch_at_c2_size_and_gated_block_at_layer_size():
    # The launch the benchmark times: M = 1, 4, 16 on the c2 layer (K = 4096, N = 14336) as three
    # problems of one w4a8_linear_chain launch, then a Llama-3-8B MLP block as a dependent chain
    # (gate/up -> silu(gate) * up quantized in the kernel -> down).  FP8 activations and scales bit
    # for bit; outputs on sampled channels, every stage on the input that stage saw.
    tw, rows, ridx, (oc, og, oz, osw) = _quantized_layer(14336, 4096, 0.02, 41, 40)
    w8 = oracle.dequant_weight(oc, og, oz)
    probs, xbs = [], []
    for M in (1, 4, 16):
        xb = inputs.make_activation(M, 4096, 40 + M, 0.01, 20.0)
        xbs.append(xb)
        probs.append(dict(x=bf16_dev(xb), weight=tw, y=torch.zeros((M, 14336), dtype=torch.bfloat16, device="cuda"),
                          x8_out=torch.zeros((M, 4096), dtype=torch.uint8, device="cuda"),
                          s_x_out=torch.zeros((M,), dtype=torch.float32, device="cuda")))
    chain = binding.LinearChain(probs)
    chain()
    chain()      # a second launch on the same workspace
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    for d, xb in zip(probs, xbs):
        x8_ref, s_x_ref = oracle.quantize_act(xb)
        assert np.array_equal(d["x8_out"].cpu().numpy(), x8_ref)
        assert np.array_equal(d["s_x_out"].cpu().numpy().view(np.uint32), s_x_ref.view(np.uint32))
        ref = oracle.linear(x8_ref, s_x_ref, w8, osw, want=("y64",))
        ok, dist = bf16_gate(bf16_bits(d["y"][:, ridx]), ref["y64"])
        assert ok, dist
    del tw, probs, chain

    H, F, M = 4096, 14336, 4
    tw_gu, rows_gu, ridx_gu, (gc, gg, gz, gsw) = _quantized_layer(2 * F, H, 0.02, 42, 40)
    tw_dn, rows_dn, ridx_dn, (dc, dg, dz, dsw) = _quantized_layer(H, F, 0.02, 43, 40)
    xb = inputs.make_activation(M, H, 44, 0.01, 20.0)
    gu = torch.zeros((M, 2 * F), dtype=torch.bfloat16, device="cuda")
    dn = torch.zeros((M, H), dtype=torch.bfloat16, device="cuda")
    h8 = torch.zeros((M, F), dtype=torch.uint8, device="cuda")
    sh = torch.zeros((M,), dtype=torch.float32, device="cuda")
    binding.LinearChain([dict(x=bf16_dev(xb), weight=tw_gu, y=gu),
                         dict(x=gu, weight=tw_dn, y=dn, kind=binding.CHAIN_INPUT_SILU_MUL, depends_on=0,
                              x8_out=h8, s_x_out=sh)])()
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    x8_ref, s_x_ref = oracle.quantize_act(xb)
    ref = oracle.linear(x8_ref, s_x_ref, oracle.dequant_weight(gc, gg, gz), gsw, want=("y64",))
    ok, dist = bf16_gate(bf16_bits(gu[:, ridx_gu]), ref["y64"])
    assert ok, dist
    want8, wants = binding.silu_mul_quantize(gu)      # the same arithmetic on the same input
    torch.cuda.synchronize()
    assert torch.equal(h8, want8) and torch.equal(sh, wants)
    ref = oracle.linear(h8.cpu().numpy(), sh.cpu().numpy(), oracle.dequant_weight(dc, dg, dz), dsw, want=("y64",))
    ok, dist = bf16_gate(bf16_bits(dn[:, ridx_dn]), ref["y64"])
    assert ok, dist


def test_two_cta_kernel_shape_exact_integers_and_gaussian():
    """A shape that the two-CTA kernel takes (many output channels, few token tiles), with a
    ragged token count: small-integer inputs make the FP32 accumulation exact, so any operand
    that lands in the wrong row, token half or k-slice changes the result visibly; then Gaussian inputs
    within the usual gates.  Sampled output channels (all 128-row blocks are hit)."""
    M, N, K = 1061, 16384, 1024
    rng = np.random.default_rng(17)
    cols = np.unique(np.concatenate([rng.integers(0, N, 700), np.arange(0, N, 128), np.arange(127, N, 128)]))
    for exact in (True, False):
        if exact:
            codes, gscale, gzero = inputs.random_codes(N, K, 5, scale_bits=0x3F80)       # group scale 1.0
            s_w = np.array([1.0], dtype=np.float32)
            xb = inputs.make_small_int_activation(M, K, 6)
        else:
            W = inputs.make_weight(N, K, 0.02, 23)
            codes, gscale, gzero, s_w = oracle.quantize_weight_rtn(W, symmetric=True)
            xb = inputs.make_activation(M, K, 24, 0.01, 20.0)
        x8_ref, s_x_ref = oracle.quantize_act(xb)
        w8 = oracle.dequant_weight(codes, gscale, gzero)
        ref = oracle.linear(x8_ref, s_x_ref, w8, s_w, cols=cols, want=("y64",))
        # random codes include 0 (= -8), which only the generic tiled format can hold
        fmt = binding.FMT_TILED if exact else binding.FMT_TILED_SIGNMAG
        tw = binding.prepack_weight(*weights_to_dev(codes, gscale, gzero, s_w), weight_format=fmt)
        x8, s_x = binding.quantize_act(bf16_dev(xb))
        y = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_FP32)
        torch.cuda.synchronize()
        assert binding.query_device_status() == 0
        got = y.cpu().numpy()[:, cols]
        if exact:
            # the integer dot products are exact in FP32; what remains is the rounding of the two scale
            # multiplications (s_x = amax / 448 is not a power of two): a misplaced operand would change
            # a sum by at least one unit, i.e. by 1/112 here
            assert np.all(np.abs(got.astype(np.float64) - ref["y64"]) <= 4e-7 * np.abs(ref["y64"]) + 1e-6)
        else:
            worst, _ = fp32_gate(got, ref["y64"], rel=2e-3)
            assert worst <= 2e-3, worst


def test_wide_tile_kernel_shape_exact_integers_and_gaussian():
    """A shape that the prefill kernel with tiles of 256 output channels x 256 tokens takes (whole
    tiles fill the SMs well), ragged in both directions -- the last token tile has 120 tokens, the
    last channel tile 80 rows -- and with more tiles than SMs, so that some CTAs run a second tile
    on the same accumulators.  Small-integer inputs (exact FP32 sums: a misplaced operand changes a
    result by at least one unit) in the generic tiled format, then Gaussian inputs in the
    sign-magnitude format within the usual gates.  Sampled output channels: the first and last row of
    every 128-row block."""
    M, N, K = 1400, 10576, 640
    rng = np.random.default_rng(31)
    cols = np.unique(np.concatenate([rng.integers(0, N, 500), np.arange(0, N, 128), np.arange(127, N, 128),
                                     np.array([N - 81, N - 80, N - 1])]))
    for exact in (True, False):
        if exact:
            codes, gscale, gzero = inputs.random_codes(N, K, 7, scale_bits=0x3F80)       # group scale 1.0
            s_w = np.array([1.0], dtype=np.float32)
            xb = inputs.make_small_int_activation(M, K, 8)
        else:
            W = inputs.make_weight(N, K, 0.02, 33)
            codes, gscale, gzero, s_w = oracle.quantize_weight_rtn(W, symmetric=True)
            xb = inputs.make_activation(M, K, 34, 0.01, 20.0)
        x8_ref, s_x_ref = oracle.quantize_act(xb)
        w8 = oracle.dequant_weight(codes, gscale, gzero)
        ref = oracle.linear(x8_ref, s_x_ref, w8, s_w, cols=cols, want=("y64",))
        fmt = binding.FMT_TILED if exact else binding.FMT_TILED_SIGNMAG
        tw = binding.prepack_weight(*weights_to_dev(codes, gscale, gzero, s_w), weight_format=fmt)
        x8, s_x = binding.quantize_act(bf16_dev(xb))
        y = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_FP32)
        yb = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_BF16)
        torch.cuda.synchronize()
        assert binding.query_device_status() == 0
        got = y.cpu().numpy()[:, cols]
        if exact:
            assert np.all(np.abs(got.astype(np.float64) - ref["y64"]) <= 4e-7 * np.abs(ref["y64"]) + 1e-6)
        else:
            worst, _ = fp32_gate(got, ref["y64"], rel=2e-3)
            assert worst <= 2e-3, worst
            ok, dist = bf16_gate(bf16_bits(yb)[:, cols], ref["y64"])
            assert ok, dist
