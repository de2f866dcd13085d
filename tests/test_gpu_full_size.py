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
    edge = [0, 1, 127, 128, 129, 255, 256, N // 2 - 1, N // 2, N - 257, N - 129, N - 128, N - 1]
    top = int(np.argmax(np.max(np.abs(W), axis=1)))  # the channel that fixes the per-tensor scale
    rows = np.unique(np.concatenate([rng.choice(N, n_random, replace=False), np.array(edge + [top])]))
    return rows.astype(np.int64)


def _run_case(M, N, K, sigma, frac, mult, seed, n_random):
    W = inputs.make_weight(N, K, sigma, seed)
    rows = _sample_channels(N, W, n_random, seed)
    Wd = torch.from_numpy(W).cuda()
    codes, gscale, gzero, s_w = binding.quantize_weight_rtn(Wd, symmetric=True)
    del Wd
    # oracle quantization of the sampled channels == the GPU's
    oc, og, oz, osw = oracle.quantize_weight_rtn(W[rows], symmetric=True)
    del W
    assert oz is None and gzero is None
    ridx = torch.from_numpy(rows).cuda()
    assert np.array_equal(codes[ridx].cpu().numpy(), oc)
    assert np.array_equal(bf16_bits(gscale[ridx]), og)
    assert np.array_equal(s_w.cpu().numpy().view(np.uint32), osw.view(np.uint32))
    tw = binding.prepack_weight(codes, gscale, gzero, s_w)
    del codes, gscale
    assert binding.query_device_status() == 0

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
    ref = oracle.linear(x8_ref, s_x_ref, oracle.dequant_weight(oc, og, None), osw, want=("y64",))
    ok, dist = bf16_gate(bf16_bits(y[:, ridx]), ref["y64"])
    assert ok, dist


def test_config_c4_prefill_sampled_channels():
    # c4: M=8192, K=8192, N=28672, sigma 0.015, 0.5 % outlier channels x30
    _run_case(8192, 28672, 8192, 0.015, 0.005, 30.0, seed=4, n_random=24)


@pytest.mark.parametrize("name,K,N,M", [("qkv", 4096, 6144, 512), ("o", 4096, 4096, 128),
                                        ("gate_up", 4096, 28672, 4096), ("down", 14336, 4096, 4096),
                                        ("down", 14336, 4096, 32), ("gate_up", 4096, 28672, 8)])
def test_config_c5_layers_sampled_channels(name, K, N, M):
    # c5: the four Llama-3-8B linears; token counts that reach the split-N kernel (<= 64), the
    # persistent kernel with shared tiles (128, 512) and with whole tiles (4096)
    _run_case(M, N, K, 0.02, 0.01, 20.0, seed=500 + M + N // 64, n_random=40)


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
