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
from gpu_utils import bf16_bits, bf16_dev
from helpers import bf16_gate
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
