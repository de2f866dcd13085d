"""GPU parity: w4a8_linear_fused (activation quantization inside the decode kernel) against the
oracle's whole forward (Sec. 3 flow: Eq. 13 -> Eq. 10 -> FP8 matmul -> Eq. 4 / Eq. 11).  The FP8
activations and scales the kernel used are read back and must be bit-exact; the output gate is
max relative error 2e-3 before the BF16 cast and 1 BF16 step after it."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_bits, bf16_dev, dev, weights_to_dev
from helpers import bf16_gate, fp32_gate
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _prepacked(wq, generic=False):
    wd = weights_to_dev(*wq)
    fmt = binding.FMT_TILED if (generic or wq[2] is not None) else binding.FMT_TILED_SIGNMAG
    return binding.prepack_weight(*wd, weight_format=fmt)


def _run(xb, wq, generic=False, pow2=False, static_scale=None):
    M, K = xb.shape
    tw = _prepacked(wq, generic)
    x = bf16_dev(xb)
    mode = binding.SCALE_POW2 if pow2 else binding.SCALE_EXACT
    ss = None if static_scale is None else dev(np.array([static_scale], dtype=np.float32))
    x8 = torch.full((M, K), 0xAA, dtype=torch.uint8, device="cuda")
    s_x = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
    y32 = binding.linear_fused(x, tw, out_dtype=binding.OUT_FP32, scale_mode=mode, static_scale=ss,
                               x8_out=x8, s_x_out=s_x)
    ybf = binding.linear_fused(x, tw, out_dtype=binding.OUT_BF16, scale_mode=mode, static_scale=ss)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    return y32.cpu().numpy(), bf16_bits(ybf), x8.cpu().numpy(), s_x.cpu().numpy()


def _check(xb, wq, generic=False, pow2=False, static_scale=None):
    x8_ref, s_x_ref = oracle.quantize_act(xb, scale_mode=1 if pow2 else 0, static_scale=static_scale)
    ref = oracle.linear(x8_ref, s_x_ref, oracle.dequant_weight(*wq[:3]), wq[3])
    ref["x8"], ref["s_x"] = x8_ref, s_x_ref
    y32, ybf, x8, s_x = _run(xb, wq, generic, pow2, static_scale)
    assert np.array_equal(s_x.view(np.uint32), ref["s_x"].astype(np.float32).view(np.uint32))
    assert np.array_equal(x8, ref["x8"])
    worst, _ = fp32_gate(y32, ref["y64"], rel=2e-3)
    assert worst <= 2e-3, worst
    ok, dist = bf16_gate(ybf, ref["y64"])
    assert ok, dist


@pytest.mark.parametrize("M,N,K", [(1, 16, 128), (3, 16, 256), (16, 128, 512), (5, 144, 384), (16, 1024, 1024),
                                   (7, 2368, 640), (16, 4736, 128), (2, 37888, 256), (1, 40960, 128),
                                   (16, 48, 14336)])
@pytest.mark.parametrize("asym", [False, True])
def test_fused_matches_oracle_forward(M, N, K, asym):
    # shapes: one range per CTA, ragged ranges, two 128-row blocks per range (N > 128*148),
    # several ranges per CTA (N > 256*148), an odd number of k-blocks, a long K
    W = inputs.make_weight(N, K, 0.02, 21)
    wq = oracle.quantize_weight_rtn(W, symmetric=not asym, per_channel=asym)
    xb = inputs.make_activation(M, K, 21, 0.01, 20.0)
    _check(xb, wq)


def test_fused_generic_tiled_format_and_scale_modes():
    M, N, K = 9, 1024, 1024
    W = inputs.make_weight(N, K, 0.02, 22)
    wq = oracle.quantize_weight_rtn(W, symmetric=True)
    xb = inputs.make_activation(M, K, 22, 0.01, 20.0)
    _check(xb, wq, generic=True)
    _check(xb, wq, pow2=True)
    _check(xb, wq, static_scale=0.0625)


def test_fused_zero_and_saturating_rows():
    # an all-zero token takes scale 1; a static scale far too small saturates at +-448
    M, N, K = 4, 256, 512
    W = inputs.make_weight(N, K, 0.02, 23)
    wq = oracle.quantize_weight_rtn(W, symmetric=True)
    xb = inputs.make_activation(M, K, 23, 0.01, 20.0)
    xb[1, :] = 0
    xb[2, ::2] = 0x8000  # negative zeros
    _check(xb, wq)
    _check(xb, wq, static_scale=1e-4)


@pytest.mark.parametrize("M", [1, 4, 16])
def test_fused_config_c2_decode_full(M):
    K, N = 4096, 14336
    W = inputs.make_weight(N, K, 0.02, 2)
    wq = oracle.quantize_weight_rtn(W, symmetric=True)
    xb = inputs.make_activation(M, K, 2, 0.01, 20.0)
    _check(xb, wq)


def test_fused_equals_the_two_kernel_path_bit_for_bit():
    M, K, N = 16, 4096, 14336
    W = inputs.make_weight(N, K, 0.02, 24)
    wq = oracle.quantize_weight_rtn(W, symmetric=True)
    tw = _prepacked(wq)
    x = bf16_dev(inputs.make_activation(M, K, 24, 0.01, 20.0))
    x8, s_x = binding.quantize_act(x)
    y2 = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_FP32)
    y1 = binding.linear_fused(x, tw, out_dtype=binding.OUT_FP32)
    torch.cuda.synchronize()
    assert torch.equal(y1.view(torch.int32), y2.view(torch.int32))


def test_fused_rejects_what_it_does_not_cover():
    W = inputs.make_weight(128, 256, 0.02, 25)
    wq = oracle.quantize_weight_rtn(W, symmetric=True)
    tw = _prepacked(wq)
    x = bf16_dev(inputs.make_activation(17, 256, 25, 0.01, 20.0))
    with pytest.raises(binding.W4A8Error) as e:
        binding.linear_fused(x, tw)
    assert e.value.status == -2  # W4A8_ERR_BAD_SHAPE
    xo = torch.zeros((4, 264), dtype=torch.bfloat16, device="cuda")[:, 4:260]  # rows not 16-byte aligned
    with pytest.raises(binding.W4A8Error) as e:
        binding.linear_fused(xo, tw)
    assert e.value.status == -3  # W4A8_ERR_BAD_ALIGNMENT
