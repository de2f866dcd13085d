"""GPU parity of the W4A16 comparison kernel (Sec. 4.3) against its oracle: BF16 activations, INT4
codes expanded to BF16 with one rounding, FP32 accumulation in the tensor core.  Small-integer
inputs give results that must be exact (layout test); Gaussian inputs must be within 2e-3 relative
before the BF16 cast and within one BF16 step after it."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_bits, bf16_dev, weights_to_dev
from helpers import bf16_gate, fp32_gate
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _bf16(v):
    return int(np.array([v], dtype=np.float32).view(np.uint32)[0] >> 16)


@pytest.mark.parametrize("M,N,K", [(1, 16, 128), (16, 128, 256), (5, 144, 384), (64, 256, 512), (37, 400, 1024),
                                   (128, 128, 128), (200, 272, 640), (24, 256, 1024), (3, 256, 4096)])
def test_exact_on_small_integers(M, N, K):
    codes, _, gzero = inputs.random_codes(N, K, 40 + M, asymmetric=True)
    gs = np.full((N, K // 128), _bf16(1.0), dtype=np.uint16)
    gs[::3] = _bf16(0.5)                                   # a second exact scale
    s_w = (np.arange(N, dtype=np.float32) % 4 + 1) * 0.25  # per channel, exact
    xb = inputs.make_small_int_activation(M, K, 50 + N)
    ref = oracle.linear_w4a16(xb, oracle.dequant_weight_bf16(codes, gs, gzero), s_w)
    wd = weights_to_dev(codes, gs, gzero, s_w)
    y = binding.linear_w4a16(bf16_dev(xb), *wd, out_dtype=binding.OUT_FP32)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert np.array_equal(y.cpu().numpy().astype(np.float64), ref)


@pytest.mark.parametrize("M,N,K", [(4, 1024, 1024), (16, 512, 4096), (96, 640, 2048), (300, 1152, 1024)])
@pytest.mark.parametrize("asym", [False, True])
def test_gaussian_within_gates(M, N, K, asym):
    W = inputs.make_weight(N, K, 0.02, 61)
    codes, gscale, gzero, s_w = oracle.quantize_weight_rtn(W, symmetric=not asym, per_channel=asym)
    xb = inputs.make_activation(M, K, 62, 0.01, 20.0)
    ref = oracle.linear_w4a16(xb, oracle.dequant_weight_bf16(codes, gscale, gzero), s_w)
    wd = weights_to_dev(codes, gscale, gzero, s_w)
    x = bf16_dev(xb)
    y32 = binding.linear_w4a16(x, *wd, out_dtype=binding.OUT_FP32)
    ybf = binding.linear_w4a16(x, *wd, out_dtype=binding.OUT_BF16)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    worst, _ = fp32_gate(y32.cpu().numpy(), ref, rel=2e-3)
    assert worst <= 2e-3, worst
    ok, dist = bf16_gate(bf16_bits(ybf), ref)
    assert ok, dist


def test_outputs_beyond_the_problem_are_untouched():
    M, N, K = 7, 48, 256
    codes, gscale, gzero, s_w = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, 5), symmetric=True)
    xb = inputs.make_activation(M, K, 6)
    y = torch.full((M + 3, N + 16), 7.0, dtype=torch.float32, device="cuda")
    binding.linear_w4a16(bf16_dev(xb), *weights_to_dev(codes, gscale, gzero, s_w), out=y[:M, :N],
                         out_dtype=binding.OUT_FP32)
    torch.cuda.synchronize()
    assert torch.all(y[M:] == 7.0) and torch.all(y[:, N:] == 7.0)


def test_split_k_workspace_is_required_and_sized():
    M, N, K = 4, 256, 4096                                  # two tiles, 32 k-blocks: K is cut into slices
    need = int(binding.lib().w4a8_linear_w4a16_workspace_bytes(M, N, K))
    assert need > 0 and need % (M * N * 4) == 0
    assert int(binding.lib().w4a8_linear_w4a16_workspace_bytes(4096, 4096, 4096)) == 0
    codes, gscale, gzero, s_w = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, 9), symmetric=True)
    wd = weights_to_dev(codes, gscale, gzero, s_w)
    x = bf16_dev(inputs.make_activation(M, K, 10))
    small = torch.empty((need - 16,), dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.W4A8Error) as e:
        binding.linear_w4a16(x, *wd, workspace=small)
    assert "workspace" in str(e.value).lower()
    y = binding.linear_w4a16(x, *wd, workspace=torch.empty((need,), dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0 and torch.isfinite(y.float()).all()


# ---- the same scheme on the persistent prefill kernel (prepacked sign-magnitude weights) ----

def _symmetric_integer_case(M, N, K, seed):
    codes, _, _ = inputs.random_codes(N, K, seed)
    u = np.clip(np.stack([codes & 15, codes >> 4], axis=-1).reshape(N, K), 1, 15).astype(np.uint8)   # the symmetric quantizer never emits 0
    codes = (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)
    gs = np.full((N, K // 128), _bf16(1.0), dtype=np.uint16)
    gs[::3] = _bf16(0.5)
    s_w = (np.arange(N, dtype=np.float32) % 4 + 1) * 0.25
    return codes, gs, s_w


@pytest.mark.parametrize("M,N,K", [(1, 16, 128), (16, 128, 256), (64, 256, 512), (37, 400, 1024), (128, 128, 128),
                                   (200, 272, 640), (300, 2064, 1152), (129, 19072, 384), (600, 272, 640),
                                   (1030, 4112, 256)])
def test_tiled_exact_on_small_integers(M, N, K):
    # ragged token and channel tiles of 64, 128 and 256 tokens, one to many tiles per CTA (two shapes have
    # more tiles than SMs)
    codes, gs, s_w = _symmetric_integer_case(M, N, K, 140 + M)
    xb = inputs.make_small_int_activation(M, K, 150 + N)
    ref = oracle.linear_w4a16(xb, oracle.dequant_weight_bf16(codes, gs, None), s_w)
    tw = binding.prepack_weight(*weights_to_dev(codes, gs, None, s_w))
    assert tw.fmt == binding.FMT_TILED_SIGNMAG
    y = binding.linear_w4a16_tiled(bf16_dev(xb), tw, out_dtype=binding.OUT_FP32)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert np.array_equal(y.cpu().numpy().astype(np.float64), ref)


@pytest.mark.parametrize("M,N,K,pc", [(16, 512, 4096, False), (96, 640, 2048, True), (300, 1152, 1024, False),
                                      (1000, 2048, 2048, True)])
def test_tiled_gaussian_within_gates_and_equal_to_the_tile_kernel(M, N, K, pc):
    W = inputs.make_weight(N, K, 0.02, 71)
    codes, gscale, gzero, s_w = oracle.quantize_weight_rtn(W, symmetric=True, per_channel=pc)
    xb = inputs.make_activation(M, K, 72, 0.01, 20.0)
    ref = oracle.linear_w4a16(xb, oracle.dequant_weight_bf16(codes, gscale, gzero), s_w)
    wd = weights_to_dev(codes, gscale, gzero, s_w)
    tw = binding.prepack_weight(*wd)
    x = bf16_dev(xb)
    y32 = binding.linear_w4a16_tiled(x, tw, out_dtype=binding.OUT_FP32)
    ybf = binding.linear_w4a16_tiled(x, tw, out_dtype=binding.OUT_BF16)
    y32_again = binding.linear_w4a16_tiled(x, tw, out_dtype=binding.OUT_FP32)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert torch.equal(y32, y32_again)
    worst, _ = fp32_gate(y32.cpu().numpy(), ref, rel=2e-3)
    assert worst <= 2e-3, worst
    ok, dist = bf16_gate(bf16_bits(ybf), ref)
    assert ok, dist


def test_tiled_rejects_other_formats_and_leaves_padding_alone():
    M, N, K = 70, 272, 256
    codes, gscale, gzero, s_w = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, 5), symmetric=True)
    wd = weights_to_dev(codes, gscale, gzero, s_w)
    x = bf16_dev(inputs.make_activation(M, K, 6))
    generic = binding.prepack_weight(*wd, weight_format=binding.FMT_TILED)
    with pytest.raises(binding.W4A8Error):
        binding.linear_w4a16_tiled(x, generic)
    tw = binding.prepack_weight(*wd)
    y = torch.full((M + 3, N + 16), 7.0, dtype=torch.float32, device="cuda")
    binding.linear_w4a16_tiled(x, tw, out=y[:M, :N], out_dtype=binding.OUT_FP32)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert torch.all(y[M:] == 7.0) and torch.all(y[:, N:] == 7.0)
