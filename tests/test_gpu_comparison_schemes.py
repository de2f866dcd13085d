"""GPU parity of the comparison schemes around the W4A8 path (Sec. 4.3, Table 3 '*' rows):
w4a8_linear_w8a8 (FP8 weights, no expansion) and w4a8_dequant_weight_gidx (activation-ordered
groups) against the oracle.  FP8 bytes bit-exact; outputs within 2e-3 relative / 1 BF16 step."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_bits, bf16_dev, dev, weights_to_dev
from helpers import bf16_gate, fp32_gate, unpack_codes
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,K", [(1, 16, 128), (16, 1024, 1024), (5, 144, 384), (100, 512, 2048),
                                   (300, 640, 1024), (16, 14336, 4096)])
def test_w8a8_linear_matches_oracle(M, N, K):
    wq = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, 31), symmetric=True)
    w8 = oracle.dequant_weight(*wq[:3])
    x8, s_x = oracle.quantize_act(inputs.make_activation(M, K, 31, 0.01, 20.0))
    ref = oracle.linear(x8, s_x, w8, wq[3])
    y32 = binding.linear_w8a8(dev(x8), dev(s_x), dev(w8), dev(wq[3]), out_dtype=binding.OUT_FP32)
    ybf = binding.linear_w8a8(dev(x8), dev(s_x), dev(w8), dev(wq[3]), out_dtype=binding.OUT_BF16)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    worst, _ = fp32_gate(y32.cpu().numpy(), ref["y64"], rel=2e-3)
    assert worst <= 2e-3, worst
    ok, dist = bf16_gate(bf16_bits(ybf), ref["y64"])
    assert ok, dist


def test_w8a8_equals_w4a8_on_the_same_fp8_weights():
    # same FP8 operands, same MMA and accumulation order per tile: the two schemes give the same bits
    M, N, K = 16, 1024, 1024
    wq = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, 32), symmetric=True)
    wd = weights_to_dev(*wq)
    x8, s_x = binding.quantize_act(bf16_dev(inputs.make_activation(M, K, 32, 0.01, 20.0)))
    y4 = binding.linear(x8, s_x, *wd, out_dtype=binding.OUT_FP32, algo=binding.ALGO_UMMA)
    y8 = binding.linear_w8a8(x8, s_x, binding.dequant_weight(*wd[:3]), wd[3], out_dtype=binding.OUT_FP32)
    torch.cuda.synchronize()
    assert torch.equal(y4.view(torch.int32), y8.view(torch.int32))


@pytest.mark.parametrize("asym", [False, True])
def test_gidx_dequant_matches_oracle(asym):
    rng = np.random.default_rng(33)
    N, K = 96, 1024
    W = inputs.make_weight(N, K, 0.02, 33)
    perm = rng.permutation(K)
    codes_p, gs, gz, s_w = oracle.quantize_weight_rtn(W[:, perm], symmetric=not asym)
    u_p = unpack_codes(codes_p)
    u = np.empty_like(u_p)
    u[:, perm] = u_p
    codes = (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)
    g_idx = np.empty(K, dtype=np.int32)
    g_idx[perm] = np.arange(K) // 128
    ref = oracle.dequant_weight_gidx(codes, gs, gz, g_idx)
    got = binding.dequant_weight_gidx(dev(codes), bf16_dev(gs), None if gz is None else dev(gz), dev(g_idx))
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy(), ref)


@pytest.mark.parametrize("asym", [False, True])
@pytest.mark.parametrize("M,N,K", [(1, 16, 128), (16, 1024, 1024), (5, 144, 384), (100, 512, 2048), (300, 640, 1024)])
def test_gidx_linear_in_one_kernel(M, N, K, asym):
    # w4a8_linear_gidx: activation-ordered weights (scattered groups), Eq. 10 weight by weight inside
    # the GEMM kernel.  Against the oracle (its g_idx dequantization + the exact matmul) within the
    # usual gates, and bit for bit against the two-launch route (w4a8_dequant_weight_gidx, then
    # w4a8_linear_w8a8): same FP8 weights, same MMAs in the same order.
    rng = np.random.default_rng(100 + M + N)
    W = inputs.make_weight(N, K, 0.02, 34)
    perm = rng.permutation(K)
    codes_p, gs, gz, s_w = oracle.quantize_weight_rtn(W[:, perm], symmetric=not asym)
    u_p = unpack_codes(codes_p)
    u = np.empty_like(u_p)
    u[:, perm] = u_p
    codes = (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)
    g_idx = np.empty(K, dtype=np.int32)
    g_idx[perm] = np.arange(K) // 128
    x8, s_x = oracle.quantize_act(inputs.make_activation(M, K, 35, 0.01, 20.0))
    w8_ref = oracle.dequant_weight_gidx(codes, gs, gz, g_idx)
    ref = oracle.linear(x8, s_x, w8_ref, s_w)
    cd, gd, zd, gi, sw = dev(codes), bf16_dev(gs), None if gz is None else dev(gz), dev(g_idx), dev(s_w)
    y32 = binding.linear_gidx(dev(x8), dev(s_x), cd, gd, zd, gi, sw, out_dtype=binding.OUT_FP32)
    ybf = binding.linear_gidx(dev(x8), dev(s_x), cd, gd, zd, gi, sw, out_dtype=binding.OUT_BF16)
    w8 = binding.dequant_weight_gidx(cd, gd, zd, gi)
    two = binding.linear_w8a8(dev(x8), dev(s_x), w8, sw, out_dtype=binding.OUT_FP32)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert np.array_equal(w8.cpu().numpy(), w8_ref)
    assert torch.equal(y32.view(torch.int32), two.view(torch.int32))
    worst, _ = fp32_gate(y32.cpu().numpy(), ref["y64"], rel=2e-3)
    assert worst <= 2e-3, worst
    ok, dist = bf16_gate(bf16_bits(ybf), ref["y64"])
    assert ok, dist
    # consecutive groups: the look-up reduces to Eq. 10 with one scale per 128 columns = w4a8_linear
    gi0 = dev((np.arange(K) // 128).astype(np.int32))
    wq = oracle.quantize_weight_rtn(W, symmetric=not asym)
    wd = weights_to_dev(*wq)
    a = binding.linear_gidx(dev(x8), dev(s_x), wd[0], wd[1], wd[2], gi0, wd[3], out_dtype=binding.OUT_FP32)
    b = binding.linear(dev(x8), dev(s_x), *wd, out_dtype=binding.OUT_FP32, algo=binding.ALGO_UMMA)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_w8a8_on_the_persistent_kernel_at_prefill_size():
    # enough 128 x 256 tiles for every SM: w4a8_linear_w8a8 runs the persistent kernel of the W4A8 path
    # with the expansion compiled out (FP8 weight tiles by TMA straight into the operand ring).  Ragged
    # in both directions; against the oracle on sampled channels, and bit for bit against w4a8_linear on
    # the same FP8 weights (same operands, same k order of the FP32 accumulation).
    M, N, K = 1900, 5008, 1024
    rng = np.random.default_rng(7)
    wq = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, 36), symmetric=True)
    cols = np.unique(np.concatenate([rng.integers(0, N, 300), np.arange(0, N, 128), np.arange(127, N, 128), [N - 1]]))
    w8 = oracle.dequant_weight(*wq[:3])
    x8, s_x = oracle.quantize_act(inputs.make_activation(M, K, 37, 0.01, 20.0))
    ref = oracle.linear(x8, s_x, w8, wq[3], cols=cols, want=("y64",))
    wd = weights_to_dev(*wq)
    y8 = binding.linear_w8a8(dev(x8), dev(s_x), dev(w8), dev(wq[3]), out_dtype=binding.OUT_FP32)
    y8b = binding.linear_w8a8(dev(x8), dev(s_x), dev(w8), dev(wq[3]), out_dtype=binding.OUT_BF16)
    tw = binding.prepack_weight(*wd)
    y4 = binding.linear_tiled(dev(x8), dev(s_x), tw, out_dtype=binding.OUT_FP32)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    worst, _ = fp32_gate(y8.cpu().numpy()[:, cols], ref["y64"], rel=2e-3)
    assert worst <= 2e-3, worst
    ok, dist = bf16_gate(bf16_bits(y8b)[:, cols], ref["y64"])
    assert ok, dist
    assert torch.equal(y8.view(torch.int32), y4.view(torch.int32))
