"""GPU parity: w4a8_dequant_weight (Eq. 10) and w4a8_quantize_weight_rtn (Eq. 6-9) against the
oracle, byte for byte."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_bits, bf16_dev, dev
from helpers import pack_codes
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _dequant(codes, gs, gz):
    out = binding.dequant_weight(dev(codes), bf16_dev(gs), None if gz is None else dev(gz))
    torch.cuda.synchronize()
    return out.cpu().numpy()


def test_brute_force_all_codes_zero_points_and_bf16_scales():
    # every code x every zero-point x every finite BF16 scale bit pattern
    bits = np.arange(65536, dtype=np.uint32)
    fin = np.isfinite((bits << 16).view(np.float32))
    sb = bits[fin].astype(np.uint16)
    u_row = np.tile(np.arange(16, dtype=np.uint8), 8)
    codes = pack_codes(np.broadcast_to(u_row, (sb.size, 128)).copy())
    for z in range(16):
        gz = np.full((sb.size, 1), z, dtype=np.uint8)
        got = _dequant(codes, sb[:, None], gz)
        ref = oracle.dequant_weight(codes, sb[:, None], gz)
        assert np.array_equal(got, ref), z
    got = _dequant(codes, sb[:, None], None)
    assert np.array_equal(got, oracle.dequant_weight(codes, sb[:, None], None))


@pytest.mark.parametrize("N,K,asym", [(16, 128, False), (48, 1024, True), (1024, 1024, False),
                                      (272, 4096, True), (14336, 4096, False)])
def test_random_codes_bit_exact(N, K, asym):
    codes, gs, gz = inputs.random_codes(N, K, seed=N + K, asymmetric=asym)
    assert np.array_equal(_dequant(codes, gs, gz), oracle.dequant_weight(codes, gs, gz))


def test_quantized_gaussian_weights_bit_exact():
    W = inputs.make_weight(512, 2048, 0.02, seed=4)
    for sym in (True, False):
        codes, gs, gz, _ = oracle.quantize_weight_rtn(W, symmetric=sym)
        assert np.array_equal(_dequant(codes, gs, gz), oracle.dequant_weight(codes, gs, gz))


@pytest.mark.parametrize("sym,pow2,pc", [(True, False, False), (False, False, False), (True, True, False),
                                         (False, True, True), (True, False, True)])
def test_rtn_quantizer_matches_oracle(sym, pow2, pc):
    W = inputs.make_weight(384, 1024, 0.02, seed=6)
    W[5, :128] = 0.0
    W[7, :] = 0.0
    W[9, 256:384] = 0.013
    codes, gs, gz, s_w = binding.quantize_weight_rtn(dev(W), symmetric=sym, pow2=pow2, per_channel=pc)
    torch.cuda.synchronize()
    rc, rgs, rgz, rsw = oracle.quantize_weight_rtn(W, symmetric=sym, pow2=pow2, per_channel=pc)
    assert np.array_equal(s_w.cpu().numpy(), rsw)
    assert np.array_equal(bf16_bits(gs), rgs)
    if not sym:
        assert np.array_equal(gz.cpu().numpy(), rgz)
    assert np.array_equal(codes.cpu().numpy(), rc)
