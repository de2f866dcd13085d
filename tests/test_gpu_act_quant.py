"""GPU parity: w4a8_quantize_act against the oracle's Eq. 13, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_dev, dev
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _run(xb, scale_mode=0, static_scale=None):
    x = bf16_dev(xb)
    ss = None if static_scale is None else torch.tensor([static_scale], dtype=torch.float32, device="cuda")
    x8, s_x = binding.quantize_act(x, scale_mode, ss)
    torch.cuda.synchronize()
    return x8.cpu().numpy(), s_x.cpu().numpy()


@pytest.mark.parametrize("M,K", [(1, 128), (3, 512), (16, 1024), (5, 2048), (7, 4096), (4, 8192),
                                 (2, 14336), (3, 16384), (2, 16384 + 1024), (33, 4096 + 16)])
@pytest.mark.parametrize("mode", [0, 1])
def test_bit_exact_against_oracle(M, K, mode):
    xb = inputs.make_activation(M, K, seed=M * 131 + K, outlier_frac=0.01, outlier_mult=20.0)
    x8, s = _run(xb, mode)
    rx8, rs = oracle.quantize_act(xb, scale_mode=mode)
    assert np.array_equal(s.view(np.uint32), rs.view(np.uint32))
    assert np.array_equal(x8, rx8)


def test_zero_rows_static_scale_and_signed_zero():
    xb = inputs.make_activation(6, 1024, seed=9, outlier_frac=0.01, outlier_mult=20.0)
    xb[2, :] = 0
    xb[3, :] = 0x8000           # all negative zeros
    xb[4, ::3] = 0x8000
    x8, s = _run(xb)
    rx8, rs = oracle.quantize_act(xb)
    assert np.array_equal(x8, rx8) and np.array_equal(s, rs)
    assert s[2] == 1.0 and np.all(x8[2] == 0) and np.all(x8[3] == 0x80)
    x8, s = _run(xb, static_scale=0.01)
    rx8, rs = oracle.quantize_act(xb, static_scale=0.01)
    assert np.array_equal(x8, rx8) and np.array_equal(s, rs)


def test_tiny_and_huge_magnitudes():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal((8, 512)) * np.exp2(rng.uniform(-30, 30, size=(8, 1)))).astype(np.float32)
    x[0, :] *= np.exp2(rng.uniform(-12, 0, size=512)).astype(np.float32)    # wide dynamic range in one row
    xb = inputs.f32_to_bf16_bits(x)
    for mode in (0, 1):
        x8, s = _run(xb, mode)
        rx8, rs = oracle.quantize_act(xb, scale_mode=mode)
        assert np.array_equal(x8, rx8) and np.array_equal(s, rs)


def test_strided_rows_and_full_size_config():
    # leading dimensions larger than K, and the largest activation of the decode/prefill configs
    M, K = 64, 4096
    xb = inputs.make_activation(M, K + 64, seed=3, outlier_frac=0.01, outlier_mult=20.0)
    x = bf16_dev(xb)[:, :K]
    x8_full = torch.zeros((M, K + 32), dtype=torch.uint8, device="cuda")
    s_x = torch.empty(M, dtype=torch.float32, device="cuda")
    binding.quantize_act(x, out=(x8_full[:, :K], s_x))
    torch.cuda.synchronize()
    rx8, rs = oracle.quantize_act(np.ascontiguousarray(xb[:, :K]))
    assert np.array_equal(x8_full[:, :K].cpu().numpy(), rx8)
    assert np.all(x8_full[:, K:].cpu().numpy() == 0)       # padding untouched
    assert np.array_equal(s_x.cpu().numpy(), rs)
    xb = inputs.make_activation(2048, 4096, seed=5, outlier_frac=0.01, outlier_mult=20.0)
    x8, s = _run(xb)
    rx8, rs = oracle.quantize_act(xb)
    assert np.array_equal(x8, rx8) and np.array_equal(s, rs)
