"""Invariants of the oracle's round-to-nearest INT4 quantizer (Eq. 6-9; symmetric variant of Eq. 1)."""
import numpy as np
import pytest

import oracle
from helpers import unpack_codes, bf16_bits_to_f64, e4m3_value_table
from paper_2505_14638_b200 import inputs

G = 128


def _w8_grid(W, s_w):
    """Eq. 7 recomputed with library pieces: fp32 division, then torch's E4M3 cast (in range)."""
    torch = pytest.importorskip("torch")
    q = (W / np.float32(s_w)).astype(np.float32)
    return torch.from_numpy(q).to(torch.float8_e4m3fn).float().numpy().astype(np.float64)


@pytest.mark.parametrize("symmetric", [True, False])
def test_ranges_and_error_bound(symmetric):
    W = inputs.make_weight(96, 512, 0.02, seed=2)
    codes, gs, gz, s_w = oracle.quantize_weight_rtn(W, G, symmetric=symmetric)
    u = unpack_codes(codes)
    assert u.min() >= (1 if symmetric else 0) and u.max() <= 15
    assert s_w.shape == (1,) and np.float32(np.abs(W).max()) / np.float32(448) == s_w[0]   # Eq. 6
    w8 = _w8_grid(W, s_w[0])
    assert np.abs(w8).max() == 448.0
    s = np.repeat(bf16_bits_to_f64(gs), G, axis=1)
    z = np.full(u.shape, 8.0) if symmetric else np.repeat(gz.astype(np.float64), G, axis=1)
    if not symmetric:
        assert gz.min() >= 0 and gz.max() <= 15
    recon = (u - z) * s
    # unclipped elements are within half a step (Eq. 8-10); BF16 rounding of the scale can clip the
    # extreme element of a group by a fraction of a step, never more than one step
    err = np.abs(w8 - recon)
    qf = w8 / s + z
    unclipped = (qf >= (1 if symmetric else 0) - 0.5) & (qf <= 15.5)
    assert np.all(err[unclipped] <= s[unclipped] / 2 + 1e-9)
    assert np.all(err <= s * 1.01)


@pytest.mark.parametrize("symmetric", [True, False])
def test_requantizing_the_reconstruction_is_a_fixed_point(symmetric):
    W = inputs.make_weight(32, 256, 0.02, seed=5)
    codes, gs, gz, s_w = oracle.quantize_weight_rtn(W, G, symmetric=symmetric, pow2=True)
    # with power-of-two group scales (u - z) * s is on the E4M3 grid, so quantizing the dequantized
    # weights (times s_w) again must return the same codes
    w8 = oracle.dequant_weight(codes, gs, gz, G)
    vals = e4m3_value_table()[w8]
    u = unpack_codes(codes).astype(np.float64)
    s = np.repeat(bf16_bits_to_f64(gs), G, axis=1)
    z = np.full(u.shape, 8.0) if symmetric else np.repeat(gz.astype(np.float64), G, axis=1)
    assert np.array_equal(vals, (u - z) * s)
    sb = bf16_bits_to_f64(gs)
    assert np.all(np.log2(sb) == np.round(np.log2(sb)))


def test_symmetric_codes_are_round_of_ratio():
    W = inputs.make_weight(16, 256, 0.02, seed=9)
    codes, gs, _, s_w = oracle.quantize_weight_rtn(W, G, symmetric=True)
    w8 = _w8_grid(W, s_w[0])
    s = np.repeat(bf16_bits_to_f64(gs), G, axis=1)
    ratio = (w8.astype(np.float32) / s.astype(np.float32)).astype(np.float32)   # fp32 division as stated
    q = np.clip(np.rint(ratio), -7, 7)
    assert np.array_equal(unpack_codes(codes), (q + 8).astype(np.int32))
    # group scale = BF16(max|w8| / 7)
    amax = np.abs(w8).reshape(16, -1, G).max(axis=2).astype(np.float32)
    assert np.array_equal(gs, inputs.f32_to_bf16_bits(amax / np.float32(7)))


def test_asymmetric_scale_and_zero_point_formulas():
    W = inputs.make_weight(16, 256, 0.02, seed=10) + np.float32(0.01)
    codes, gs, gz, s_w = oracle.quantize_weight_rtn(W, G, symmetric=False)
    w8 = _w8_grid(W, s_w[0]).reshape(16, -1, G).astype(np.float32)
    lo = np.minimum(w8.min(axis=2), 0)
    hi = np.maximum(w8.max(axis=2), 0)
    sb = inputs.f32_to_bf16_bits((hi - lo) / np.float32(15))
    assert np.array_equal(gs, sb)
    s = inputs.bf16_bits_to_f32(sb)
    z = np.clip(np.rint(-lo / s), 0, 15).astype(np.uint8)
    assert np.array_equal(gz, z)
    u = np.clip(np.rint(w8 / s[:, :, None] + z[:, :, None].astype(np.float32)), 0, 15)
    assert np.array_equal(unpack_codes(codes), u.reshape(16, -1).astype(np.int32))


def test_degenerate_groups_and_per_channel():
    W = inputs.make_weight(4, 256, 0.02, seed=1)
    W[1, :128] = 0.0
    W[2, :] = 0.0
    codes, gs, gz, s_w = oracle.quantize_weight_rtn(W, G, symmetric=False, per_channel=True)
    assert s_w.shape == (4,) and s_w[2] == 1.0
    assert s_w[0] == np.float32(np.abs(W[0]).max()) / np.float32(448)
    u = unpack_codes(codes)
    assert np.all(u[1, :128] == gz[1, 0]) and bf16_bits_to_f64(gs)[1, 0] == 1.0
    assert np.all(oracle.dequant_weight(codes, gs, gz, G)[2] == 0)
    codes, gs, _, _ = oracle.quantize_weight_rtn(W, G, symmetric=True)
    assert np.all(unpack_codes(codes)[2] == 8)
