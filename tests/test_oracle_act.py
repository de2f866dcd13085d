"""Pins for the oracle's per-token activation FP8 quantization (Eq. 13 with Eq. 3)."""
import numpy as np
import pytest

import oracle
from helpers import e4m3_encode_search, e4m3_value_table
from paper_2505_14638_b200 import inputs


def _x(M=12, K=512, seed=0):
    return inputs.make_activation(M, K, seed, outlier_frac=0.01, outlier_mult=20.0)


def test_scale_is_amax_over_448_and_argmax_hits_the_top_code():
    xb = _x()
    x = inputs.bf16_bits_to_f32(xb)
    x8, s = oracle.quantize_act(xb)
    amax = np.abs(x).max(axis=1)
    assert np.array_equal(s, amax / np.float32(448))            # Eq. 13, fp32 division
    rows = np.arange(x.shape[0])
    top = x8[rows, np.abs(x).argmax(axis=1)]
    assert np.all((top & 0x7F) == 0x7E)                         # +-448
    assert np.array_equal(top >> 7, (x[rows, np.abs(x).argmax(axis=1)] < 0).astype(np.uint8))


def test_error_is_within_half_a_grid_step():
    xb = _x(M=8, K=1024, seed=4)
    x = inputs.bf16_bits_to_f32(xb).astype(np.float64)
    x8, s = oracle.quantize_act(xb)
    tab = e4m3_value_table()
    q = x / s[:, None].astype(np.float64)            # Eq. 13 over the reals
    d = tab[x8]
    a = np.minimum(np.abs(q), 448.0)
    step = np.where(a < 2.0 ** -6, 2.0 ** -9, 2.0 ** (np.floor(np.log2(np.maximum(a, 2.0 ** -6))) - 3))
    slack = 4 * np.abs(q) * 2.0 ** -24 + 1e-300     # two fp32 roundings on the way
    assert np.all(np.abs(np.clip(q, -448, 448) - d) <= step / 2 + slack)
    assert np.array_equal(np.sign(d), np.sign(x) * (d != 0))


def test_matches_stated_fp32_steps_via_independent_encoder():
    xb = _x(M=6, K=384, seed=5)
    x = inputs.bf16_bits_to_f32(xb)
    x8, s = oracle.quantize_act(xb)
    inv = np.float32(448) / np.abs(x).max(axis=1)
    q = (x * inv[:, None]).astype(np.float32)        # one fp32 multiply
    assert np.array_equal(x8, e4m3_encode_search(q.astype(np.float64)))


def test_reciprocal_multiply_vs_true_division_differ_by_at_most_one_code():
    xb = _x(M=64, K=2048, seed=6)
    x = inputs.bf16_bits_to_f32(xb)
    x8, s = oracle.quantize_act(xb)
    lit = e4m3_encode_search((x / s[:, None]).astype(np.float32).astype(np.float64))  # literal X/s in fp32
    diff = (x8 != lit)
    assert diff.mean() < 2e-3
    mag = lambda c: (c & 0x7F).astype(np.int32)
    assert np.all(np.abs(mag(x8[diff]) - mag(lit[diff])) <= 1)


def test_power_of_two_mode_is_exact_and_idempotent():
    xb = _x(M=8, K=512, seed=7)
    x = inputs.bf16_bits_to_f32(xb).astype(np.float64)
    x8, s = oracle.quantize_act(xb, scale_mode=1)
    assert np.all(np.log2(s) == np.round(np.log2(s)))
    amax = np.abs(x).max(axis=1)
    assert np.all(s >= amax / 448) and np.all(s / 2 < amax / 448)
    assert np.array_equal(x8, e4m3_encode_search(x / s[:, None]))     # exact quotient, one rounding
    # re-quantizing the dequantized activations (Eq. 4) with the same scale reproduces the codes
    xhat = e4m3_value_table()[x8] * s[:, None]
    assert np.array_equal(e4m3_encode_search(xhat / s[:, None]), x8)


def test_zero_row_and_static_scale():
    xb = _x(M=3, K=256, seed=8)
    xb[1, :] = 0
    x8, s = oracle.quantize_act(xb)
    assert s[1] == 1.0 and np.all(x8[1] == 0)
    x = inputs.bf16_bits_to_f32(xb)
    st = np.float32(0.01)
    x8s, ss = oracle.quantize_act(xb, static_scale=float(st))
    assert np.all(ss == st)
    q = (x * (np.float32(1) / st)).astype(np.float32)
    assert np.array_equal(x8s, e4m3_encode_search(q.astype(np.float64)))
    assert np.any((x8s & 0x7F) == 0x7E)              # the static scale clips the outliers


def test_in_range_agrees_with_library_cast():
    torch = pytest.importorskip("torch")
    xb = _x(M=4, K=512, seed=9)
    x = inputs.bf16_bits_to_f32(xb)
    x8, s = oracle.quantize_act(xb)
    inv = np.float32(448) / np.abs(x).max(axis=1)
    q = torch.from_numpy((x * inv[:, None]).astype(np.float32)).clamp(-448, 448)
    assert np.array_equal(x8, q.to(torch.float8_e4m3fn).view(torch.uint8).numpy())
