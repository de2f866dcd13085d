"""Pins of the W4A16 comparison oracle (Sec. 4.3): the BF16 expansion of the INT4 codes against
hand-computed values (exact cases, a rounding case, a tie), its relation to the FP8 expansion of
Eq. 10 where both are exact, and the matmul against integer arithmetic."""
import struct

import numpy as np

import oracle
from paper_2505_14638_b200 import inputs


def _bf16(v):
    b = struct.unpack("<I", struct.pack("<f", v))[0]
    assert b & 0xFFFF == 0, v
    return b >> 16


def _one_group(codes16, scale, zero=None):
    """A 1 x 128 weight whose first 16 codes are given (the rest are 8)."""
    u = np.full(128, 8, dtype=np.uint8)
    u[:16] = codes16
    packed = (u[0::2] | (u[1::2] << 4)).astype(np.uint8)[None, :]
    gs = np.array([[_bf16(scale)]], dtype=np.uint16)
    gz = None if zero is None else np.array([[zero]], dtype=np.uint8)
    return packed, gs, gz


def test_exact_values_and_nibble_order():
    packed, gs, gz = _one_group(np.arange(16), 0.5)
    w = oracle.bf16_to_f32(oracle.dequant_weight_bf16(packed, gs, gz))[0]
    assert np.array_equal(w[:16], (np.arange(16) - 8) * 0.5)      # even k in the low nibble, z = 8
    assert np.all(w[16:] == 0.0)
    packed, gs, gz = _one_group(np.arange(16), 2.0, zero=3)
    w = oracle.bf16_to_f32(oracle.dequant_weight_bf16(packed, gs, gz))[0]
    assert np.array_equal(w[:16], (np.arange(16) - 3) * 2.0)
    assert np.all(w[16:] == 10.0)


def test_single_rounding_and_tie():
    # s = 1 + 2^-7 (the BF16 neighbour of 1): 7 s = 7.0546875 lies between 7.03125 and 7.0625 (spacing
    # 2^-5 in [4, 8)) and is nearer to 7.0625; 4 s = 4.03125 is representable; 6 s = 6.046875 is a tie
    # between 6.03125 and 6.0625 and goes to the even mantissa (6.0625 = 1.515625 * 4: mantissa 0x42)
    s = 1.0 + 2.0 ** -7
    packed, gs, _ = _one_group(np.array([15, 12, 14, 1] + [8] * 12), s)
    w = oracle.bf16_to_f32(oracle.dequant_weight_bf16(packed, gs))[0]
    assert w[0] == 7.0625 and w[1] == 4.03125 and w[3] == -7.0625
    assert w[2] in (6.03125, 6.0625)
    bits = int(oracle.dequant_weight_bf16(packed, gs)[0, 2])
    assert bits & 1 == 0                                             # tie to even


def test_agrees_with_the_fp8_expansion_where_both_are_exact():
    # power-of-two scales in E4M3's exact range: (u - z) * 2^e is representable in E4M3 and in BF16
    codes, _, gzero = inputs.random_codes(32, 512, 3, asymmetric=True)
    gs = np.full((32, 4), _bf16(0.25), dtype=np.uint16)
    w8 = oracle.e4m3_decode_array(oracle.dequant_weight(codes, gs, gzero)).astype(np.float32)
    w16 = oracle.bf16_to_f32(oracle.dequant_weight_bf16(codes, gs, gzero))
    assert np.array_equal(w8, w16)


def test_matmul_against_integers():
    rng = np.random.default_rng(4)
    codes, _, gzero = inputs.random_codes(24, 256, 9, asymmetric=True)
    gs = np.full((24, 2), _bf16(1.0), dtype=np.uint16)
    xb = inputs.make_small_int_activation(5, 256, 2)
    w16 = oracle.dequant_weight_bf16(codes, gs, gzero)
    y = oracle.linear_w4a16(xb, w16, np.array([0.5], dtype=np.float32))
    u = np.empty((24, 256), dtype=np.int64)
    u[:, 0::2] = codes & 15
    u[:, 1::2] = codes >> 4
    wi = u - np.repeat(gzero.astype(np.int64), 128, axis=1)
    xi = oracle.bf16_to_f32(xb).astype(np.int64)
    assert np.array_equal(y, (xi @ wi.T) * 0.5)
    cols = np.array([3, 17, 5])
    assert np.array_equal(oracle.linear_w4a16(xb, w16, np.arange(24, dtype=np.float32), cols=cols),
                          (xi @ wi.T)[:, cols] * cols[None, :])
    del rng
